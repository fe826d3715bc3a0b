"""End-to-end parity of marche_step / marche_full_step with the CPU oracle, teacher-forced:
both sides are driven with the oracle's index sets at every step, and per step the
active rows of hidden_out, the relevance scores and (at the end) every cache layer are
compared.  Plus the invariants that hold at any size and the error behaviour."""
import numpy as np
import pytest
import torch

import synth
from oracle import marche_oracle as orc
from paper_2506_12035_b200.binding import MarcheError
from paper_2506_12035_b200.generation import Generation
from helpers import TOL, assert_close, cache_to_oracle_layout, dev, host, idx_dev, make_model, max_abs, rel_l2

pytestmark = pytest.mark.gpu

CASES = {
    # the fp32 configuration of the benchmark list, whole 8-step generation
    "tiny_f32": synth.CONFIGS["tiny"],
    # same stack in bf16
    "tiny_bf16": synth.CONFIGS["tiny"].replace(dtype="bf16"),
    # MAR-B-shaped rows (D 768, 12 heads, S 320), cut down in depth, batch and steps
    "marb_slice": synth.CONFIGS["mar_b"].replace(L=3, E=1, B=4, T=6),
    # head_dim 80 (MAR-H-shaped rows)
    "marh_slice": synth.CONFIGS["mar_h"].replace(L=2, E=0, B=2, T=4),
    # the same 16-bit stacks with bf16 projection operands (MARCHE_BF16) instead of fp16 ones
    "tiny_bf16_bf16op": synth.CONFIGS["tiny"].replace(dtype="bf16"),
    "marb_slice_bf16op": synth.CONFIGS["mar_b"].replace(L=3, E=1, B=4, T=6),
}
OPERAND = {name: ("bf16" if name.endswith("_bf16op") else "f16") for name in CASES}


def oracle_run(cfg, blocks, hidden0, ratio, mode="marche"):
    sets = synth.new_token_sets(cfg, synth.generation_orders(cfg))
    rep = lambda t, n: synth.replacement_rows(cfg, t, n)
    log, cache = orc.generate(blocks, hidden0, sets, rep, ratio, n_heads=cfg.H, score_layer=cfg.score_layer,
                              ln_eps=cfg.ln_eps, mode=mode)
    return sets, log, cache


def gpu_generation(cfg, blocks, sets, ratio, operand="f16"):
    m = make_model(cfg, blocks, operand=operand)
    rows = [dev(synth.replacement_rows(cfg, t, sets[t].shape[1])) for t in range(cfg.T)]
    return m, Generation(m, sets, ratio, rows)


@pytest.mark.parametrize("case", list(CASES))
@pytest.mark.parametrize("ratio", [0.10, 0.0])
def test_teacher_forced_generation(case, ratio):
    cfg = CASES[case]
    if ratio == 0.0 and case != "tiny_bf16":
        pytest.skip("zero-refresh variant runs on one case")
    blocks = synth.make_weights(cfg)
    hidden0 = synth.make_hidden(cfg)
    sets, log, cache = oracle_run(cfg, blocks, hidden0, ratio)
    m, gen = gpu_generation(cfg, blocks, sets, ratio, OPERAND[case])
    forced = [idx_dev(rec["refresh"]) for rec in log]
    glog = gen.run(dev(hidden0), record=True, forced_refresh=forced)
    assert m.device_status() == 0
    mask = torch.empty(cfg.B * cfg.S, dtype=torch.uint8, device="cuda")
    for rec, g in zip(log, glog):
        A = rec["active"]
        assert g["n_active"] == A.shape[1]
        if g["active"] is not None:
            assert np.array_equal(g["active"], A)                      # device-built A = G u N u R
        for b in range(cfg.B):
            assert_close(g["hidden_out"][b, A[b]], rec["hidden_out"][b, A[b]], cfg.dtype,
                         "%s step %d hidden_out" % (case, rec["t"]))
        nG = rec["new"].shape[1]
        unit = cfg.H * nG / cfg.S                                      # mean score
        assert max_abs(g["scores"], rec["scores"]) <= (5e-2 if cfg.dtype == "bf16" else 1e-4) * unit
        assert np.allclose(g["scores"].sum(-1), cfg.H * nG, rtol=1e-3)
        # the step's own selection (head-partial reduction + top-K at the end of the step), taken before
        # the teacher forcing: bit-exact against the oracle's selection on the device's own scores
        k = rec["refresh"].shape[1]
        assert g["refresh_own"].shape == (cfg.B, k)
        if k:
            assert np.array_equal(g["refresh_own"],
                                  orc.select_refresh(g["scores"], rec["new"], rec["exclude"] if rec["exclude"].shape[1] else None, k))
        # selection: fed the oracle's fp32 scores, the device's top-k is bit-exact
        if k:
            out = torch.empty(cfg.B, k, dtype=torch.int32, device="cuda")
            excl = rec["exclude"]
            m.select_refresh(dev(rec["scores"]), idx_dev(rec["new"]), idx_dev(excl) if excl.shape[1] else None,
                             k, out, mask)
            assert np.array_equal(out.cpu().numpy(), rec["refresh"])
    K, V = cache_to_oracle_layout(gen.cache)
    assert_close(K, cache.K, cfg.dtype, case + " cache K")
    assert_close(V, cache.V, cfg.dtype, case + " cache V")


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_invariants_untouched_rows_full_equivalence_reproducibility(dtype):
    cfg = synth.CONFIGS["tiny"].replace(dtype=dtype, B=3)
    blocks = synth.make_weights(cfg)
    m = make_model(cfg, blocks)
    rng = np.random.default_rng(0)
    B, S, D = cfg.B, cfg.S, cfg.D
    hidden = dev(synth.make_hidden(cfg))
    cache = m.alloc_cache()
    ws = m.alloc_workspace(S)
    out_full = torch.zeros(B, S, D, device="cuda")
    refresh = torch.zeros(B, S, dtype=torch.int32, device="cuda")
    A = np.stack([rng.permutation(S)[:9] for _ in range(B)]).astype(np.int32)
    G = A[:, :3]
    # a step on a never-filled cache is an error and enqueues nothing
    m.init_cache(cache)
    with pytest.raises(MarcheError) as e:
        m.step(hidden, cache, idx_dev(A), idx_dev(G), None, 0.1, out_full, refresh, ws)
    assert e.value.code == -4
    k_full = m.full_step(hidden, cache, idx_dev(G), None, 0.1, out_full, refresh, ws)
    sc_full = torch.empty(B, S, device="cuda")
    m.get_scores(ws, sc_full)
    cache_full = cache.clone()

    # P5: rows outside A are byte-identical after a cache-aware step (sentinel in hidden_out)
    hidden2 = hidden.clone()
    for b in range(B):
        # (not a constant shift: LayerNorm would remove it and leave K, V unchanged)
        hidden2[b, torch.as_tensor(A[b], dtype=torch.long)] = torch.randn(A.shape[1], D, device="cuda")
    out = torch.full((B, S, D), 777.0, device="cuda")
    m.step(hidden2, cache, idx_dev(A), idx_dev(G), None, 0.1, out, refresh, ws)
    torch.cuda.synchronize()
    for b in range(B):
        rest = torch.as_tensor(np.setdiff1d(np.arange(S), A[b]), dtype=torch.long)
        act = torch.as_tensor(A[b], dtype=torch.long)
        assert torch.equal(cache[:, :, b, rest], cache_full[:, :, b, rest])
        assert not torch.equal(cache[:, :, b, act], cache_full[:, :, b, act])
        assert (out[b, rest] == 777.0).all() and (out[b, act] != 777.0).all()

    # P1/P3: active = every token (any order) reproduces the full step
    cache2 = m.alloc_cache()
    m.init_cache(cache2)
    out_b = torch.zeros(B, S, D, device="cuda")
    m.full_step(hidden, cache2, idx_dev(G), None, 0.1, out_b, refresh, ws)
    perm = np.stack([rng.permutation(S) for _ in range(B)]).astype(np.int32)
    out_c = torch.zeros(B, S, D, device="cuda")
    refresh_c = torch.zeros(B, S, dtype=torch.int32, device="cuda")
    k_c = m.step(hidden, cache2, idx_dev(perm), idx_dev(G), None, 0.1, out_c, refresh_c, ws)
    sc_c = torch.empty(B, S, device="cuda")
    m.get_scores(ws, sc_c)
    tol = 2e-2 if dtype == "bf16" else 1e-5
    assert max_abs(host(out_c), host(out_full)) <= tol
    assert max_abs(host(cache2), host(cache_full)) <= tol
    assert max_abs(host(sc_c), host(sc_full)) <= 1e-3 and k_c == k_full

    # run-to-run bit reproducibility (scores use a fixed-order reduction, no atomics)
    res = []
    for _ in range(2):
        c3 = cache_full.clone()
        m.init_cache(c3)
        o3 = torch.zeros(B, S, D, device="cuda")
        r3 = torch.zeros(B, S, dtype=torch.int32, device="cuda")
        m.full_step(hidden, c3, idx_dev(G), None, 0.1, o3, r3, ws)
        m.step(hidden2, c3, idx_dev(A), idx_dev(G), None, 0.1, o3, r3, ws)
        s3 = torch.empty(B, S, device="cuda")
        m.get_scores(ws, s3)
        res.append((o3.clone(), c3, s3, r3.clone()))
    for x, y in zip(*res):
        assert torch.equal(x, y)


@pytest.mark.parametrize("B,nA", [(8, 41), (16, 45), (4, 27)])
def test_untouched_cache_rows_byte_identical_under_fused_write_back(B, nA):
    """Rows outside the active set keep their bytes (Algorithm 1 line 11 touches only rows of A) on the
    production path, where the QKV projection's epilogue writes K and V straight into the cache (more than
    128 rows: 328 and 720, the latter with a ragged last row tile); 108 rows take the separate write-back
    kernel.  Every cache layer and hidden_out are compared byte for byte; the active rows must change."""
    cfg = synth.CONFIGS["mar_b"].replace(L=3, E=1, B=B, T=6)
    blocks = synth.make_weights(cfg)
    m = make_model(cfg, blocks)
    rng = np.random.default_rng(B)
    S, D = cfg.S, cfg.D
    hidden = dev(synth.make_hidden(cfg))
    cache = m.alloc_cache()
    ws = m.alloc_workspace(S)
    m.init_cache(cache)
    out = torch.zeros(B, S, D, device="cuda")
    refresh = torch.zeros(B, S, dtype=torch.int32, device="cuda")
    A = np.stack([rng.permutation(S)[:nA] for _ in range(B)]).astype(np.int32)
    G = A[:, :5]
    m.full_step(hidden, cache, idx_dev(G), None, 0.1, out, refresh, ws)
    torch.cuda.synchronize()
    before = cache.clone()
    hidden2 = hidden.clone()
    for b in range(B):
        hidden2[b, torch.as_tensor(A[b], dtype=torch.long)] = torch.randn(nA, D, device="cuda")
    out2 = torch.full((B, S, D), 777.0, device="cuda")
    m.step(hidden2, cache, idx_dev(A), idx_dev(G), None, 0.1, out2, refresh, ws)
    torch.cuda.synchronize()
    assert m.device_status() == 0
    for b in range(B):
        rest = torch.as_tensor(np.setdiff1d(np.arange(S), A[b]), dtype=torch.long)
        act = torch.as_tensor(A[b], dtype=torch.long)
        assert torch.equal(cache[:, :, b, rest].view(torch.int16), before[:, :, b, rest].view(torch.int16))
        changed = (cache[:, :, b, act].view(torch.int16) != before[:, :, b, act].view(torch.int16)).any(-1)
        assert bool(changed.all())                      # every active row of every layer, K and V, was rewritten
        assert (out2[b, rest] == 777.0).all() and (out2[b, act] != 777.0).all()


def test_full_ratio_equals_full_recompute():
    """Refresh ratio 100 %: every step's active set is all tokens, so the cache-aware
    generation equals the full-recompute generation (Appendix A)."""
    cfg = synth.CONFIGS["tiny"].replace(dtype="bf16")
    blocks = synth.make_weights(cfg)
    hidden0 = dev(synth.make_hidden(cfg))
    sets = synth.new_token_sets(cfg, synth.generation_orders(cfg))
    m, gen = gpu_generation(cfg, blocks, sets, 1.0)
    log_m = gen.run(hidden0, mode="marche", record=True)
    cache_m = gen.cache.clone()
    log_f = gen.run(hidden0, mode="full", record=True)
    for a, f in zip(log_m, log_f):
        assert a["n_active"] == cfg.S
        assert max_abs(a["hidden_out"], f["hidden_out"]) <= 2e-2
        assert rel_l2(a["hidden_out"], f["hidden_out"]) <= 2e-3
    assert max_abs(host(cache_m), host(gen.cache)) <= 2e-2


@pytest.mark.parametrize("case", ["tiny_f32", "tiny_bf16", "marb_slice"])
def test_in_step_selection_schedule(case):
    """The paper's own schedule (full attention up to the scoring block, selection there,
    cache-aware blocks after it; fixed active budget; periodic full refresh), teacher-forced
    with the oracle's refresh sets."""
    cfg = CASES[case]
    if cfg.score_layer >= cfg.L - 1:
        cfg = cfg.replace(E=cfg.E - 1)
    budget = 24 if cfg.S < 100 else 64
    blocks = synth.make_weights(cfg)
    hidden0 = synth.make_hidden(cfg)
    sets = synth.new_token_sets(cfg, synth.generation_orders(cfg))
    log, cache = orc.generate_in_step(blocks, hidden0, sets, lambda t, n: synth.replacement_rows(cfg, t, n),
                                      n_heads=cfg.H, score_layer=cfg.score_layer, budget=budget, period=3,
                                      ln_eps=cfg.ln_eps)
    m, gen = gpu_generation(cfg, blocks, sets, 0.0)
    forced = [idx_dev(r["refresh"]) if r["kind"] == "in_step" and r["refresh"].shape[1] else None for r in log]
    glog = gen.run_in_step(dev(hidden0), budget=budget, period=3, record=True, forced_refresh=forced)
    assert m.device_status() == 0
    mask = torch.empty(cfg.B * cfg.S, dtype=torch.uint8, device="cuda")
    for rec, g in zip(log, glog):
        A = rec["active"]
        assert g["n_active"] == A.shape[1]
        if rec["kind"] == "in_step":
            assert np.array_equal(g["active"], A)
            assert A.shape[1] == min(budget, cfg.S) or rec["new"].shape[1] + rec["prev"].shape[1] >= budget
        for b in range(cfg.B):
            assert_close(g["hidden_out"][b, A[b]], rec["hidden_out"][b, A[b]], cfg.dtype,
                         "%s step %d (%s)" % (case, rec["t"], rec["kind"]))
        nG = rec["new"].shape[1]
        unit = cfg.H * nG / cfg.S
        assert max_abs(g["scores"], rec["scores"]) <= (5e-2 if cfg.dtype == "bf16" else 1e-4) * unit
        k = rec["refresh"].shape[1]
        if k:   # fed the oracle's scores, the device's selection is bit-exact
            out = torch.empty(cfg.B, k, dtype=torch.int32, device="cuda")
            m.select_refresh(dev(rec["scores"]), idx_dev(rec["new"]), idx_dev(rec["prev"]), k, out, mask)
            assert np.array_equal(out.cpu().numpy(), rec["refresh"])
    K, V = cache_to_oracle_layout(gen.cache)
    assert_close(K, cache.K, cfg.dtype, case + " cache K")
    assert_close(V, cache.V, cfg.dtype, case + " cache V")


def test_host_driven_step_matches_device_loop():
    """marche_step_host (inputs and results in host buffers) reproduces the device-resident
    loop bit for bit: same kernels, same order; only the copies differ."""
    cfg = synth.CONFIGS["tiny"].replace(dtype="bf16")
    blocks = synth.make_weights(cfg)
    hidden0 = synth.make_hidden(cfg)
    sets = synth.new_token_sets(cfg, synth.generation_orders(cfg))
    rows = [synth.replacement_rows(cfg, t, sets[t].shape[1]) for t in range(cfg.T)]
    m, gen = gpu_generation(cfg, blocks, sets, 0.1)
    log = gen.run(dev(hidden0), record=True)
    gen.alloc_host_buffers(hidden0, rows, sets)
    h2d, d2h = gen.run_host()
    torch.cuda.synchronize()
    assert h2d > hidden0.nbytes and d2h > 0
    for t, rec in enumerate(log):
        for b in range(cfg.B):
            assert np.array_equal(gen.h_out_rows[t][b].numpy(), rec["hidden_out"][b, sets[t][b]])
    k = log[-1]["refresh"].shape[1]
    assert np.array_equal(gen.h_refresh[: cfg.B * k].view(cfg.B, k).numpy(), log[-1]["refresh"])
    # profiling hooks: every launch is charged to a class, and the counter agrees
    n0 = m.launch_count()
    m.profile_begin()
    gen.run(dev(hidden0))
    prof = m.profile_end()
    assert sum(v[1] for v in prof.values()) == m.launch_count() - n0
    assert prof["attention"][1] == cfg.L * cfg.T and prof["gemm_qkv"][1] == cfg.L * cfg.T
    assert all(v[0] >= 0 for v in prof.values())


def test_argument_errors():
    cfg = synth.CONFIGS["tiny"]
    blocks = synth.make_weights(cfg)
    m = make_model(cfg, blocks)
    B, S, D = cfg.B, cfg.S, cfg.D
    hidden = dev(synth.make_hidden(cfg))
    out = torch.zeros(B, S, D, device="cuda")
    cache = m.alloc_cache()
    m.init_cache(cache)
    small_ws = m.alloc_workspace(4)
    refresh = torch.zeros(B, S, dtype=torch.int32, device="cuda")
    G = idx_dev(np.array([[4, 5], [6, 7]]))
    with pytest.raises(MarcheError) as e:
        m.full_step(hidden, cache, G, None, 0.1, out, refresh, small_ws)
    assert e.value.code == -3
    ws = m.alloc_workspace(S)
    with pytest.raises(MarcheError) as e:
        m.full_step(hidden, cache, G, None, 0.1, hidden, refresh, ws)          # out aliases in
    assert e.value.code == -1
    m.full_step(hidden, cache, G, None, 0.1, out, refresh, ws)
    with pytest.raises(MarcheError) as e:                                       # n_new > n_active
        m.step(hidden, cache, idx_dev(np.array([[4], [6]])), G, None, 0.1, out, refresh, ws)
    assert e.value.code == -1
    from paper_2506_12035_b200.binding import Marche, upload_weights
    with pytest.raises(MarcheError) as e:                                       # width not a multiple of 128
        Marche(L=1, E=0, D=192, H=3, F=128, S=8, B=1, dtype="f32", weights=upload_weights(blocks[:1], "f32"))
    assert e.value.code == -2


@pytest.mark.parametrize("case", ["tiny_f32", "marb_slice"])
def test_scores_at_several_blocks(case):
    """Extra scoring blocks (for the top-K overlap statistics across layers): each block's scores
    match the oracle's, the step's outputs and its selection do not change, and the overlap of the
    per-block top-K sets can be computed from them."""
    cfg = CASES[case]
    blocks = synth.make_weights(cfg)
    hidden0 = synth.make_hidden(cfg)
    sets = synth.new_token_sets(cfg, synth.generation_orders(cfg))
    G, X = sets[0], sets[1]
    layers = list(range(cfg.L))
    want = {l: None for l in layers}
    cache_o = orc.KVCache(cfg.L, cfg.B, cfg.S, cfg.D)
    out_o = np.zeros_like(hidden0)
    s_o, r_o = orc.full_step(blocks, hidden0, cache_o, G, X, cfg.ratio, out_o, n_heads=cfg.H, score_layer=cfg.score_layer,
                             ln_eps=cfg.ln_eps, layer_scores=want)

    m_plain = make_model(cfg, blocks)
    m = make_model(cfg, blocks)
    ws_plain = m_plain.alloc_workspace(cfg.S)
    m.set_score_layers(layers)
    ws = m.alloc_workspace(cfg.S)
    assert ws.numel() > ws_plain.numel()
    outs = []
    for mm, w in ((m_plain, ws_plain), (m, ws)):
        cache = mm.alloc_cache()
        mm.init_cache(cache)
        out = torch.zeros(cfg.B, cfg.S, cfg.D, device="cuda")
        refresh = torch.zeros(cfg.B * cfg.S, dtype=torch.int32, device="cuda")
        k = mm.full_step(dev(hidden0), cache, idx_dev(G), idx_dev(X), cfg.ratio, out, refresh, w)
        outs.append((out, refresh[: cfg.B * k].clone(), cache))
    if cfg.dtype == "f32":      # one attention kernel: registering blocks changes nothing at all
        assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1]) and torch.equal(outs[0][2], outs[1][2])
    else:                       # the scoring flavour of the tensor-core kernel is two-pass: same values within rounding
        assert_close(host(outs[1][0]), host(outs[0][0]), cfg.dtype, "outputs with extra scoring blocks")
    assert_close(host(outs[1][0]), out_o, cfg.dtype, "outputs vs oracle")
    unit = cfg.H * G.shape[1] / cfg.S
    lim = (5e-2 if cfg.dtype == "bf16" else 1e-4) * unit
    sc = torch.empty(cfg.B, cfg.S, device="cuda")
    per_layer = {}
    for l in layers:
        m.get_layer_scores(ws, l, sc)
        per_layer[l] = sc.cpu().numpy().copy()
        assert max_abs(per_layer[l], want[l]) <= lim, l
        assert np.allclose(per_layer[l].sum(-1), cfg.H * G.shape[1], rtol=2e-3)
    m.get_scores(ws, sc)
    assert np.array_equal(sc.cpu().numpy(), per_layer[cfg.score_layer])
    # top-K overlap between two blocks from the device's scores, via the device's selection
    k = 7
    mask = torch.empty(cfg.B * cfg.S, dtype=torch.uint8, device="cuda")
    tops = []
    for l in (layers[0], layers[-1]):
        out = torch.empty(cfg.B, k, dtype=torch.int32, device="cuda")
        m.select_refresh(dev(per_layer[l]), idx_dev(G), None, k, out, mask)
        assert np.array_equal(out.cpu().numpy(), orc.select_refresh(per_layer[l], G, None, k))
        tops.append(out.cpu().numpy())
    overlap = np.mean([len(set(a) & set(b)) / k for a, b in zip(*tops)])
    assert 0.0 <= overlap <= 1.0
    # a block that was not registered is refused; clearing the list restores the plain workspace size
    with pytest.raises(MarcheError):
        m_plain.get_layer_scores(ws_plain, (cfg.score_layer + 1) % cfg.L, sc)
    m.set_score_layers([])
    assert m.workspace_bytes(cfg.S) == m_plain.workspace_bytes(cfg.S)


def _one_step_pair(cfg, blocks, hidden0, G0, A, G, X, ratio):
    """Full step then one cache-aware step on both sides; returns (oracle, device) results."""
    kw = dict(n_heads=cfg.H, score_layer=cfg.score_layer, ln_eps=cfg.ln_eps)
    cache_o = orc.KVCache(cfg.L, cfg.B, cfg.S, cfg.D)
    out_o = np.zeros_like(hidden0)
    orc.full_step(blocks, hidden0, cache_o, G0, None, ratio, out_o, **kw)
    full_o = out_o.copy()
    s_o, r_o = orc.marche_step(blocks, hidden0, cache_o, A, G, X, ratio, out_o, **kw)
    m = make_model(cfg, blocks)
    cache = m.alloc_cache()
    ws = m.alloc_workspace(cfg.S)
    m.init_cache(cache)
    out = torch.zeros(cfg.B, cfg.S, cfg.D, device="cuda")
    refresh = torch.full((cfg.B * cfg.S,), -1, dtype=torch.int32, device="cuda")
    h = dev(hidden0)
    m.full_step(h, cache, idx_dev(G0), None, ratio, out, refresh, ws)
    full_d = out.cpu().numpy().copy()
    k = m.step(h, cache, idx_dev(A), None if G.shape[1] == 0 else idx_dev(G), None if X is None else idx_dev(X), ratio,
               out, refresh, ws)
    sc = torch.empty(cfg.B, cfg.S, device="cuda")
    m.get_scores(ws, sc)
    torch.cuda.synchronize()
    assert m.device_status() == 0
    return (full_o, out_o, s_o, r_o, cache_o), (full_d, out.cpu().numpy(), sc.cpu().numpy(),
                                                 refresh[: cfg.B * k].view(cfg.B, k).cpu().numpy(), cache)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_degenerate_active_sets(dtype):
    """One active token; no generating token at all (all scores zero, so the selection falls back
    to the lowest-index candidates); an active set that is every token but one."""
    cfg = synth.CONFIGS["tiny"].replace(dtype=dtype)
    blocks = synth.make_weights(cfg)
    hidden0 = synth.make_hidden(cfg)
    B, S = cfg.B, cfg.S
    G0 = np.array([[5, 9], [4, 6]], dtype=np.int32)
    empty = np.zeros((B, 0), dtype=np.int32)
    cases = [
        (np.array([[17], [33]], np.int32), np.array([[17], [33]], np.int32), None, 0.1),          # nA = nG = 1
        (np.array([[17, 3], [33, 8]], np.int32), empty, np.array([[0], [1]], np.int32), 0.1),     # nG = 0
        (np.stack([np.delete(np.arange(S, dtype=np.int32), 11), np.delete(np.arange(S, dtype=np.int32), 60)]),
         np.array([[1, 2, 3], [4, 5, 6]], np.int32), None, 0.0),                                   # nA = S - 1, k = 0
    ]
    for A, G, X, ratio in cases:
        (fo, oo, so, ro, co), (fd, od, sd, rd, cd) = _one_step_pair(cfg, blocks, hidden0, G0, A, G, X, ratio)
        for b in range(B):
            assert_close(od[b, A[b]], oo[b, A[b]], dtype, "active rows")
            rest = np.setdiff1d(np.arange(S), A[b])
            assert np.array_equal(od[b, rest], fd[b, rest])                # rows outside A keep the full step's bytes
        unit = cfg.H * max(G.shape[1], 1) / S
        assert max_abs(sd, so) <= (5e-2 if dtype == "bf16" else 1e-4) * unit
        assert rd.shape == ro.shape
        if G.shape[1] == 0:
            assert (sd == 0).all() and np.array_equal(rd, ro)              # ties -> lowest indices, bit-exact
        K, V = cache_to_oracle_layout(cd)
        assert_close(K, co.K, dtype, "cache K")
        assert_close(V, co.V, dtype, "cache V")


@pytest.mark.parametrize("shape", ["S2048", "D2048"])
def test_maximum_sizes(shape):
    """The largest sequence length and the largest width the library accepts (one block, bf16)."""
    base = synth.CONFIGS["tiny"].replace(dtype="bf16", L=1, E=0, B=2, T=4)
    cfg = base.replace(S=2048, n_buffer=64, D=128, H=2, F=256) if shape == "S2048" else \
        base.replace(S=72, n_buffer=8, D=2048, H=32, F=2048)
    blocks = synth.make_weights(cfg)
    hidden0 = synth.make_hidden(cfg)
    rng = np.random.default_rng(3)
    perm = np.stack([rng.permutation(cfg.S) for _ in range(cfg.B)]).astype(np.int32)
    G0, G, N = perm[:, :5], perm[:, 5:9], perm[:, 9:40]
    A = np.concatenate([G, N], axis=1)
    (fo, oo, so, ro, co), (fd, od, sd, rd, cd) = _one_step_pair(cfg, blocks, hidden0, G0, A, G, None, 0.05)
    assert_close(fd, fo, "bf16", "full step")
    for b in range(cfg.B):
        assert_close(od[b, A[b]], oo[b, A[b]], "bf16", "active rows")
    assert max_abs(sd, so) <= 5e-2 * cfg.H * G.shape[1] / cfg.S
    assert rd.shape == ro.shape == (cfg.B, int(np.floor(0.05 * cfg.S + 0.5)))
    K, V = cache_to_oracle_layout(cd)
    assert_close(K, co.K, "bf16", "cache K")
    assert_close(V, co.V, "bf16", "cache V")
    m = make_model(cfg, blocks)
    mask = torch.empty(cfg.B * cfg.S, dtype=torch.uint8, device="cuda")
    out = torch.empty(cfg.B, rd.shape[1], dtype=torch.int32, device="cuda")
    m.select_refresh(dev(so), idx_dev(G), None, rd.shape[1], out, mask)
    assert np.array_equal(out.cpu().numpy(), ro)


def test_generation_replayed_from_a_cuda_graph():
    """A generation recorded in a CUDA graph writes the same bytes as the eager one."""
    cfg = CASES["marb_slice"]
    blocks = synth.make_weights(cfg)
    hidden0 = dev(synth.make_hidden(cfg))
    sets = synth.new_token_sets(cfg, synth.generation_orders(cfg))
    m, gen = gpu_generation(cfg, blocks, sets, cfg.ratio)
    gen.run(hidden0)
    torch.cuda.synchronize()
    want_out, want_cache = gen.hidden_out.clone(), gen.cache.clone()
    graph = gen.capture(hidden0)
    gen.hidden_out.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert m.device_status() == 0
    assert torch.equal(gen.hidden_out, want_out) and torch.equal(gen.cache, want_cache)
