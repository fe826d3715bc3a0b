"""Parity at the full sizes of the benchmark configurations, in the launch configuration
bench.py times: the MAR-L-shaped stack (32 blocks, width 1024, 16 heads, S 320, batch 128) and
likewise MAR-B, MAR-H (head_dim 80) and the high-resolution case (S 1088, batch 64).  The GPU runs the
whole batch; the oracle runs the first and the last classifier-free-guidance pair - samples are
independent (pinned by the oracle's sample-independence test), so their rows must match the
oracle's.  One full step and two cache-aware steps, teacher-forced with the oracle's refresh
sets for the sampled rows (the other rows use the device's own selection, which is itself
compared bit for bit with the oracle's selection on the device's scores)."""
import numpy as np
import pytest
import torch

import synth
from oracle import marche_oracle as orc
from helpers import TOL, dev, idx_dev, make_model, max_abs, rel_l2

pytestmark = pytest.mark.gpu


def _sampled_parity(cfg, ratio, n_steps=3, also_full_recompute=False, operand="f16", bound=None):
    """GPU on the whole batch against the oracle on the first and the last guidance pair
    (rows 0, B/2 and B/2-1, B-1: the last rows sit in the clipped tail tile of every projection).
    `bound` replaces the acceptance bound on hidden rows and cache (index work stays bit-exact).
    Returns the largest max-abs seen on the hidden rows."""
    if torch.cuda.get_device_properties(0).total_memory < 40e9:
        pytest.skip("needs a large GPU")
    half = cfg.B // 2
    rows_s = [0, half, half - 1, cfg.B - 1]            # sampled batch rows
    ratio = float(np.float32(ratio))                   # the C ABI takes a float
    blocks = synth.make_weights(cfg)
    m = make_model(cfg, blocks, operand=operand)
    hidden_np = synth.make_hidden(cfg)
    sets = synth.new_token_sets(cfg, synth.generation_orders(cfg))

    # ---- oracle on the sampled rows
    ns = len(rows_s)
    h2 = hidden_np[rows_s].copy()
    s2 = [g[rows_s] for g in sets]
    cache2 = orc.KVCache(cfg.L, ns, cfg.S, cfg.D)
    out2 = np.zeros_like(h2)
    kw = dict(n_heads=cfg.H, score_layer=cfg.score_layer, ln_eps=cfg.ln_eps)
    recs = []
    sc, R = orc.full_step(blocks, h2, cache2, s2[0], s2[1], ratio, out2, **kw)
    recs.append(dict(active=np.tile(np.arange(cfg.S, dtype=np.int32), (ns, 1)), out=out2.copy(), scores=sc, refresh=R))
    for t in range(1, n_steps):
        rows = synth.replacement_rows(cfg, t - 1, s2[t - 1].shape[1], batch=cfg.B)[rows_s]
        for i in range(ns):
            h2[i, s2[t - 1][i]] = rows[i]
        A = orc.active_set(s2[t], s2[t - 1], R)
        sc, R = orc.marche_step(blocks, h2, cache2, A, s2[t], s2[t + 1], ratio, out2, **kw)
        recs.append(dict(active=A, out=out2.copy(), scores=sc, refresh=R))
    full2 = None
    if also_full_recompute:
        # Appendix A: with every token active the cache-aware step is the full recompute
        full2 = np.zeros_like(h2)
        orc.full_step(blocks, h2, orc.KVCache(cfg.L, ns, cfg.S, cfg.D), s2[n_steps - 1], s2[n_steps], ratio, full2, **kw)
    del blocks

    # ---- device on the whole batch
    B, S, D = cfg.B, cfg.S, cfg.D
    hidden = dev(hidden_np)
    hidden_out = torch.zeros(B, S, D, device="cuda")
    cache = m.alloc_cache()
    ws = m.alloc_workspace(S)
    m.init_cache(cache)
    refresh = torch.zeros(B * S, dtype=torch.int32, device="cuda")
    scores = torch.empty(B, S, device="cuda")
    ma, rl = TOL["bf16"] if bound is None else bound
    k_prev = 0
    worst = 0.0
    for t in range(n_steps):
        G, X = idx_dev(sets[t]), idx_dev(sets[t + 1])
        if t == 0:
            k = m.full_step(hidden, cache, G, X, ratio, hidden_out, refresh, ws)
        else:
            m.scatter_rows(dev(synth.replacement_rows(cfg, t - 1, sets[t - 1].shape[1])), idx_dev(sets[t - 1]), hidden)
            nA = sets[t].shape[1] + sets[t - 1].shape[1] + k_prev
            active = torch.empty(B, nA, dtype=torch.int32, device="cuda")
            m.build_active(G, idx_dev(sets[t - 1]), refresh, k_prev, active)
            assert np.array_equal(active[rows_s].cpu().numpy(), recs[t]["active"])
            k = m.step(hidden, cache, active, G, X, ratio, hidden_out, refresh, ws)
        m.get_scores(ws, scores)
        torch.cuda.synchronize()
        assert m.device_status() == 0
        rec = recs[t]
        assert k == rec["refresh"].shape[1]
        got = hidden_out[rows_s].cpu().numpy()
        for i in range(ns):
            a, w = got[i, rec["active"][i]], rec["out"][i, rec["active"][i]]
            worst = max(worst, max_abs(a, w))
            assert max_abs(a, w) <= ma and rel_l2(a, w) <= rl, \
                "step %d sample %d: max-abs %.3g rel-L2 %.3g" % (t, rows_s[i], max_abs(a, w), rel_l2(a, w))
        unit = cfg.H * sets[t].shape[1] / cfg.S
        assert max_abs(scores[rows_s].cpu().numpy(), rec["scores"]) <= 5e-2 * unit
        # the step's own selection (head-partial reduction + top-K inside the step): bit-exact against
        # the oracle's selection applied to the very scores the device produced, for EVERY batch row
        if k:
            r_dev = refresh[: B * k].view(B, k).cpu().numpy()
            assert np.array_equal(r_dev, orc.select_refresh(scores.cpu().numpy(), sets[t], sets[t + 1], k)), "step %d" % t
        # teacher forcing: the sampled rows continue with the oracle's refresh set
        if k:
            r = refresh[: B * k].view(B, k)
            r[rows_s] = torch.as_tensor(rec["refresh"]).cuda()
        k_prev = k
    if n_steps > 1:
        # run-to-run bit reproducibility at full size (the residual projections use stream-K with ordered
        # reduce-adds here): repeating the last step on the unchanged inputs rewrites the same bytes
        out_again = torch.zeros(B, S, D, device="cuda")
        refresh_again = torch.zeros(B * S, dtype=torch.int32, device="cuda")
        k_again = m.step(hidden, cache, active, G, X, ratio, out_again, refresh_again, ws)
        torch.cuda.synchronize()
        assert k_again == k
        for b in (0, B - 1):
            sel = torch.as_tensor(active[b].cpu().numpy().astype(np.int64))
            assert torch.equal(out_again[b, sel], hidden_out[b, sel])
    Kc = cache[:, 0][:, rows_s].float().cpu().numpy()
    Vc = cache[:, 1][:, rows_s].float().cpu().numpy()
    assert max_abs(Kc, cache2.K) <= ma and rel_l2(Kc, cache2.K) <= rl
    assert max_abs(Vc, cache2.V) <= ma and rel_l2(Vc, cache2.V) <= rl
    if also_full_recompute:
        # device: full step on the same inputs into a second cache; and both against the oracle's full step
        cache_f = m.alloc_cache()
        m.init_cache(cache_f)
        out_f = torch.zeros(B, S, D, device="cuda")
        m.full_step(hidden, cache_f, G, X, ratio, out_f, None, ws)
        torch.cuda.synchronize()
        assert max_abs(out_f[rows_s].cpu().numpy(), full2) <= ma and rel_l2(out_f[rows_s].cpu().numpy(), full2) <= rl
        assert max_abs(hidden_out[rows_s].cpu().numpy(), full2) <= ma
        d = float((out_f - hidden_out).abs().max())
        dk = float((cache_f.float() - cache.float()).abs().max())
        print("all-active step vs full step on the device: hidden max-abs %.3g, cache max-abs %.3g" % (d, dk))
        assert d <= ma / 3 and dk <= ma / 3
    print("full-size parity %s ratio %.2f, %s operands: hidden max-abs %.3g, cache K max-abs %.3g"
          % (cfg.name, ratio, operand, worst, max_abs(Kc, cache2.K)))
    return worst


@pytest.mark.parametrize("name", ["mar_l", "mar_b", "mar_h", "hires"])
def test_full_size_sampled_parity(name):
    cfg = synth.CONFIGS[name]
    _sampled_parity(cfg, cfg.ratio)


@pytest.mark.parametrize("ratio", [0.0, 0.05, 0.2, 1.0])
def test_full_size_refresh_ratio_sweep(ratio):
    """The MAR-L refresh-ratio sweep at full size: ratio 0 (active sets of 2..14 tokens: the smallest attention
    variants), 5 %, 20 % (66..77 tokens) and 100 %, where every token is active in a permuted order and the
    step must equal the full recompute (Appendix A)."""
    _sampled_parity(synth.CONFIGS["mar_l"], ratio, also_full_recompute=(ratio == 1.0))


def test_full_size_all_bf16_operands_recorded(record_property):
    """The MAR-L stack with bf16 projection operands (MARCHE_BF16), all 32 blocks: the rounding of the
    LayerNorm / attention / GELU outputs to bf16 puts the hidden rows outside the 3e-2 bound that the fp16
    operand mode meets, which is why that mode exists.  The figure is recorded, not gated: the test only
    requires that the path runs, stays within a loose sanity bound and keeps its index work exact."""
    cfg = synth.CONFIGS["mar_l"]
    worst = _sampled_parity(cfg, cfg.ratio, operand="bf16", bound=(0.25, 3e-2))
    record_property("all_bf16_hidden_max_abs", worst)
    print("MAR-L, bf16 operands throughout: hidden max-abs %.3g (acceptance bound of the fp16-operand mode: 3e-2)" % worst)


def test_full_size_high_resolution_256_steps():
    """The high-resolution case under its 256-step schedule (1..7 generating tokens per step, 109 refreshing
    tokens: active sets of 111..122 rows, a single query tile of the tcgen05 attention)."""
    _sampled_parity(synth.CONFIGS["hires"].replace(T=256), 0.1)


def test_full_size_two_stage_sampled_parity():
    """The two-stage step (encoder over the known tokens, cache-aware decoder) at the MAR-L shape and
    batch 128: a full-decoder step and two in-step-selection steps with the fixed budget of 64,
    the oracle on one guidance pair, teacher-forced for that pair."""
    from paper_2506_12035_b200.binding import upload_mar_weights
    cfg = synth.CONFIGS["mar_l"]
    if torch.cuda.get_device_properties(0).total_memory < 40e9:
        pytest.skip("needs a large GPU")
    pair = [0, cfg.B // 2]
    budget, n_steps = 64, 3
    blocks = synth.make_weights(cfg)
    mar = synth.make_mar_weights(cfg)
    m = make_model(cfg, blocks)
    m.set_mar_weights(upload_mar_weights(mar, cfg.dtype))
    tokens_np = synth.make_hidden(cfg)
    sets = synth.new_token_sets(cfg, synth.generation_orders(cfg))
    known = synth.known_token_sets(cfg, sets)

    # ---- oracle on the pair
    t2 = tokens_np[pair].copy()
    s2 = [g[pair] for g in sets]
    k2 = [k[pair] for k in known]
    cache2 = orc.KVCache(cfg.L, 2, cfg.S, cfg.D)
    z2 = np.zeros_like(t2)
    kw = dict(n_heads=cfg.H, n_enc=cfg.E, score_layer=cfg.score_layer, ln_eps=cfg.ln_eps)
    recs = []
    for t in range(n_steps):
        if t > 0:
            rows = synth.replacement_rows(cfg, t - 1, s2[t - 1].shape[1], batch=cfg.B)[pair]
            for i in range(2):
                t2[i, s2[t - 1][i]] = rows[i]
        N = s2[t - 1] if t > 0 else None
        kk = 0 if t == 0 else budget - s2[t].shape[1] - s2[t - 1].shape[1]
        sc, R, A = orc.mar_step(blocks, mar, t2, k2[t], cache2, s2[t], N, kk, z2, full_decoder=(t == 0), **kw)
        recs.append(dict(active=A, z=z2.copy(), scores=sc, refresh=R))
    del blocks

    # ---- device on the whole batch
    B, S, D = cfg.B, cfg.S, cfg.D
    tokens = dev(tokens_np)
    z = torch.zeros(B, S, D, device="cuda")
    cache = m.alloc_cache()
    ws = m.alloc_workspace(S)
    m.init_cache(cache)
    scores = torch.empty(B, S, device="cuda")
    ma, rl = TOL["bf16"]
    worst = 0.0
    for t in range(n_steps):
        G, Kn = idx_dev(sets[t]), idx_dev(known[t])
        rec = recs[t]
        if t == 0:
            m.mar_step(True, tokens, Kn, cache, G, None, 0, None, z, None, None, ws)
        else:
            N = idx_dev(sets[t - 1])
            m.scatter_rows(dev(synth.replacement_rows(cfg, t - 1, sets[t - 1].shape[1])), N, tokens)
            k = budget - sets[t].shape[1] - sets[t - 1].shape[1]
            refresh = torch.empty(B, k, dtype=torch.int32, device="cuda")
            active = torch.empty(B, budget, dtype=torch.int32, device="cuda")
            # The device's own selection for the rows the oracle does not cover: a pre-pass with no
            # refreshing tokens leaves the relevance scores in the workspace.  It rewrites only cache
            # rows of G u N, which the real step rewrites again from inputs the pre-pass did not touch.
            m.mar_step(False, tokens, Kn, cache, G, N, 0, None, torch.zeros_like(z), None,
                       torch.empty(B, budget - k, dtype=torch.int32, device="cuda"), ws)
            m.get_scores(ws, scores)
            forced = torch.empty(B, k, dtype=torch.int32, device="cuda")
            m.select_refresh(scores, G, N, k, forced, torch.empty(B * S, dtype=torch.uint8, device="cuda"))
            forced[pair] = torch.as_tensor(rec["refresh"]).cuda()
            m.mar_step(False, tokens, Kn, cache, G, N, k, forced, z, refresh, active, ws)
            assert np.array_equal(active[pair].cpu().numpy(), rec["active"])
        m.get_scores(ws, scores)
        torch.cuda.synchronize()
        assert m.device_status() == 0
        got = z[pair].cpu().numpy()
        for i in range(2):
            a, w = got[i, rec["active"][i]], rec["z"][i, rec["active"][i]]
            worst = max(worst, max_abs(a, w))
            assert max_abs(a, w) <= ma and rel_l2(a, w) <= rl, \
                "step %d sample %d: max-abs %.3g rel-L2 %.3g" % (t, pair[i], max_abs(a, w), rel_l2(a, w))
        unit = cfg.H * sets[t].shape[1] / cfg.S
        assert max_abs(scores[pair].cpu().numpy(), rec["scores"]) <= 5e-2 * unit
    Kc = cache[cfg.E:, 0][:, pair].float().cpu().numpy()
    Vc = cache[cfg.E:, 1][:, pair].float().cpu().numpy()
    assert max_abs(Kc, cache2.K[cfg.E:]) <= ma and rel_l2(Kc, cache2.K[cfg.E:]) <= rl
    assert max_abs(Vc, cache2.V[cfg.E:]) <= ma and rel_l2(Vc, cache2.V[cfg.E:]) <= rl
    print("two-stage full-size parity: z max-abs %.3g" % worst)
