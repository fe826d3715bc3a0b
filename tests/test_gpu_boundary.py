"""Boundary behaviour of the C ABI beyond the arithmetic: a bounded device wait that runs out and the
MARCHE_ETIMEOUT it produces, the kernel-selection switches (every alternative computes the same
step), the refusal of misaligned operands in 16-bit contexts, the saturation rule of the fp16
operand mode, and the library's own conversion of unrounded weights."""
import numpy as np
import pytest
import torch

import synth
from oracle import marche_oracle as orc
from paper_2506_12035_b200 import binding
from paper_2506_12035_b200.binding import MarcheError
from helpers import TOL, dev, host, idx_dev, make_model, max_abs, rel_l2

pytestmark = pytest.mark.gpu


def _one_step(m, cfg, hidden, A, G, ratio=0.1):
    B, S, D = cfg.B, cfg.S, cfg.D
    cache = m.alloc_cache()
    ws = m.alloc_workspace(S)
    m.init_cache(cache)
    out = torch.zeros(B, S, D, device="cuda")
    refresh = torch.zeros(B * S, dtype=torch.int32, device="cuda")
    m.full_step(hidden, cache, idx_dev(G), None, ratio, out, refresh, ws)
    out2 = torch.zeros(B, S, D, device="cuda")
    k = m.step(hidden, cache, idx_dev(A), idx_dev(G), None, ratio, out2, refresh, ws)
    scores = torch.empty(B, S, device="cuda")
    m.get_scores(ws, scores)
    torch.cuda.synchronize()
    return out2, cache, refresh[: B * k].view(B, k).clone(), scores


def test_bounded_wait_runs_out_and_is_reported_as_timeout():
    """A wait on a barrier nothing arrives on gives up after its cycle limit: the kernel returns, the
    status word is set, the synchronous calls answer MARCHE_ETIMEOUT, and after clearing the word the
    context computes a correct step again (nothing trapped, nothing hung)."""
    cfg = synth.CONFIGS["tiny"].replace(dtype="bf16", B=4)
    blocks = synth.make_weights(cfg)
    m = make_model(cfg, blocks)
    assert m.device_status() == 0
    m.check_status()                                                   # clean: no exception
    m.debug_bounded_wait(1_000_000)                                    # about half a millisecond
    with pytest.raises(MarcheError) as e:
        m.check_status()
    assert e.value.code == -7
    assert m.device_status() != 0
    act = np.array([[1, 2, 3, 4]] * cfg.B, np.int32)
    with pytest.raises(MarcheError) as e:                              # the other synchronous calls report it too
        m.validate_indices(idx_dev(act), idx_dev(act[:, :2]), None)
    assert e.value.code == -7
    with pytest.raises(MarcheError) as e:
        m.debug_bounded_wait(0)                                        # limit out of range: nothing enqueued
    assert e.value.code == -1
    m.clear_device_status()
    assert m.device_status() == 0
    m.check_status()
    # the context is fully usable: a step against the oracle
    rng = np.random.default_rng(0)
    hidden_np = synth.make_hidden(cfg)
    A = np.stack([rng.permutation(cfg.S)[:9] for _ in range(cfg.B)]).astype(np.int32)
    G = A[:, :3]
    out, cache, _, _ = _one_step(m, cfg, dev(hidden_np), A, G)
    oc = orc.KVCache(cfg.L, cfg.B, cfg.S, cfg.D)
    want = np.zeros_like(hidden_np)
    kw = dict(n_heads=cfg.H, score_layer=cfg.score_layer, ln_eps=cfg.ln_eps)
    orc.full_step(blocks, hidden_np, oc, G, None, 0.1, want, **kw)
    orc.marche_step(blocks, hidden_np, oc, A, G, None, 0.1, want, **kw)
    for b in range(cfg.B):
        assert max_abs(host(out)[b, A[b]], want[b, A[b]]) <= TOL["bf16"][0]
    assert m.device_status() == 0


def test_tuning_alternatives_compute_the_same_step():
    """Every switch of marche_tuning only selects a kernel: the step's outputs stay within the parity
    bound of the oracle and the refresh selection on the device's own scores stays bit-exact."""
    cfg = synth.CONFIGS["mar_b"].replace(L=2, E=0, B=8, T=6)
    blocks = synth.make_weights(cfg)
    m = make_model(cfg, blocks)
    defaults = m.get_tuning()
    assert defaults == dict(stream_k=1, fuse_qkv_scatter=1, attention_kernel=0, attention_tc_min_rows=48,
                            two_segment_attention=0, gemm_kernel=0, tail_split=1, tile_n=0, pdl=1)
    rng = np.random.default_rng(1)
    hidden_np = synth.make_hidden(cfg)
    nA = 41
    A = np.stack([rng.permutation(cfg.S)[:nA] for _ in range(cfg.B)]).astype(np.int32)
    G = A[:, :5]
    oc = orc.KVCache(cfg.L, cfg.B, cfg.S, cfg.D)
    want = np.zeros_like(hidden_np)
    kw = dict(n_heads=cfg.H, score_layer=cfg.score_layer, ln_eps=cfg.ln_eps)
    orc.full_step(blocks, hidden_np, oc, G, None, 0.1, want, **kw)
    orc.marche_step(blocks, hidden_np, oc, A, G, None, 0.1, want, **kw)
    hidden = dev(hidden_np)
    ma, rl = TOL["bf16"]
    variants = [dict(), dict(fuse_qkv_scatter=0), dict(two_segment_attention=1), dict(attention_kernel=binding.ATTENTION_TCGEN05),
                dict(attention_kernel=binding.ATTENTION_TCGEN05_TWO_PASS),
                dict(attention_kernel=binding.ATTENTION_MMA, attention_tc_min_rows=8), dict(gemm_kernel=binding.GEMM_SINGLE),
                dict(gemm_kernel=binding.GEMM_PAIR, tile_n=128), dict(stream_k=0, tail_split=0), dict(tail_split=4), dict(pdl=0)]
    for v in variants:
        m.set_tuning(**defaults)
        m.set_tuning(**v)
        out, cache, R, scores = _one_step(m, cfg, hidden, A, G)
        assert m.device_status() == 0, v
        for b in range(cfg.B):
            assert max_abs(host(out)[b, A[b]], want[b, A[b]]) <= ma and rel_l2(host(out)[b, A[b]], want[b, A[b]]) <= rl, v
        assert max_abs(host(cache[:, 0]), oc.K) <= ma and max_abs(host(cache[:, 1]), oc.V) <= ma, v
        assert np.array_equal(R.cpu().numpy(), orc.select_refresh(scores.cpu().numpy(), G, None, R.shape[1])), v
    m.set_tuning(**defaults)
    for bad in (dict(attention_kernel=4), dict(gemm_kernel=-1), dict(tail_split=3), dict(tile_n=64)):
        with pytest.raises(MarcheError) as e:
            m.set_tuning(**bad)
        assert e.value.code == -1
    assert m.get_tuning() == defaults


def test_misaligned_operands_are_refused_in_16bit_contexts():
    """There is no slower fall-back kernel behind the tensor-core path: an operand that TMA cannot address
    is an argument error that names the rule, and nothing is enqueued."""
    cfg = synth.CONFIGS["tiny"].replace(dtype="bf16", L=1, E=0)
    m = make_model(cfg, synth.make_weights(cfg))
    M, N, K = 40, 256, 256
    a = torch.zeros(M * K + 8, dtype=torch.float16, device="cuda")
    w = torch.zeros(N, K, dtype=torch.float16, device="cuda")
    bias = torch.zeros(N, device="cuda")
    out = torch.full((M, N), 3.0, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(MarcheError) as e:
        m.linear(a[1:1 + M * K].view(M, K), w, bias, 0, out)              # 2-byte offset
    assert e.value.code == -1 and "16-byte" in str(e.value)
    q = torch.zeros(2 * 4 * 3 * cfg.D + 8, dtype=torch.bfloat16, device="cuda")
    cache = torch.zeros(2, cfg.B, cfg.S, cfg.D, dtype=torch.bfloat16, device="cuda")
    o = torch.full((cfg.B * 4, cfg.D), 3.0, dtype=torch.float16, device="cuda")
    with pytest.raises(MarcheError) as e:
        m.attention(q[1:], 3 * cfg.D, 4, cache, None, None, o)
    assert e.value.code == -1
    torch.cuda.synchronize()
    assert (out == 3.0).all() and (o == 3.0).all()


@pytest.mark.parametrize("operand", ["f16", "bf16"])
def test_activation_range_rule(operand):
    """fp16 operand mode: an activation beyond the fp16 range is stored as +-65504 (the header's range rule),
    never as infinity.  Attention over V rows of magnitude 1e5 (which the bf16 cache holds) must give exactly
    65504 per output element; LayerNorm with a gain of 1e5 and GELU of 1e5 likewise.  The bf16 operand mode
    has the range for these values and returns them."""
    cfg = synth.CONFIGS["tiny"].replace(dtype="bf16", L=1, E=0, B=2)
    m = make_model(cfg, synth.make_weights(cfg), operand=operand)
    adt = torch.float16 if operand == "f16" else torch.bfloat16
    B, S, D, n = cfg.B, cfg.S, cfg.D, 5
    big = 1.0e5
    cache = torch.zeros(2, B, S, D, dtype=torch.bfloat16, device="cuda")
    cache[1] = big
    cache[1, :, :, ::2] = -big
    o = torch.zeros(B * n, D, dtype=adt, device="cuda")
    m.attention(torch.randn(B * n, D, device="cuda").to(torch.bfloat16), D, n, cache, None, None, o)
    # LayerNorm: rows of +-1 normalise to +-1, times a gain of 1e5
    x = torch.ones(B, S, D, device="cuda")
    x[:, :, ::2] = -1.0
    u = torch.zeros(B * n, D, dtype=adt, device="cuda")
    m.gather_layernorm(x, None, n, torch.full((D,), big, device="cuda"), torch.zeros(D, device="cuda"), None, u)
    # GELU epilogue: acc = 0, bias = 1e5 -> GELU(1e5) = 1e5
    g = torch.zeros(B * n, 256, dtype=adt, device="cuda")
    m.linear(torch.zeros(B * n, 256, dtype=adt, device="cuda"), torch.zeros(256, 256, dtype=adt, device="cuda"),
             torch.full((256,), big, device="cuda"), 2, g)
    torch.cuda.synchronize()
    for t in (o, u, g):
        assert torch.isfinite(t.float()).all()
    if operand == "f16":
        assert (o.float().abs() == 65504.0).all() and (o.float()[:, 1::2] > 0).all() and (o.float()[:, ::2] < 0).all()
        assert (u.float().abs() == 65504.0).all() and (g.float() == 65504.0).all()
    else:
        for t in (o, u, g):
            assert ((t.float().abs() - big).abs() <= big * 2.0 ** -8).all()
    assert m.device_status() == 0


def test_unrounded_fp32_weights_are_converted_by_the_library_side():
    """Weights that were never rounded to a 16-bit grid: the oracle computes with the fp32 values, the
    device with whatever the binding's cast to the operand type made of them (including the fp16
    subnormal range below 6.1e-5, where about 0.2 % of N(0, 0.02) weights fall), and the step still
    meets the bound.  The conversion error is inside the measured difference, where it belongs."""
    cfg = synth.CONFIGS["mar_b"].replace(L=3, E=1, B=4, T=6)
    blocks = synth.make_weights(cfg.replace(dtype="f32"))               # same recipe without the bf16 rounding
    w = blocks[0]["w_qkv"]
    assert not np.array_equal(w, synth.round_to_bf16(w)) and (np.abs(w) < 6.1e-5).mean() > 1e-3
    hidden_np = synth.make_hidden(cfg)
    rng = np.random.default_rng(2)
    A = np.stack([rng.permutation(cfg.S)[:41] for _ in range(cfg.B)]).astype(np.int32)
    G = A[:, :5]
    oc = orc.KVCache(cfg.L, cfg.B, cfg.S, cfg.D)
    want = np.zeros_like(hidden_np)
    kw = dict(n_heads=cfg.H, score_layer=cfg.score_layer, ln_eps=cfg.ln_eps)
    orc.full_step(blocks, hidden_np, oc, G, None, 0.1, want, **kw)
    orc.marche_step(blocks, hidden_np, oc, A, G, None, 0.1, want, **kw)
    ma, rl = TOL["bf16"]
    for operand in ("f16", "bf16"):
        m = make_model(cfg, blocks, operand=operand)
        out, cache, _, _ = _one_step(m, cfg, dev(hidden_np), A, G)
        worst = max(max_abs(host(out)[b, A[b]], want[b, A[b]]) for b in range(cfg.B))
        print("unrounded weights, %s operands: hidden max-abs %.3g" % (operand, worst))
        assert worst <= ma
        assert max_abs(host(cache[:, 0]), oc.K) <= ma and max_abs(host(cache[:, 1]), oc.V) <= ma


def test_context_is_bound_to_its_device():
    """A context used while another device is current is an argument error, not a launch on the wrong GPU."""
    if torch.cuda.device_count() < 2:
        pytest.skip("needs two devices")
    cfg = synth.CONFIGS["tiny"].replace(L=1, E=0)
    with torch.cuda.device(0):
        m = make_model(cfg, synth.make_weights(cfg))
        sc = torch.zeros(cfg.B, cfg.S, device="cuda")
        out = torch.full((cfg.B, 3), -1, dtype=torch.int32, device="cuda")
    with torch.cuda.device(1):
        with pytest.raises(MarcheError) as e:
            m.select_refresh_static(sc, None, None, 3, out)
        assert e.value.code == -1 and "device" in str(e.value)
    with torch.cuda.device(0):
        torch.cuda.synchronize()
        assert (out == -1).all()


def test_measurement_hooks_change_launches_only_as_documented():
    """marche_debug_repeat_classes / marche_debug_skip_classes: doubling the idempotent classes (LayerNorm, QKV
    projection, attention, fc1) leaves the step's results bit-identical and adds exactly one launch per launch of
    the class; leaving a class out removes its launches; other classes are refused."""
    cfg = synth.CONFIGS["mar_b"].replace(L=2, E=0, B=8, T=6)
    blocks = synth.make_weights(cfg)
    m = make_model(cfg, blocks)
    rng = np.random.default_rng(4)
    hidden = dev(synth.make_hidden(cfg))
    A = np.stack([rng.permutation(cfg.S)[:41] for _ in range(cfg.B)]).astype(np.int32)
    G = A[:, :5]
    n0 = m.launch_count()
    out_ref, cache_ref, R_ref, _ = _one_step(m, cfg, hidden, A, G)
    per_step = m.launch_count() - n0
    idem = ["gather_layernorm", "gemm_qkv", "attention", "gemm_fc1_gelu"]
    m.debug_repeat_classes(idem)
    n0 = m.launch_count()
    out_rep, cache_rep, R_rep, _ = _one_step(m, cfg, hidden, A, G)
    assert m.launch_count() - n0 == per_step + 2 * cfg.L * 5           # two calls (full step, step): LN x2, qkv, attention, fc1
    assert torch.equal(out_rep, out_ref) and torch.equal(cache_rep, cache_ref) and torch.equal(R_rep, R_ref)
    m.debug_repeat_classes(())
    m.debug_skip_classes(["attention"])
    n0 = m.launch_count()
    _one_step(m, cfg, hidden, A, G)
    assert m.launch_count() - n0 == per_step - 2 * cfg.L
    m.debug_skip_classes(())
    with pytest.raises(MarcheError) as e:
        m.debug_skip_classes(["topk"])
    assert e.value.code == -1
    out_again, _, _, _ = _one_step(m, cfg, hidden, A, G)
    assert torch.equal(out_again, out_ref) and m.device_status() == 0
