"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests touches the CUDA path.  Each one is chosen so that a
plausible slip in the oracle (dropped term, wrong sign/index, transposed
operand, wrong slice of the fused QKV matrix, missing scale) breaks it.
"""
import itertools
import math
import os

import numpy as np
import pytest

import synth
from oracle import marche_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def small_cfg(**kw):
    base = synth.CONFIGS["tiny"].replace(L=3, E=1, D=64, H=4, F=128, S=20, n_buffer=4, B=2, T=4)
    return base.replace(**kw)


def setup(cfg, seed=0):
    blocks = synth.make_weights(cfg, seed=1234 + seed)
    hidden = synth.make_hidden(cfg, seed=2025 + seed)
    return blocks, hidden


def kw(cfg):
    return dict(n_heads=cfg.H, score_layer=cfg.score_layer, ln_eps=cfg.ln_eps)


def fresh_full(cfg, blocks, hidden, new_idx, excl=None, ratio=0.1):
    cache = orc.KVCache(cfg.L, cfg.B, cfg.S, cfg.D)
    out = np.zeros_like(hidden)
    scores, ref = orc.full_step(blocks, hidden, cache, new_idx, excl, ratio, out, **kw(cfg))
    return cache, out, scores, ref


# ---------------------------------------------------------------- sub-steps (textbook values)

def test_layer_norm_textbook():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((5, 32)) * 3 + 100.0          # large mean: cancellation check
    y = orc.layer_norm(x, np.ones(32), np.zeros(32), 0.0)
    assert np.allclose(y.mean(-1), 0, atol=1e-10)
    assert np.allclose(y.var(-1), 1, atol=1e-9)
    # affine part and eps: hand values for a 2-element row (mean 2, biased var 1)
    y2 = orc.layer_norm(np.array([[1.0, 3.0]]), np.array([2.0, 3.0]), np.array([0.5, -0.5]), 3.0)
    assert np.allclose(y2, [[-1.0 / 2.0 * 2.0 + 0.5, 1.0 / 2.0 * 3.0 - 0.5]])


def test_gelu_textbook():
    assert orc.gelu(np.array([0.0]))[0] == 0.0
    # GELU(1) = Phi(1)
    assert abs(orc.gelu(np.array([1.0]))[0] - 0.8413447460685429) < 1e-15
    x = np.linspace(-6, 6, 41)
    assert np.allclose(orc.gelu(x) - orc.gelu(-x), x, atol=1e-14)     # x*Phi(x) - (-x)*Phi(-x) = x
    assert abs(orc.gelu(np.array([40.0]))[0] - 40.0) < 1e-12
    assert abs(orc.gelu(np.array([-40.0]))[0]) < 1e-12
    # differs from the tanh approximation (flavour check)
    tanh_form = 0.5 * 3.0 * (1 + math.tanh(math.sqrt(2 / math.pi) * (3.0 + 0.044715 * 27.0)))
    assert abs(orc.gelu(np.array([3.0]))[0] - tanh_form) > 1e-5


def test_linear_vs_triple_loop():
    rng = np.random.default_rng(1)
    x, W, b = rng.standard_normal((3, 5)), rng.standard_normal((4, 5)), rng.standard_normal(4)
    y = orc.linear(x, W, b)
    for i in range(3):
        for o in range(4):
            acc = b[o]
            for k in range(5):
                acc += x[i, k] * W[o, k]
            assert abs(y[i, o] - acc) < 1e-12


def test_attention_closed_form_two_keys():
    # d = 4, q = (2,0,0,0); k1 = (1,0,0,0), k2 = 0 -> logits (2*1/sqrt 4, 0) = (1, 0)
    q = np.array([[2.0, 0, 0, 0]])
    K = np.array([[1.0, 0, 0, 0], [0, 0, 0, 0]])
    V = np.array([[1.0, 2, 3, 4], [-1.0, 0, 1, 2]])
    z, p = orc.softmax_attention(q, K, V)
    e = math.e
    assert np.allclose(p, [[e / (1 + e), 1 / (1 + e)]], atol=1e-15)
    assert np.allclose(z, (e * V[0] + V[1]) / (1 + e), atol=1e-15)


def test_attention_vs_bruteforce_loops():
    rng = np.random.default_rng(2)
    q, K, V = rng.standard_normal((3, 8)), rng.standard_normal((7, 8)), rng.standard_normal((7, 8))
    z, p = orc.softmax_attention(q, K, V)
    for i in range(3):
        w = [math.exp(sum(q[i, c] * K[j, c] for c in range(8)) / math.sqrt(8)) for j in range(7)]
        tot = sum(w)
        for j in range(7):
            assert abs(p[i, j] - w[j] / tot) < 1e-14
        for c in range(8):
            assert abs(z[i, c] - sum(w[j] / tot * V[j, c] for j in range(7))) < 1e-13


@pytest.mark.parametrize("nA", [0, 1, 5, 12])
def test_two_segment_equals_standard(nA):
    """Eq. 6-10 on a split into A and C equals Eq. 5 on the whole (Appendix A)."""
    rng = np.random.default_rng(3 + nA)
    N, d = 12, 16
    q = rng.standard_normal((4, d)) * 4          # wide logits exercise the shared max
    K, V = rng.standard_normal((N, d)) * 4, rng.standard_normal((N, d))
    perm = rng.permutation(N)
    A, C = perm[:nA], perm[nA:]
    z = orc.two_segment_attention(q, K[A], V[A], K[C], V[C])
    z_ref, _ = orc.softmax_attention(q, K, V)
    assert np.allclose(z, z_ref, rtol=1e-12, atol=1e-13)


def test_large_logits_are_safe():
    rng = np.random.default_rng(4)
    q, K, V = rng.standard_normal((2, 8)) * 200, rng.standard_normal((6, 8)) * 200, rng.standard_normal((6, 8))
    z, p = orc.softmax_attention(q, K, V)
    assert np.isfinite(z).all() and np.allclose(p.sum(-1), 1)


# ---------------------------------------------------------------- whole-step invariants

def test_P1_all_active_equals_full_step():
    cfg = small_cfg()
    blocks, hidden = setup(cfg)
    G = synth.new_token_sets(cfg, synth.generation_orders(cfg))[1]
    cache_f, out_f, sc_f, ref_f = fresh_full(cfg, blocks, hidden, G)
    cache = orc.KVCache(cfg.L, cfg.B, cfg.S, cfg.D)
    out = np.zeros_like(hidden)
    all_idx = np.tile(np.arange(cfg.S, dtype=np.int32), (cfg.B, 1))
    sc, ref = orc.marche_step(blocks, hidden, cache, all_idx, G, None, 0.1, out,
                              require_filled=False, **kw(cfg))
    assert np.array_equal(out, out_f) and np.array_equal(cache.K, cache_f.K)
    assert np.array_equal(cache.V, cache_f.V) and np.array_equal(sc, sc_f) and np.array_equal(ref, ref_f)


def test_step_before_fill_is_an_error():
    cfg = small_cfg()
    blocks, hidden = setup(cfg)
    cache = orc.KVCache(cfg.L, cfg.B, cfg.S, cfg.D)
    idx = np.tile(np.arange(3, dtype=np.int32), (cfg.B, 1))
    with pytest.raises(RuntimeError):
        orc.marche_step(blocks, hidden, cache, idx, idx[:, :1], None, 0.1, np.zeros_like(hidden), **kw(cfg))


def test_P3_idempotence_on_unchanged_input():
    """With exact caches the cache-aware step reproduces the full step (Appendix A)."""
    cfg = small_cfg()
    blocks, hidden = setup(cfg)
    rng = np.random.default_rng(5)
    cache, out_f, _, _ = fresh_full(cfg, blocks, hidden, np.zeros((cfg.B, 0), np.int32))
    before = cache.copy()
    A = np.stack([rng.permutation(cfg.S)[:7] for _ in range(cfg.B)]).astype(np.int32)
    out = np.full_like(hidden, 777.0)
    orc.marche_step(blocks, hidden, cache, A, A[:, :2], None, 0.1, out, **kw(cfg))
    for b in range(cfg.B):
        assert np.allclose(out[b, A[b]], out_f[b, A[b]], rtol=1e-5, atol=1e-6)   # fp32 hidden_out
    assert np.allclose(cache.K, before.K, rtol=1e-10, atol=1e-12)
    assert np.allclose(cache.V, before.V, rtol=1e-10, atol=1e-12)


def test_P4_block0_cache_is_exact_and_P5_untouched_rows():
    cfg = small_cfg()
    blocks, hidden = setup(cfg)
    rng = np.random.default_rng(6)
    cache, _, _, _ = fresh_full(cfg, blocks, hidden, np.zeros((cfg.B, 0), np.int32))
    before = cache.copy()
    A = np.stack([rng.permutation(cfg.S)[:6] for _ in range(cfg.B)]).astype(np.int32)
    hidden2 = hidden.copy()
    for b in range(cfg.B):
        hidden2[b, A[b]] = rng.standard_normal((6, cfg.D))
    out = np.full_like(hidden, 777.0)
    orc.marche_step(blocks, hidden2, cache, A, A[:, :2], None, 0.1, out, **kw(cfg))
    cache_full2, _, _, _ = fresh_full(cfg, blocks, hidden2, np.zeros((cfg.B, 0), np.int32))
    # P4: block 0's K/V depend only on each token's own input row
    assert np.allclose(cache.K[0], cache_full2.K[0], rtol=1e-10, atol=1e-12)
    assert np.allclose(cache.V[0], cache_full2.V[0], rtol=1e-10, atol=1e-12)
    # deeper blocks are stale for cached tokens -> must differ from the full recompute
    assert not np.allclose(cache.K[2], cache_full2.K[2], atol=1e-6)
    # P5: rows outside A byte-identical (cache, every block; hidden_out sentinel)
    for b in range(cfg.B):
        rest = np.setdiff1d(np.arange(cfg.S), A[b])
        assert np.array_equal(cache.K[:, b, rest], before.K[:, b, rest])
        assert np.array_equal(cache.V[:, b, rest], before.V[:, b, rest])
        assert (out[b, rest] == 777.0).all() and (out[b, A[b]] != 777.0).all()
        # active rows did change in every block
        assert not np.array_equal(cache.K[:, b, A[b]], before.K[:, b, A[b]])


def test_P6_score_checksum_and_sign():
    cfg = small_cfg()
    blocks, hidden = setup(cfg)
    G = np.array([[5, 9, 11], [4, 6, 19]], dtype=np.int32)
    _, _, scores, _ = fresh_full(cfg, blocks, hidden, G)
    assert (scores >= 0).all()
    assert np.allclose(scores.sum(-1), cfg.H * G.shape[1], rtol=1e-6)
    # no scoring queries -> all-zero scores -> lowest-index candidates
    _, _, s0, r0 = fresh_full(cfg, blocks, hidden, np.zeros((cfg.B, 0), np.int32), ratio=0.2)
    assert (s0 == 0).all() and np.array_equal(r0, np.tile(np.arange(4, dtype=np.int32), (cfg.B, 1)))


def test_P7_uniform_attention_closed_form():
    cfg = small_cfg(L=1, E=0)
    blocks, hidden = setup(cfg)
    D = cfg.D
    blocks[0]["w_qkv"][:D] = 0
    blocks[0]["b_qkv"][:D] = 0
    G = np.array([[5, 9], [4, 6]], dtype=np.int32)
    X = np.array([[0, 1], [2, 3]], dtype=np.int32)
    cfg1 = cfg.replace()
    cache = orc.KVCache(1, cfg.B, cfg.S, D)
    out = np.zeros_like(hidden)
    scores, ref = orc.full_step(blocks, hidden, cache, G, X, 0.25, out, n_heads=cfg.H, score_layer=0)
    assert np.allclose(scores, cfg.H * 2 / cfg.S, rtol=1e-6)
    # ties -> the k = round(0.25*20) = 5 lowest-index candidates
    assert ref.tolist() == [[2, 3, 4, 6, 7], [0, 1, 5, 7, 8]]
    # O is the column mean of V for every row -> check through the residual wiring
    blk = {k: v.astype(np.float64) for k, v in blocks[0].items()}
    for b in range(cfg.B):
        x = hidden[b].astype(np.float64)
        Vm = cache.V[0, b].mean(axis=0)
        x1 = x + Vm @ blk["w_o"].T + blk["b_o"]
        u2 = orc.layer_norm(x1, blk["ln2_g"], blk["ln2_b"], cfg.ln_eps)
        x2 = x1 + orc.gelu(u2 @ blk["w_fc1"].T + blk["b_fc1"]) @ blk["w_fc2"].T + blk["b_fc2"]
        assert np.allclose(out[b], x2, rtol=1e-5, atol=1e-6)


def test_block_wiring_by_hand():
    """Zero/identity weights make the block's output a closed form that exposes the
    q|k|v slice order, both residual adds and both biases."""
    cfg = small_cfg(L=1, E=0, B=1)
    D, F, S = cfg.D, cfg.F, cfg.S
    rng = np.random.default_rng(8)
    blk = {
        "ln1_g": np.ones(D), "ln1_b": np.zeros(D), "w_qkv": np.zeros((3 * D, D)),
        "b_qkv": np.concatenate([rng.standard_normal(D), rng.standard_normal(D), np.arange(D) * 0.01]),
        "w_o": np.eye(D), "b_o": np.full(D, 0.25), "ln2_g": np.ones(D), "ln2_b": np.zeros(D),
        "w_fc1": np.zeros((F, D)), "b_fc1": np.linspace(-1, 1, F), "w_fc2": np.full((D, F), 0.5),
        "b_fc2": np.full(D, -0.125),
    }
    hidden = rng.standard_normal((1, S, D)).astype(np.float32)
    cache = orc.KVCache(1, 1, S, D)
    out = np.zeros((1, S, D), dtype=np.float64)
    orc.full_step([blk], hidden, cache, np.zeros((1, 0), np.int32), None, 0.0, out, n_heads=cfg.H, score_layer=0)
    b_v = np.arange(D) * 0.01
    ffn = 0.5 * orc.gelu(np.linspace(-1, 1, F)).sum() - 0.125
    expect = hidden[0].astype(np.float64) + b_v + 0.25 + ffn
    assert np.allclose(out[0], expect, rtol=1e-12, atol=1e-12)
    assert np.allclose(cache.V[0, 0], np.tile(b_v, (S, 1)))
    assert np.allclose(cache.K[0, 0], np.tile(blk["b_qkv"][D:2 * D], (S, 1)))


def test_block0_cache_entry_by_explicit_loops():
    """K and V of block 0 for one token, written out with scalar loops."""
    cfg = small_cfg()
    blocks, hidden = setup(cfg)
    cache, _, _, _ = fresh_full(cfg, blocks, hidden, np.zeros((cfg.B, 0), np.int32))
    b, t, D = 1, 7, cfg.D
    x = hidden[b, t].astype(np.float64)
    mu = sum(x) / D
    var = sum((v - mu) ** 2 for v in x) / D
    blk = blocks[0]
    u = [(x[i] - mu) / math.sqrt(var + cfg.ln_eps) * float(blk["ln1_g"][i]) + float(blk["ln1_b"][i]) for i in range(D)]
    for c in (0, 13, D - 1):
        kk = float(blk["b_qkv"][D + c]) + sum(u[i] * float(blk["w_qkv"][D + c, i]) for i in range(D))
        vv = float(blk["b_qkv"][2 * D + c]) + sum(u[i] * float(blk["w_qkv"][2 * D + c, i]) for i in range(D))
        assert abs(cache.K[0, b, t, c] - kk) < 1e-12 and abs(cache.V[0, b, t, c] - vv) < 1e-12


def test_P8_peaked_attention_is_one_hot():
    cfg = small_cfg(L=1, E=0)
    blocks, hidden = setup(cfg)
    blocks = synth.peaked_weights(blocks, cfg, gain=4096.0)
    G = np.array([[5], [6]], dtype=np.int32)
    cache = orc.KVCache(1, cfg.B, cfg.S, cfg.D)
    out = np.zeros_like(hidden)
    scores, _ = orc.full_step(blocks, hidden, cache, G, None, 0.1, out, n_heads=cfg.H, score_layer=0)
    assert np.isfinite(out).all() and np.isfinite(scores).all()
    # each head puts (almost) all its weight on one key: scores are ~integers summing to H
    assert np.allclose(scores, np.round(scores), atol=1e-3)
    assert np.allclose(scores.sum(-1), cfg.H, rtol=1e-6)


def test_P9_full_ratio_reproduces_full_recompute():
    cfg = small_cfg()
    blocks, hidden = setup(cfg)
    sets = synth.new_token_sets(cfg, synth.generation_orders(cfg))
    rep = lambda t, n: synth.replacement_rows(cfg, t, n)
    log_m, cache_m = orc.generate(blocks, hidden, sets, rep, 1.0, mode="marche", **kw(cfg))
    log_f, cache_f = orc.generate(blocks, hidden, sets, rep, 1.0, mode="full", **kw(cfg))
    for a, f in zip(log_m, log_f):
        assert a["active"].shape[1] == cfg.S
        assert np.allclose(a["hidden_out"], f["hidden_out"], rtol=1e-5, atol=1e-6)
        assert np.array_equal(a["refresh"], f["refresh"])
    assert np.allclose(cache_m.K, cache_f.K, rtol=1e-9, atol=1e-11)
    # and a small ratio does drift away from the full recompute (the method is an approximation)
    log_s, _ = orc.generate(blocks, hidden, sets, rep, 0.1, mode="marche", **kw(cfg))
    assert log_s[2]["active"].shape[1] < cfg.S
    assert not np.allclose(log_s[-1]["hidden_out"], log_f[-1]["hidden_out"], atol=1e-4)


def test_P11_order_and_sample_independence():
    cfg = small_cfg()
    blocks, hidden = setup(cfg)
    rng = np.random.default_rng(9)
    cache0, _, _, _ = fresh_full(cfg, blocks, hidden, np.zeros((cfg.B, 0), np.int32))
    A = np.stack([rng.permutation(cfg.S)[:8] for _ in range(cfg.B)]).astype(np.int32)
    G = A[:, 2:5]
    h2 = hidden.copy()
    h2[:, 3] += 1.0
    res = []
    for perm in (np.arange(8), rng.permutation(8)):
        c = cache0.copy()
        out = np.zeros_like(hidden)
        sc, ref = orc.marche_step(blocks, h2, c, A[:, perm], G, None, 0.2, out, **kw(cfg))
        res.append((out, c.K, c.V, sc, ref))
    for x, y in zip(res[0], res[1]):
        assert np.allclose(x, y, rtol=1e-6, atol=1e-7)
    assert np.array_equal(res[0][4], res[1][4])
    # sample independence: perturbing sample 1 leaves sample 0 bit-identical
    h3 = h2.copy()
    h3[1] += 0.5
    c = cache0.copy()
    out = np.zeros_like(hidden)
    sc, ref = orc.marche_step(blocks, h3, c, A, G, None, 0.2, out, **kw(cfg))
    assert np.array_equal(out[0], res[0][0][0]) and np.array_equal(c.K[:, 0], res[0][1][:, 0])
    assert np.array_equal(sc[0], res[0][3][0]) and np.array_equal(ref[0], res[0][4][0])
    assert not np.array_equal(out[1], res[0][0][1])


def test_in_step_selection_schedule_pins():
    """The paper's own schedule (Section 4.2-4.3): with every candidate refreshed it equals a
    full step (Appendix A); the blocks up to the scoring block always hold a fully fresh cache;
    only rows of A change beyond it; the fixed budget fixes #A."""
    cfg = small_cfg(L=4, E=1)                      # score layer 2, blocks 3 cache-aware
    blocks, hidden = setup(cfg)
    sl = cfg.score_layer
    sets = synth.new_token_sets(cfg, synth.generation_orders(cfg))
    G, N = sets[2], sets[1]
    cache0, _, _, _ = fresh_full(cfg, blocks, hidden, np.zeros((cfg.B, 0), np.int32))
    rng = np.random.default_rng(3)
    h2 = hidden.copy()
    for b in range(cfg.B):
        h2[b, N[b]] = rng.standard_normal((N.shape[1], cfg.D))
    cache_f, out_f, sc_f, _ = fresh_full(cfg, blocks, h2, G)
    kws = dict(n_heads=cfg.H, score_layer=sl, ln_eps=cfg.ln_eps)
    # (a) K = every candidate: A = all tokens -> the full step
    c = cache0.copy()
    out = np.zeros_like(hidden)
    k_all = cfg.S - G.shape[1] - N.shape[1]
    sc, R, A = orc.in_step_selection_step(blocks, h2, c, G, N, k_all, out, **kws)
    assert A.shape[1] == cfg.S and np.array_equal(sc, sc_f)
    assert np.allclose(out, out_f, rtol=1e-5, atol=1e-6) and np.allclose(c.K, cache_f.K, rtol=1e-9, atol=1e-11)
    # (b) small K: blocks <= score layer are exactly the full step's, later blocks change only on A
    c = cache0.copy()
    out = np.full_like(hidden, 777.0)
    sc, R, A = orc.in_step_selection_step(blocks, h2, c, G, N, 3, out, **kws)
    assert A.shape[1] == G.shape[1] + N.shape[1] + 3 and np.array_equal(sc, sc_f)
    assert np.array_equal(c.K[: sl + 1], cache_f.K[: sl + 1]) and np.array_equal(c.V[: sl + 1], cache_f.V[: sl + 1])
    for b in range(cfg.B):
        rest = np.setdiff1d(np.arange(cfg.S), A[b])
        assert np.array_equal(c.K[sl + 1:, b, rest], cache0.K[sl + 1:, b, rest])
        assert (out[b, rest] == 777.0).all() and (out[b, A[b]] != 777.0).all()
        # the refreshing tokens are the top-3 by score among tokens outside G u N
        cand = [t for t in range(cfg.S) if t not in set(G[b].tolist()) | set(N[b].tolist())]
        best = sorted(cand, key=lambda t: (-float(sc[b, t]), t))[:3]
        assert sorted(best) == R[b].tolist()
    # (c) forced refresh set is honoured but the selection is still reported
    c2 = cache0.copy()
    forced = np.stack([np.array([t for t in range(cfg.S) if t not in set(G[b].tolist()) | set(N[b].tolist())][:3]) for b in range(cfg.B)]).astype(np.int32)
    sc2, R2, A2 = orc.in_step_selection_step(blocks, h2, c2, G, N, 3, np.zeros_like(hidden), forced_refresh=forced, **kws)
    assert np.array_equal(R2, R) and np.array_equal(A2[:, -3:], forced)
    # (d) whole generation: full step at t = 0 and every 3rd step, fixed budget elsewhere
    log, _ = orc.generate_in_step(blocks, hidden, sets, lambda t, n: synth.replacement_rows(cfg, t, n),
                                  n_heads=cfg.H, score_layer=sl, budget=12, period=3)
    assert [r["kind"] for r in log] == ["full", "in_step", "in_step", "full"]
    assert log[1]["active"].shape[1] == 12 and log[2]["active"].shape[1] == 12


def test_float32_variant_agrees():
    cfg = small_cfg()
    blocks, hidden = setup(cfg)
    G = np.array([[5, 9, 11], [4, 6, 19]], dtype=np.int32)
    outs = []
    for real in (np.float64, np.float32):
        cache = orc.KVCache(cfg.L, cfg.B, cfg.S, cfg.D, real=real)
        out = np.zeros_like(hidden)
        sc, _ = orc.full_step(blocks, hidden, cache, G, None, 0.1, out, real=real, **kw(cfg))
        outs.append((out, sc, cache.K))
    assert np.abs(outs[0][0] - outs[1][0]).max() < 2e-5
    assert np.abs(outs[0][1] - outs[1][1]).max() < 1e-5
    assert np.abs(outs[0][2] - outs[1][2]).max() < 2e-5


# ---------------------------------------------------------------- selection

def brute_force_topk(score, cand, k):
    """All k-subsets; the winner is the one no swap can improve under
    (score desc, index asc).  Tiny inputs only."""
    key = lambda t: (-float(score[t]), t)
    best = None
    for sub in itertools.combinations(cand, k):
        rest = [c for c in cand if c not in sub]
        if all(key(s) < key(r) for s in sub for r in rest):
            assert best is None
            best = sub
    return sorted(best)


@pytest.mark.parametrize("seed", range(6))
def test_P10_topk_vs_bruteforce_tiny(seed):
    rng = np.random.default_rng(seed)
    S = 9
    score = rng.integers(0, 4, size=(1, S)).astype(np.float32)      # many ties
    new = np.array([[int(rng.integers(0, S))]], dtype=np.int32)
    excl = np.array([[int((new[0, 0] + 1 + rng.integers(0, S - 1)) % S)]], dtype=np.int32)
    cand = [t for t in range(S) if t not in (new[0, 0], excl[0, 0])]
    for k in (0, 1, 3, len(cand)):
        got = orc.select_refresh(score, new, excl, k)[0].tolist()
        assert got == (brute_force_topk(score[0], cand, k) if k else [])


@pytest.mark.parametrize("S,k", [(5, 2), (68, 7), (320, 32), (1088, 109), (320, 0), (320, 300)])
def test_P10_topk_vs_stable_argsort(S, k):
    rng = np.random.default_rng(S + k)
    B = 3
    kinds = [rng.random((B, S)), np.ones((B, S)), rng.integers(0, 3, (B, S)).astype(float),
             rng.random((B, S)) * 1e-42, np.exp(rng.uniform(-80, 10, (B, S)))]
    new = np.stack([rng.permutation(S)[:2] for _ in range(B)]).astype(np.int32)
    for sc in kinds:
        sc = sc.astype(np.float32)
        got = orc.select_refresh(sc, new, None, k)
        for b in range(B):
            masked = sc[b].astype(np.float64).copy()
            masked[new[b]] = -1.0                                     # scores are >= 0
            order = np.argsort(-masked, kind="stable")               # ties keep index order
            assert got[b].tolist() == sorted(order[:k].tolist())


def test_selection_ablation_policies():
    rng = np.random.default_rng(11)
    S, B, k = 40, 3, 6
    sc = rng.random((B, S)).astype(np.float32)
    new = np.stack([rng.permutation(S)[:3] for _ in range(B)]).astype(np.int32)
    hi = orc.select_refresh(sc, new, None, k, policy="high")
    lo = orc.select_refresh(sc, new, None, k, policy="low")
    for b in range(B):
        cand = [t for t in range(S) if t not in set(new[b].tolist())]
        assert sorted(sorted(cand, key=lambda t: sc[b, t])[:k]) == lo[b].tolist()
        assert sc[b, lo[b]].max() < sc[b, hi[b]].min()
    # low policy == high policy on negated scores (distinct values)
    assert np.array_equal(lo, orc.select_refresh(1.0 - sc, new, None, k, policy="high"))
    r1 = orc.select_refresh(sc, new, None, k, policy="random", seed=5)
    r2 = orc.select_refresh(sc * 0, new, None, k, policy="random", seed=5)
    r3 = orc.select_refresh(sc, new, None, k, policy="random", seed=6)
    assert np.array_equal(r1, r2) and not np.array_equal(r1, r3)          # scores ignored, seed matters
    for b in range(B):
        assert not set(r1[b].tolist()) & set(new[b].tolist()) and len(set(r1[b].tolist())) == k
    # the hash spreads: over many tokens the selected fraction per half is balanced
    big = orc.select_refresh(np.zeros((1, 1000), np.float32), np.zeros((1, 0), np.int32), None, 500, policy="random", seed=1)
    assert 200 < (big[0] < 500).sum() < 300
    assert orc._mix32(0, 0, 0) == 0 and orc._mix32(1, 2, 3) == orc._mix32(1, 2, 3) and orc._mix32(1, 2, 3) != orc._mix32(1, 3, 2)


def test_random_policy_hash_golden_values_and_inverse():
    """Pins the hash of the random-selection ablation (Section 5.3) to something other than itself:
    (i) two values derived long-hand from the formula printed in include/marche.h, stored with every
    intermediate in tests/golden/random_policy_hash.txt; (ii) the mixing steps are a bijection on 32-bit
    words, so undoing them - xor-shifts unwound, multipliers replaced by their inverses modulo 2^32,
    which are computed here from the header's constants by modular inversion - must return the input
    word; a wrong multiplier, shift amount or step order in the oracle fails one of the two."""
    here = os.path.dirname(os.path.abspath(__file__))
    rows = [ln.split() for ln in open(os.path.join(here, "golden", "random_policy_hash.txt"))
            if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 2
    for seed, b, t, want in rows:
        assert orc._mix32(int(seed, 16), int(b, 16), int(t, 16)) == int(want, 16)

    M = (1 << 32) - 1
    inv1, inv2 = pow(0x7FEB352D, -1, 1 << 32), pow(0x846CA68B, -1, 1 << 32)

    def unshift(y, s):                      # inverse of x ^= x >> s on 32 bits
        x = y
        for _ in range(32 // s + 1):
            x = y ^ (x >> s)
        return x

    rng = np.random.default_rng(3)
    for _ in range(200):
        seed, b, t = (int(v) for v in rng.integers(0, 1 << 32, 3))
        b, t = b % 4096, t % 2048
        x = unshift(orc._mix32(seed, b, t), 16)
        x = (x * inv2) & M
        x = unshift(x, 15)
        x = (x * inv1) & M
        x = unshift(x, 16)
        assert x == (seed ^ (b * 0x9E3779B1) ^ (t * 0x85EBCA77)) & M


def test_topk_signed_zero_and_errors():
    sc = np.array([[0.0, -0.0, 0.0, -0.0]], dtype=np.float32)
    assert orc.select_refresh(sc, np.zeros((1, 0), np.int32), None, 2).tolist() == [[0, 1]]
    with pytest.raises(ValueError):
        orc.select_refresh(sc, np.array([[0]], np.int32), None, 4)


def test_refresh_count_readings():
    assert [orc.refresh_count(r, 320, 10 ** 6) for r in (0, .05, .10, .20)] == [0, 16, 32, 64]
    assert orc.refresh_count(0.10, 1088, 10 ** 6) == 109 and orc.refresh_count(0.10, 68, 10 ** 6) == 7
    assert orc.refresh_count(1.0, 320, 311) == 311


def test_P13_fixed_budget_worked_example():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "fixed_budget_example.txt")) if l.strip() and l[0] != "#"]
    for budget, ng, nn, expect in rows:
        assert orc.fixed_budget_refresh_count(int(budget), int(ng), int(nn)) == int(expect)
    assert orc.fixed_budget_refresh_count(64, 40, 40) == 0


def test_active_set_union():
    G = np.array([[3, 4]], np.int32)
    N = np.array([[7]], np.int32)
    R = np.array([[0, 9]], np.int32)
    assert orc.active_set(G, N, R).tolist() == [[3, 4, 7, 0, 9]]
    with pytest.raises(ValueError):
        orc.active_set(G, N, np.array([[4, 9]], np.int32))


def test_layer_scores_match_the_scoring_block_and_closed_forms():
    """Scores requested at several blocks: at block l they are what a run with score_layer = l
    returns; each obeys the checksum H * #G; a block with zero query weights gives H * #G / S."""
    cfg = small_cfg()
    blocks, hidden = setup(cfg)
    D = cfg.D
    blocks[2]["w_qkv"][:D] = 0
    blocks[2]["b_qkv"][:D] = 0
    G = np.array([[5, 9, 11], [4, 6, 19]], dtype=np.int32)
    per_layer = []
    for l in range(cfg.L):
        cache = orc.KVCache(cfg.L, cfg.B, cfg.S, D)
        s, _ = orc.full_step(blocks, hidden, cache, G, None, 0.0, np.zeros_like(hidden), n_heads=cfg.H, score_layer=l)
        per_layer.append(s)
    want = {0: None, 1: None, 2: None}
    cache = orc.KVCache(cfg.L, cfg.B, cfg.S, D)
    out_a = np.zeros_like(hidden)
    main, ref_a = orc.full_step(blocks, hidden, cache, G, None, 0.2, out_a, n_heads=cfg.H, score_layer=1, layer_scores=want)
    for l in range(cfg.L):
        assert np.array_equal(want[l], per_layer[l])
        assert np.allclose(want[l].sum(-1), cfg.H * G.shape[1], rtol=1e-6)
    assert np.array_equal(main, per_layer[1])
    assert np.allclose(want[2], cfg.H * G.shape[1] / cfg.S, rtol=1e-6)
    assert not np.allclose(want[0], want[1])
    # asking for extra blocks changes neither the outputs nor the selection
    cache_b = orc.KVCache(cfg.L, cfg.B, cfg.S, D)
    out_b = np.zeros_like(hidden)
    main_b, ref_b = orc.full_step(blocks, hidden, cache_b, G, None, 0.2, out_b, n_heads=cfg.H, score_layer=1)
    assert np.array_equal(out_a, out_b) and np.array_equal(ref_a, ref_b) and np.array_equal(cache.K, cache_b.K)
    # cache-aware step: same property on the active rows' queries
    A = np.concatenate([G, np.array([[0, 1], [2, 3]], np.int32)], axis=1)
    w2 = {0: None, 2: None}
    s2, _ = orc.marche_step(blocks, hidden, cache, A, G, None, 0.0, out_a, n_heads=cfg.H, score_layer=1, layer_scores=w2)
    assert np.allclose(w2[0].sum(-1), cfg.H * G.shape[1], rtol=1e-6)
    assert np.allclose(w2[2], cfg.H * G.shape[1] / cfg.S, rtol=1e-6)
