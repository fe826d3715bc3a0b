"""Per-kernel parity: each C-ABI kernel call against the matching oracle sub-step on the
same seeded inputs (small and odd shapes spanning several tiles and ragged tails)."""
import math

import numpy as np
import pytest
import torch

import synth
from oracle import marche_oracle as orc
from helpers import (TOL, assert_close, dev, host, idx_dev, make_model, max_abs, rel_l2)

pytestmark = pytest.mark.gpu


def model_for(dtype, D, H, F, S, B, L=1):
    """dtype "f32", "bf16" (bf16 cache, fp16 projection operands) or "bf16b" (bf16 throughout)."""
    cfg = synth.CONFIGS["tiny"].replace(L=L, E=0, D=D, H=H, F=F, S=S, B=B, dtype="f32" if dtype == "f32" else "bf16",
                                        n_buffer=0)
    blocks = synth.make_weights(cfg)
    return cfg, blocks, make_model(cfg, blocks, operand="bf16" if dtype == "bf16b" else "f16")


def tdt(dtype):
    """element type of q/k/v and the K/V cache"""
    return torch.float32 if dtype == "f32" else torch.bfloat16


def adt(dtype):
    """element type of the projections' operands: weight matrices and the activations that feed them"""
    return {"f32": torch.float32, "bf16": torch.float16, "bf16b": torch.bfloat16}[dtype]


def quant_a(a, dtype):
    """What the device holds for a projection operand."""
    a = np.asarray(a, np.float32)
    if dtype == "bf16":
        return a.astype(np.float16).astype(np.float64)
    return synth.round_to_bf16(a).astype(np.float64) if dtype == "bf16b" else a.astype(np.float64)


def quant(a, dtype):
    """What the device holds for q/k/v and cache entries."""
    return np.asarray(a, np.float32).astype(np.float64) if dtype == "f32" else synth.round_to_bf16(a).astype(np.float64)


LOW = ("bf16", "bf16b")        # the 16-bit contexts


# ------------------------------------------------------------------ K1 gather + LayerNorm
@pytest.mark.parametrize("dtype", ["f32", "bf16", "bf16b"])
@pytest.mark.parametrize("D,H", [(256, 4), (768, 12), (1024, 16), (1280, 16)])
@pytest.mark.parametrize("n", [1, 2, 41, 68])
def test_gather_layernorm(dtype, D, H, n):
    S, B = 68, 3
    cfg, blocks, m = model_for(dtype, D, H, 128, S, B)
    rng = np.random.default_rng(n + D)
    hidden = rng.standard_normal((B, S, D)).astype(np.float32)
    hidden[0] += 100.0                                   # large mean: variance cancellation
    patterns = [np.stack([rng.permutation(S)[:n] for _ in range(B)]),
                np.tile(np.arange(S - 1, S - 1 - n, -1), (B, 1))]
    g, be = blocks[0]["ln1_g"], blocks[0]["ln1_b"]
    for idx in patterns:
        x_out = torch.full((B * n, D), -7.0, device="cuda")
        u_out = torch.zeros(B * n, D, dtype=adt(dtype), device="cuda")
        m.gather_layernorm(dev(hidden), idx_dev(idx), n, dev(g), dev(be), x_out, u_out)
        X = np.stack([hidden[b, idx[b]] for b in range(B)]).reshape(B * n, D)
        assert np.array_equal(x_out.cpu().numpy(), X)                       # the gather is a copy: exact
        want = orc.layer_norm(X.astype(np.float64), g.astype(np.float64), be.astype(np.float64), cfg.ln_eps)
        assert_close(host(u_out), want, dtype, "LN", scale=1.0 if dtype in LOW else 10.0)
    # identity index (idx NULL), no compact copy
    u_out = torch.zeros(B * n, D, dtype=adt(dtype), device="cuda")
    m.gather_layernorm(dev(hidden), None, n, dev(g), dev(be), None, u_out)
    want = orc.layer_norm(hidden[:, :n].reshape(B * n, D).astype(np.float64), g.astype(np.float64),
                          be.astype(np.float64), cfg.ln_eps)
    assert_close(host(u_out), want, dtype, "LN identity", scale=1.0 if dtype in LOW else 10.0)


# ------------------------------------------------------------------ K2 projections
@pytest.mark.parametrize("dtype", ["f32", "bf16", "bf16b"])
@pytest.mark.parametrize("M", [1, 24, 62, 129, 300])
@pytest.mark.parametrize("N,K", [(768, 256), (256, 256), (1024, 256), (256, 1024), (384, 128), (128, 320)])
def test_linear_all_epilogues(dtype, M, N, K):
    cfg, blocks, m = model_for(dtype, 256, 4, 1024, 68, 2)
    rng = np.random.default_rng(M * 7 + N + K)
    a = rng.standard_normal((M, K)).astype(np.float32)
    w = (rng.standard_normal((N, K)) * 0.05).astype(np.float32)
    bias = rng.standard_normal(N).astype(np.float32)
    aq, wq = quant_a(a, dtype), quant_a(w, dtype)
    acc = orc.linear(aq, wq, bias.astype(np.float64))
    a_d, w_d, b_d = dev(a, adt(dtype)), dev(w, adt(dtype)), dev(bias)
    ma, rl = TOL[dtype]
    # bias
    out = torch.zeros(M, N, dtype=tdt(dtype), device="cuda")
    m.linear(a_d, w_d, b_d, 0, out)
    assert rel_l2(host(out), acc) <= (4e-3 if dtype in LOW else 1e-6)
    assert max_abs(host(out), acc) <= (3e-2 if dtype in LOW else 1e-4)
    # bias + residual (fp32 read-modify-write)
    res = rng.standard_normal((M, N)).astype(np.float32)
    out = dev(res)
    m.linear(a_d, w_d, b_d, 1, out)
    assert max_abs(host(out), acc + res) <= 1e-4 * max(1.0, math.sqrt(K / 256))
    # bias + GELU
    out = torch.zeros(M, N, dtype=adt(dtype), device="cuda")
    m.linear(a_d, w_d, b_d, 2, out)
    want = orc.gelu(acc)
    assert rel_l2(host(out), want) <= (4e-3 if dtype in LOW else 1e-6)
    assert max_abs(host(out), want) <= (3e-2 if dtype in LOW else 1e-4)


@pytest.mark.parametrize("dtype", ["bf16", "bf16b"])
def test_gelu_epilogue_over_the_whole_input_range(dtype):
    """The GELU of the tensor-core epilogue (a polynomial for erf, saturating beyond |x| = 3 sqrt 2) against the
    oracle's erf GELU on a dense grid: a selection matrix as the weight and the grid as bias make the accumulator
    equal the grid value exactly, so the only differences are the approximation and the 16-bit rounding of the
    result.  Grid: -12 .. 12 in steps of 1/512 (covers the fitted range, the clamp point and the saturated tails),
    plus large magnitudes up to the fp16 maximum."""
    cfg, blocks, m = model_for(dtype, 256, 4, 1024, 68, 2)
    M, N, K = 128, 12288 + 128, 64
    grid = np.concatenate([np.arange(-12.0, 12.0, 1.0 / 512.0),
                           np.array([-65000.0, -1000.0, -100.0, -13.0, 13.0, 100.0, 1000.0, 60000.0]),
                           np.zeros(120)]).astype(np.float32)
    assert grid.shape[0] == N
    a = np.zeros((M, K), np.float32)                                    # accumulator = bias exactly
    w = np.zeros((N, K), np.float32)
    out = torch.zeros(M, N, dtype=adt(dtype), device="cuda")
    m.linear(dev(a, adt(dtype)), dev(w, adt(dtype)), dev(grid), 2, out)
    torch.cuda.synchronize()
    got = host(out)
    assert (got == got[0:1]).all()                                      # every row the same function of the bias
    want = orc.gelu(grid.astype(np.float64))
    if dtype == "bf16":                                                 # fp16 result: saturates at 65504
        want = np.clip(want, -65504.0, 65504.0)
    eps = 2.0 ** -11 if dtype == "bf16" else 2.0 ** -8                  # half an ulp, relative
    err = np.abs(got[0] - want)
    bound = eps * np.abs(want) + 1.0e-4                                 # rounding + the approximation (<= 4.8e-5)
    worst = int(np.argmax(err - bound))
    assert (err <= bound).all(), "x = %g: got %g, want %g" % (grid[worst], got[0][worst], want[worst])
    assert (got[0][grid <= -13.0] == 0).all() and np.isfinite(got).all()


@pytest.mark.parametrize("dtype", ["f32", "bf16", "bf16b"])
def test_linear_strided_input_and_row_guard(dtype):
    """a is a column slice of a wider matrix (lda > K); rows >= M of `out` stay untouched."""
    cfg, blocks, m = model_for(dtype, 256, 4, 1024, 68, 2)
    rng = np.random.default_rng(5)
    M, N, K = 70, 256, 256
    wide = rng.standard_normal((M, 3 * K)).astype(np.float32)
    w = (rng.standard_normal((N, K)) * 0.05).astype(np.float32)
    bias = rng.standard_normal(N).astype(np.float32)
    wide_d = dev(wide, adt(dtype))
    out = torch.full((M + 60, N), 5.0, dtype=tdt(dtype), device="cuda")
    m.linear(wide_d[:, K:2 * K], dev(w, adt(dtype)), dev(bias), 0, out, M=M, lda=3 * K)
    want = orc.linear(quant_a(wide[:, K:2 * K], dtype), quant_a(w, dtype), bias.astype(np.float64))
    assert rel_l2(host(out[:M]), want) <= (4e-3 if dtype in LOW else 1e-6)
    assert (host(out[M:]) == 5.0).all()


# ------------------------------------------------------------------ K5 scatter
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("n", [1, 7, 41])
def test_scatter_kv_and_untouched_rows(dtype, n):
    S, B, D = 68, 3, 256
    cfg, blocks, m = model_for(dtype, D, 4, 128, S, B)
    rng = np.random.default_rng(n)
    qkv = dev(rng.standard_normal((B * n, 3 * D)).astype(np.float32), tdt(dtype))
    cache = dev(rng.standard_normal((2, B, S, D)).astype(np.float32), tdt(dtype))
    before = cache.clone()
    idx = np.stack([rng.permutation(S)[:n] for _ in range(B)]).astype(np.int32)
    m.scatter_kv(qkv[:, D:], qkv[:, 2 * D:], 3 * D, idx_dev(idx), n, cache)
    torch.cuda.synchronize()
    want = before.clone()
    q3 = qkv.view(B, n, 3 * D)
    for b in range(B):
        want[0, b, torch.as_tensor(idx[b], dtype=torch.long)] = q3[b, :, D:2 * D]
        want[1, b, torch.as_tensor(idx[b], dtype=torch.long)] = q3[b, :, 2 * D:]
    assert torch.equal(cache, want)                                     # byte-identical everywhere


def test_scatter_rows_and_build_active():
    S, B, D = 68, 3, 256
    cfg, blocks, m = model_for("f32", D, 4, 128, S, B)
    rng = np.random.default_rng(0)
    rows = dev(rng.standard_normal((B, 5, D)).astype(np.float32))
    idx = np.stack([rng.permutation(S)[:5] for _ in range(B)]).astype(np.int32)
    dst = torch.full((B, S, D), 3.0, device="cuda")
    m.scatter_rows(rows, idx_dev(idx), dst)
    want = torch.full((B, S, D), 3.0, device="cuda")
    for b in range(B):
        want[b, torch.as_tensor(idx[b], dtype=torch.long)] = rows[b]
    assert torch.equal(dst, want)
    G, N, R = idx[:, :2], idx[:, 2:3], idx[:, 3:]
    act = torch.zeros(B, 5, dtype=torch.int32, device="cuda")
    m.build_active(idx_dev(G), idx_dev(N), idx_dev(R), 2, act)
    assert np.array_equal(act.cpu().numpy(), orc.active_set(G, N, R))
    act2 = torch.zeros(B, 2, dtype=torch.int32, device="cuda")
    m.build_active(idx_dev(G), None, None, 0, act2)
    assert np.array_equal(act2.cpu().numpy(), G)


# ------------------------------------------------------------------ K3 attention (+ scores)
@pytest.mark.parametrize("dtype", ["f32", "bf16", "bf16b"])
@pytest.mark.parametrize("S", [68, 320])
@pytest.mark.parametrize("dh,H", [(64, 4), (80, 2)])
@pytest.mark.parametrize("n,nG", [(1, 1), (2, 0), (12, 7), (41, 25), (77, 77)])
def test_attention_and_score_partials(dtype, S, dh, H, n, nG):
    if n > S:
        pytest.skip("n > S")
    B, D = 2, dh * H
    if D % 128:
        H = {64: 4, 80: 8}[dh]
        D = dh * H
    cfg, blocks, m = model_for(dtype, D, H, 128, S, B)
    rng = np.random.default_rng(S + n + dh)
    gain = 3.0                                                       # logits of order a few units
    q = (rng.standard_normal((B * n, 3 * D)) * gain).astype(np.float32)
    cache = rng.standard_normal((2, B, S, D)).astype(np.float32)
    flags = np.zeros((B, n), dtype=np.uint8)
    for b in range(B):
        flags[b, rng.permutation(n)[:nG]] = 1
    q_d = dev(q, tdt(dtype))
    o = torch.zeros(B * n, D, dtype=adt(dtype), device="cuda")
    partial = torch.full((B, H, S), -1.0, device="cuda")
    m.attention(q_d, 3 * D, n, dev(cache, tdt(dtype)), dev(flags), partial, o)
    qq, cc = quant(q, dtype), quant(cache, dtype)
    want_o = np.zeros((B * n, D))
    want_p = np.zeros((B, H, S))
    for b in range(B):
        for h in range(H):
            c = slice(h * dh, (h + 1) * dh)
            z, p = orc.softmax_attention(qq[b * n:(b + 1) * n, c], cc[0, b][:, c], cc[1, b][:, c])
            want_o[b * n:(b + 1) * n, c] = z
            want_p[b, h] = p[flags[b].astype(bool)].sum(axis=0)
    got_o, got_p = host(o), host(partial)
    assert rel_l2(got_o, want_o) <= (8e-3 if dtype in LOW else 1e-5)
    assert max_abs(got_o, want_o) <= (3e-2 if dtype in LOW else 1e-4)
    assert max_abs(got_p, want_p) <= (2e-2 if dtype in LOW else 1e-5) * max(1, nG) / 8 + 1e-6
    assert np.allclose(got_p.sum(-1), nG, rtol=(5e-3 if dtype in LOW else 1e-5), atol=1e-6)   # each row sums to 1
    # scores off: partial buffer untouched
    partial2 = torch.full((B, H, S), -1.0, device="cuda")
    m.attention(q_d, 3 * D, n, dev(cache, tdt(dtype)), None, partial2, o)
    assert (partial2 == -1.0).all()


@pytest.mark.parametrize("S", [68, 320, 1088])
@pytest.mark.parametrize("dh,H", [(64, 4), (80, 8)])
@pytest.mark.parametrize("n,nG", [(1, 1), (12, 7), (41, 5), (77, 0), (130, 25)])
def test_two_segment_attention_equals_scatter_then_attend(S, dh, H, n, nG):
    """The two-segment kernel (Eq. 6-10 + write-back) against the oracle's plain attention over
    the updated cache, and bit-exact cache contents against marche_scatter_kv."""
    if n > S:
        pytest.skip("n > S")
    B, D = 2, dh * H
    cfg, blocks, m = model_for("bf16", D, H, 128, S, B)
    rng = np.random.default_rng(S + n + dh)
    qkv = (rng.standard_normal((B * n, 3 * D)) * np.array([3.0] * D + [1.0] * 2 * D)).astype(np.float32)
    cache = rng.standard_normal((2, B, S, D)).astype(np.float32)
    idx = np.stack([rng.permutation(S)[:n] for _ in range(B)]).astype(np.int32)
    flags = np.zeros((B, n), dtype=np.uint8)
    for b in range(B):
        flags[b, rng.permutation(n)[:nG]] = 1
    qkv_d = dev(qkv, torch.bfloat16)
    cache_a, cache_b = dev(cache, torch.bfloat16), dev(cache, torch.bfloat16)
    o_a = torch.zeros(B * n, D, dtype=torch.float16, device="cuda")
    p_a = torch.full((B, H, S), -1.0, device="cuda")
    m.attention_two_segment(qkv_d, 3 * D, n, idx_dev(idx), cache_a, dev(flags), p_a, o_a)
    m.scatter_kv(qkv_d[:, D:], qkv_d[:, 2 * D:], 3 * D, idx_dev(idx), n, cache_b)
    torch.cuda.synchronize()
    assert m.device_status() == 0
    assert torch.equal(cache_a, cache_b)                               # write-back: byte-identical
    qq, cc = quant(qkv, "bf16"), host(cache_b)
    want_o, want_p = np.zeros((B * n, D)), np.zeros((B, H, S))
    for b in range(B):
        for h in range(H):
            c = slice(h * dh, (h + 1) * dh)
            z, p = orc.softmax_attention(qq[b * n:(b + 1) * n, c], cc[0, b][:, c], cc[1, b][:, c])
            want_o[b * n:(b + 1) * n, c] = z
            want_p[b, h] = p[flags[b].astype(bool)].sum(axis=0)
    assert rel_l2(host(o_a), want_o) <= 8e-3 and max_abs(host(o_a), want_o) <= 3e-2
    assert max_abs(host(p_a), want_p) <= 2e-2 * max(1, nG) / 8 + 1e-6
    assert np.allclose(host(p_a).sum(-1), nG, rtol=5e-3, atol=1e-6)


@pytest.mark.parametrize("dtype", ["f32", "bf16", "bf16b"])
def test_attention_uniform_and_peaked(dtype):
    S, B, H, dh, n = 68, 2, 4, 64, 5
    D = H * dh
    cfg, blocks, m = model_for(dtype, D, H, 128, S, B)
    rng = np.random.default_rng(1)
    cache = rng.standard_normal((2, B, S, D)).astype(np.float32)
    flags = np.ones((B, n), dtype=np.uint8)
    # q = 0 -> uniform weights: o = mean of V, partial = n / S
    o = torch.zeros(B * n, D, dtype=adt(dtype), device="cuda")
    partial = torch.zeros(B, H, S, device="cuda")
    m.attention(torch.zeros(B * n, D, dtype=tdt(dtype), device="cuda"), D, n, dev(cache, tdt(dtype)), dev(flags),
                partial, o)
    vm = quant(cache, dtype)[1].mean(axis=1)
    assert max_abs(host(o).reshape(B, n, D), np.repeat(vm[:, None], n, 1)) <= (4e-3 if dtype in LOW else 1e-5)
    assert np.allclose(host(partial), n / S, rtol=1e-3 if dtype in LOW else 1e-5)
    # q = 64 * k_t -> one-hot on key t: o = V[t]; no inf/nan
    tsel = rng.integers(0, S, size=(B, n))
    kq = quant(cache, dtype)
    q = np.stack([kq[0, b, tsel[b]] for b in range(B)]).reshape(B * n, D) * 64.0
    m.attention(dev(q.astype(np.float32), tdt(dtype)), D, n, dev(cache, tdt(dtype)), dev(flags), partial, o)
    got = host(o).reshape(B, n, D)
    assert np.isfinite(got).all()
    for b in range(B):
        assert max_abs(got[b], kq[1, b, tsel[b]]) <= (2e-2 if dtype in LOW else 1e-4)
    assert np.allclose(host(partial).sum(-1), n, rtol=1e-3)


# ------------------------------------------------------------------ K4 top-k (bit-exact)
@pytest.mark.parametrize("S,k", [(5, 2), (68, 7), (320, 32), (320, 0), (320, 311), (1088, 109), (1088, 1), (2048, 205),
                                 (2048, 2043), (33, 28)])
def test_select_refresh_bit_exact(S, k):
    B = 4
    cfg, blocks, m = model_for("f32", 128, 2, 128, S, B)
    rng = np.random.default_rng(S * 3 + k)
    n_new, n_excl = (2, 3) if S > 5 else (1, 1)
    kinds = [rng.random((B, S)), np.ones((B, S)), rng.integers(0, 3, (B, S)).astype(float),
             rng.random((B, S)) * 1e-42, np.exp(rng.uniform(-80, 10, (B, S))), np.zeros((B, S))]
    kinds[5][:, ::2] = -0.0
    mask = torch.empty(B * S, dtype=torch.uint8, device="cuda")
    for sc in kinds:
        sc = sc.astype(np.float32)
        perm = np.stack([rng.permutation(S) for _ in range(B)]).astype(np.int32)
        for new, excl in ((perm[:, :n_new], perm[:, n_new:n_new + n_excl]), (perm[:, :n_new], None),
                          (np.tile(np.arange(n_new, dtype=np.int32), (B, 1)), np.tile(np.arange(S - n_excl, S, dtype=np.int32), (B, 1)))):
            kk = min(k, S - n_new - (0 if excl is None else n_excl))
            out = torch.full((B, max(kk, 1)), -1, dtype=torch.int32, device="cuda")
            m.select_refresh(dev(sc), idx_dev(new), None if excl is None else idx_dev(excl), kk, out, mask)
            want = orc.select_refresh(sc, new, excl, kk)
            if kk:
                assert np.array_equal(out.cpu().numpy(), want)
            else:
                assert (out.cpu().numpy() == -1).all()


@pytest.mark.parametrize("policy,name", [(0, "high"), (1, "low"), (2, "random")])
def test_select_refresh_policies_bit_exact(policy, name):
    B, S, k = 5, 320, 32
    cfg, blocks, m = model_for("f32", 128, 2, 128, S, B)
    rng = np.random.default_rng(policy)
    mask = torch.empty(B * S, dtype=torch.uint8, device="cuda")
    for sc in (rng.random((B, S)), rng.integers(0, 4, (B, S)).astype(float), np.zeros((B, S))):
        sc = sc.astype(np.float32)
        perm = np.stack([rng.permutation(S) for _ in range(B)]).astype(np.int32)
        new, excl = perm[:, :4], perm[:, 4:9]
        out = torch.full((B, k), -1, dtype=torch.int32, device="cuda")
        m.select_refresh_policy(dev(sc), idx_dev(new), idx_dev(excl), k, policy, 1234, out, mask)
        assert np.array_equal(out.cpu().numpy(), orc.select_refresh(sc, new, excl, k, policy=name, seed=1234))


def test_validate_indices():
    from paper_2506_12035_b200.binding import MarcheError
    S, B = 68, 2
    cfg, blocks, m = model_for("f32", 128, 2, 128, S, B)
    act = np.array([[1, 2, 3, 4], [5, 6, 7, 8]], np.int32)
    new = act[:, :2]
    excl = np.array([[9], [10]], np.int32)
    m.validate_indices(idx_dev(act), idx_dev(new), idx_dev(excl))
    for bad_act, bad_new, bad_excl in [
        (np.array([[1, 2, 3, 3], [5, 6, 7, 8]], np.int32), new, excl),            # duplicate
        (np.array([[1, 2, 3, 68], [5, 6, 7, 8]], np.int32), new, excl),           # out of range
        (act, np.array([[1, 9], [5, 6]], np.int32), None),                         # new not in active
        (act, new, np.array([[2], [10]], np.int32)),                               # exclude overlaps new
    ]:
        with pytest.raises(MarcheError) as e:
            m.validate_indices(idx_dev(bad_act), idx_dev(bad_new), None if bad_excl is None else idx_dev(bad_excl))
        assert e.value.code == -5


@pytest.mark.parametrize("M,N,K", [(4800, 1024, 256), (9000, 768, 128), (5248, 3072, 192), (19100, 256, 128)])
def test_linear_many_tiles_all_epilogues(M, N, K):
    """Shapes with more output tiles than CTA pairs and a partial last round, where the pair GEMM
    cuts the left-over tiles into column slices (and, for the residual epilogue with long K, uses
    stream-K): every element against the oracle's product."""
    dtype = "bf16"
    cfg, blocks, m = model_for(dtype, 256, 4, 1024, 68, 2)
    rng = np.random.default_rng(M + N + K)
    a = rng.standard_normal((M, K)).astype(np.float32)
    w = (rng.standard_normal((N, K)) * 0.05).astype(np.float32)
    bias = rng.standard_normal(N).astype(np.float32)
    aq, wq = quant_a(a, dtype), quant_a(w, dtype)
    acc = orc.linear(aq, wq, bias.astype(np.float64))
    a_d, w_d, b_d = dev(a, adt(dtype)), dev(w, adt(dtype)), dev(bias)
    out = torch.zeros(M + 3, N, dtype=tdt(dtype), device="cuda")
    m.linear(a_d, w_d, b_d, 0, out, M=M)
    assert max_abs(host(out[:M]), acc) <= 3e-2 and rel_l2(host(out[:M]), acc) <= 4e-3
    assert (host(out[M:]) == 0).all()                                    # rows beyond M untouched
    res = rng.standard_normal((M, N)).astype(np.float32)
    out = dev(res)
    m.linear(a_d, w_d, b_d, 1, out)
    assert max_abs(host(out), acc + res) <= 1e-4 * max(1.0, math.sqrt(K / 256))
    out = torch.zeros(M, N, dtype=adt(dtype), device="cuda")
    m.linear(a_d, w_d, b_d, 2, out)
    want = orc.gelu(acc)
    assert max_abs(host(out), want) <= 3e-2 and rel_l2(host(out), want) <= 4e-3
    assert m.device_status() == 0


@pytest.mark.parametrize("D,F", [(768, 3072), (1024, 4096), (1280, 5120)])
@pytest.mark.parametrize("M", [256, 4352, 5760, 10176])
def test_projection_shapes_of_the_configs(D, F, M):
    """The four projections of a block at the row counts of the benchmark configurations (K = 1280 and
    5120 loop counts included); 384 sampled rows of each output against the oracle's product."""
    dtype = "bf16"
    cfg, blocks, m = model_for(dtype, 256, 4, 1024, 68, 2)
    rng = np.random.default_rng(D + M)
    rows = np.unique(np.concatenate([[0, M - 1], rng.integers(0, M, 382)]))
    for (N, K, epi) in ((3 * D, D, 0), (D, D, 1), (F, D, 2), (D, F, 1)):
        a = rng.standard_normal((M, K)).astype(np.float32)
        w = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
        bias = (rng.standard_normal(N) * 0.02).astype(np.float32)
        acc = orc.linear(quant_a(a[rows], dtype), quant_a(w, dtype), bias.astype(np.float64))
        a_d, w_d, b_d = dev(a, adt(dtype)), dev(w, adt(dtype)), dev(bias)
        if epi == 0:
            out = torch.zeros(M, N, dtype=tdt(dtype), device="cuda")
            want = acc
        elif epi == 1:
            res = rng.standard_normal((M, N)).astype(np.float32)
            out = dev(res)
            want = acc + res[rows]
        else:
            out = torch.zeros(M, N, dtype=adt(dtype), device="cuda")
            want = orc.gelu(acc)
        m.linear(a_d, w_d, b_d, epi, out)
        got = host(out)[rows]
        lim = 1e-4 * max(1.0, math.sqrt(K / 256)) if epi == 1 else 3e-2
        assert max_abs(got, want) <= lim, (N, K, epi, max_abs(got, want))
        if epi != 1:
            assert rel_l2(got, want) <= 4e-3
    assert m.device_status() == 0


@pytest.mark.parametrize("S", [320, 1088])
@pytest.mark.parametrize("dh,H", [(64, 4), (80, 8)])
@pytest.mark.parametrize("n,nG", [(159, 25), (320, 320), (97, 1)])
def test_attention_many_rows(S, dh, H, n, nG):
    """Active sets beyond one query tile (both tensor-core kernels are reached: tcgen05 for head_dim 64,
    mma.sync with seven consumer warps for head_dim 80), every query scoring in one case."""
    dtype = "bf16"
    B, D = 2, dh * H
    cfg, blocks, m = model_for(dtype, D, H, 128, S, B)
    rng = np.random.default_rng(S + n + dh)
    q = (rng.standard_normal((B * n, 3 * D)) * 3.0).astype(np.float32)
    cache = rng.standard_normal((2, B, S, D)).astype(np.float32)
    flags = np.zeros((B, n), dtype=np.uint8)
    for b in range(B):
        flags[b, rng.permutation(n)[:nG]] = 1
    o = torch.zeros(B * n, D, dtype=adt(dtype), device="cuda")
    partial = torch.full((B, H, S), -1.0, device="cuda")
    m.attention(dev(q, tdt(dtype)), 3 * D, n, dev(cache, tdt(dtype)), dev(flags), partial, o)
    qq, cc = quant(q, dtype), quant(cache, dtype)
    want_o = np.zeros((B * n, D))
    want_p = np.zeros((B, H, S))
    for b in range(B):
        for h in range(H):
            c = slice(h * dh, (h + 1) * dh)
            z, p = orc.softmax_attention(qq[b * n:(b + 1) * n, c], cc[0, b][:, c], cc[1, b][:, c])
            want_o[b * n:(b + 1) * n, c] = z
            want_p[b, h] = p[flags[b].astype(bool)].sum(axis=0)
    got_o, got_p = host(o), host(partial)
    assert rel_l2(got_o, want_o) <= 8e-3 and max_abs(got_o, want_o) <= 3e-2
    assert max_abs(got_p, want_p) <= 2e-2 * max(1, nG) / 8 + 1e-6
    assert np.allclose(got_p.sum(-1), nG, rtol=5e-3, atol=1e-6)
    o2 = torch.zeros_like(o)
    m.attention(dev(q, tdt(dtype)), 3 * D, n, dev(cache, tdt(dtype)), None, None, o2)       # plain flavour
    assert rel_l2(host(o2), want_o) <= 8e-3 and max_abs(host(o2), want_o) <= 3e-2
    assert m.device_status() == 0


@pytest.mark.parametrize("operand", ["bf16", "bf16b"])
@pytest.mark.parametrize("dh", [64, 80])
@pytest.mark.parametrize("B,H,S,n", [(2, 4, 68, 1), (3, 4, 257, 7), (2, 8, 320, 16), (2, 8, 320, 17), (5, 4, 64, 32),
                                     (80, 16, 200, 5), (140, 8, 130, 20)])
def test_attention_small_sets_persistent(operand, dh, B, H, S, n):
    """Plain attention at up to 32 query rows takes the persistent mma.sync launch: one and two consumer warps,
    both head sizes, ragged key tiles, fewer items than resident CTAs and several items per CTA (1280 and 1120
    items), where a CTA's loads run ahead into its next item."""
    if dh == 80:
        H = (H + 7) // 8 * 8                                # the model width must be a multiple of 128
    D = H * dh
    if operand == "bf16b" and B > 5:
        pytest.skip("one operand type is enough for the large shapes")
    cfg, blocks, m = model_for(operand, D, H, 128, S, B)
    rng = np.random.default_rng(7 * B + H + S + n + dh)
    cache = rng.standard_normal((2, B, S, D)).astype(np.float32)
    q = (rng.standard_normal((B * n, D)) * 2.0).astype(np.float32)
    o = torch.zeros(B * n, D, dtype=adt(operand), device="cuda")
    m.attention(dev(q, torch.bfloat16), D, n, dev(cache, torch.bfloat16), None, None, o)
    torch.cuda.synchronize()
    assert m.device_status() == 0
    got = host(o).reshape(B, n, D)
    assert np.isfinite(got).all()
    qq, cc = quant(q, "bf16").reshape(B, n, D), quant(cache, "bf16")
    for b in sorted(set([0, 1, B // 2, B - 2, B - 1])):
        want = np.zeros((n, D))
        for h in range(H):
            c = slice(h * dh, (h + 1) * dh)
            want[:, c], _ = orc.softmax_attention(qq[b][:, c], cc[0, b][:, c], cc[1, b][:, c])
        assert rel_l2(got[b], want) <= 8e-3 and max_abs(got[b], want) <= 3e-2, \
            "b=%d: max-abs %.3g rel-L2 %.3g" % (b, max_abs(got[b], want), rel_l2(got[b], want))


@pytest.mark.parametrize("operand", ["bf16", "bf16b"])
@pytest.mark.parametrize("B,H,S,n", [(2, 4, 68, 5), (2, 4, 128, 128), (3, 4, 320, 41), (40, 4, 320, 41), (2, 4, 320, 129),
                                     (2, 4, 320, 320), (100, 4, 320, 77), (2, 16, 1088, 122), (2, 16, 1088, 159),
                                     (1, 4, 1088, 1088), (2, 4, 2048, 300), (37, 8, 300, 257)])
def test_attention_single_pass_tcgen05(operand, B, H, S, n):
    """The single-pass tcgen05 kernel (weights kept in tensor memory, persistent over (sample, head) items) on
    its own: one, two and more query tiles, one key tile up to sixteen with ragged tails, more items than SMs,
    and logits whose row maximum keeps growing from tile to tile (the lazy rescaling of the accumulator)."""
    from paper_2506_12035_b200 import binding
    dh = 64
    D = H * dh
    if operand == "bf16b" and B * H * n * S > 3e6:
        pytest.skip("one operand type is enough for the large shapes")
    cfg, blocks, m = model_for(operand, D, H, 128, S, B)
    m.set_tuning(attention_kernel=binding.ATTENTION_TCGEN05)
    rng = np.random.default_rng(B + H + S + n)
    cache = rng.standard_normal((2, B, S, D)).astype(np.float32)
    # (i) ordinary logits; (ii) logits that grow with the key index: every tile raises the row maximum by
    # far more than 2^8, so each tile rescales the accumulator; (iii) one-hot rows on a late key
    q_rand = (rng.standard_normal((B * n, D)) * 3.0).astype(np.float32)
    ramp = np.linspace(0.0, 40.0, S, dtype=np.float32)
    cache_ramp = cache.copy()
    cache_ramp[0, :, :, 0::dh] = ramp[None, :, None]                   # first channel of every head's keys
    q_ramp = q_rand.copy()
    q_ramp[:, 0::dh] = 16.0                                            # logit contribution 16 * ramp / 8 = 0 .. 80
    kq = quant(cache, "bf16")
    tsel = rng.integers(max(0, S - 40), S, size=(B, n))
    q_hot = np.stack([kq[0, b, tsel[b]] for b in range(B)]).reshape(B * n, D).astype(np.float32) * 64.0
    sample_b = sorted(set([0, B // 2, B - 1]))
    for name, q, cch in (("random", q_rand, cache), ("ramp", q_ramp, cache_ramp), ("one-hot", q_hot, cache)):
        o = torch.zeros(B * n, D, dtype=adt(operand), device="cuda")
        m.attention(dev(q, torch.bfloat16), D, n, dev(cch, torch.bfloat16), None, None, o)
        torch.cuda.synchronize()
        assert m.device_status() == 0
        got = host(o).reshape(B, n, D)
        assert np.isfinite(got).all(), name
        qq, cc = quant(q, "bf16").reshape(B, n, D), quant(cch, "bf16")
        for b in sample_b:
            want = np.zeros((n, D))
            for h in range(H):
                c = slice(h * dh, (h + 1) * dh)
                want[:, c], _ = orc.softmax_attention(qq[b][:, c], cc[0, b][:, c], cc[1, b][:, c])
            assert rel_l2(got[b], want) <= 8e-3 and max_abs(got[b], want) <= 3e-2, \
                "%s b=%d: max-abs %.3g rel-L2 %.3g" % (name, b, max_abs(got[b], want), rel_l2(got[b], want))
