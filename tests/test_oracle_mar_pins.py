"""Pins of the oracle's two-stage (encoder over known tokens, decoder over all tokens) step.

CPU only.  The orchestration is pinned to the already pinned uniform-stack functions on inputs
where both must agree, to closed forms of the decoder input, and to invariants of Eq. 1 / Eq. 2.
"""
import numpy as np
import pytest

import synth
from oracle import marche_oracle as orc


def cfg6(**kw):
    base = synth.CONFIGS["tiny"].replace(L=6, E=2, D=64, H=4, F=128, S=20, n_buffer=4, B=2, T=4)
    return base.replace(**kw)


def setup(cfg, seed=0):
    blocks = synth.make_weights(cfg, seed=1234 + seed)
    mar = synth.make_mar_weights(cfg, seed=4321 + seed)
    tokens = synth.make_hidden(cfg, seed=2025 + seed)
    return blocks, mar, tokens


def sets(cfg):
    new_sets = synth.new_token_sets(cfg, synth.generation_orders(cfg))
    return new_sets, synth.known_token_sets(cfg, new_sets)


def kw(cfg, **extra):
    d = dict(n_heads=cfg.H, n_enc=cfg.E, score_layer=cfg.score_layer, ln_eps=cfg.ln_eps)
    d.update(extra)
    return d


def test_known_sets_partition_the_sequence():
    cfg = cfg6()
    new_sets, known = sets(cfg)
    for t, (G, K) in enumerate(zip(new_sets, known)):
        assert K.shape[1] == cfg.n_buffer + sum(g.shape[1] for g in new_sets[:t])
        for b in range(cfg.B):
            assert np.all(np.diff(K[b]) > 0)
            assert not set(K[b].tolist()) & set(G[b].tolist())          # generating tokens are still masked
            assert set(range(cfg.n_buffer)) <= set(K[b].tolist())


def test_encoder_equals_uniform_stack_on_the_compacted_sequence():
    """Eq. 1: the encoder over the known tokens is an ordinary full pass over a shorter sequence."""
    cfg = cfg6()
    blocks, mar, tokens = setup(cfg)
    known = np.array([0, 1, 2, 3, 7, 9, 15], dtype=np.int64)
    got = orc.mar_encoder([{k: v.astype(np.float64) for k, v in b.items()} for b in blocks[:cfg.E]],
                          tokens[0].astype(np.float64), known, n_heads=cfg.H, ln_eps=cfg.ln_eps)
    short = tokens[:1, known]
    cache = orc.KVCache(cfg.E, 1, len(known), cfg.D)
    out = np.zeros_like(short, dtype=np.float64)
    orc.full_step(blocks[:cfg.E], short, cache, np.zeros((1, 0), np.int32), None, 0.0, out,
                  n_heads=cfg.H, score_layer=0, ln_eps=cfg.ln_eps)
    assert np.allclose(got, out[0], atol=1e-12)


def test_encoder_ignores_masked_rows():
    cfg = cfg6()
    blocks, mar, tokens = setup(cfg)
    new_sets, known = sets(cfg)
    z1 = np.zeros(tokens.shape)
    z2 = np.zeros(tokens.shape)
    c1 = orc.KVCache(cfg.L, cfg.B, cfg.S, cfg.D)
    c2 = orc.KVCache(cfg.L, cfg.B, cfg.S, cfg.D)
    poisoned = tokens.copy()
    for b in range(cfg.B):
        masked = np.setdiff1d(np.arange(cfg.S), known[1][b])
        poisoned[b, masked] = np.nan
    a = orc.mar_step(blocks, mar, tokens, known[1], c1, new_sets[1], new_sets[0], 0, z1, full_decoder=True, **kw(cfg))
    b_ = orc.mar_step(blocks, mar, poisoned, known[1], c2, new_sets[1], new_sets[0], 0, z2, full_decoder=True, **kw(cfg))
    assert np.isfinite(z2).all() and np.array_equal(z1, z2) and np.array_equal(a[0], b_[0])
    # the encoder blocks keep nothing in the cache
    assert not c1.K[:cfg.E].any() and not c1.V[:cfg.E].any() and c1.K[cfg.E:].any()


def test_decoder_input_closed_form():
    """Masked rows: mask embedding + position.  Known rows with an identity map and unit norm:
    the standardised encoder row + position; a +-1 row is already standardised."""
    cfg = cfg6()
    _, mar, _ = setup(cfg)
    D, S = cfg.D, cfg.S
    mar = {k: v.astype(np.float64) for k, v in mar.items()}
    mar.update(enc_norm_g=np.ones(D), enc_norm_b=np.zeros(D), w_dec_embed=np.eye(D), b_dec_embed=np.zeros(D))
    known = np.array([1, 4, 5], dtype=np.int64)
    h = np.tile(np.where(np.arange(D) % 2 == 0, 1.0, -1.0), (3, 1)) * np.array([[1.0], [3.0], [-2.0]])
    x = orc.mar_decoder_input(h, known, S, mar, 0.0)
    unit = np.where(np.arange(D) % 2 == 0, 1.0, -1.0)
    for j, t in enumerate(known):
        assert np.allclose(x[t], np.sign([1.0, 3.0, -2.0][j]) * unit + mar["dec_pos"][t], atol=1e-12)
    for t in np.setdiff1d(np.arange(S), known):
        assert np.array_equal(x[t], mar["mask_token"] + mar["dec_pos"][t])
    # a non-trivial map: transposed-operand check, y = W h + b with W [out][in]
    W = np.zeros((D, D)); W[3, 5] = 2.0
    mar.update(w_dec_embed=W, b_dec_embed=np.full(D, 0.25))
    x = orc.mar_decoder_input(h, known, S, mar, 0.0)
    want = np.full(D, 0.25); want[3] += 2.0 * unit[5]
    assert np.allclose(x[1], want + mar["dec_pos"][1], atol=1e-12)


def decoder_input_all(cfg, blocks, mar, tokens, known):
    b64 = [{k: v.astype(np.float64) for k, v in b.items()} for b in blocks]
    m64 = {k: v.astype(np.float64) for k, v in mar.items()}
    rows = []
    for b in range(cfg.B):
        kn = known[b].astype(np.int64)
        h = orc.mar_encoder(b64[:cfg.E], tokens[b].astype(np.float64), kn, n_heads=cfg.H, ln_eps=cfg.ln_eps)
        rows.append(orc.mar_decoder_input(h, kn, cfg.S, m64, cfg.ln_eps))
    return np.stack(rows)


def test_decoder_matches_uniform_stack_functions():
    """Given the decoder input, the decoder of mar_step is the pinned full step / in-step-selection
    step over blocks[E:], followed by the final norm on the rows that were computed."""
    cfg = cfg6()
    blocks, mar, tokens = setup(cfg)
    new_sets, known = sets(cfg)
    dec = blocks[cfg.E:]
    sl = cfg.score_layer - cfg.E
    # step 0: full decoder
    cache = orc.KVCache(cfg.L, cfg.B, cfg.S, cfg.D)
    z = np.zeros(tokens.shape)
    s0, _, _ = orc.mar_step(blocks, mar, tokens, known[0], cache, new_sets[0], None, 0, z, full_decoder=True, **kw(cfg))
    x0 = decoder_input_all(cfg, blocks, mar, tokens, known[0])
    ref_cache = orc.KVCache(len(dec), cfg.B, cfg.S, cfg.D)
    out = np.zeros(tokens.shape)
    r0, _ = orc.full_step(dec, x0, ref_cache, new_sets[0], None, 0.0, out, n_heads=cfg.H, score_layer=sl, ln_eps=cfg.ln_eps)
    want = orc.layer_norm(out, mar["dec_norm_g"].astype(np.float64), mar["dec_norm_b"].astype(np.float64), cfg.ln_eps)
    assert np.allclose(z, want, atol=1e-11) and np.array_equal(s0, r0)
    assert np.allclose(cache.K[cfg.E:], ref_cache.K, atol=1e-12)
    # step 1: in-step selection
    tokens1 = tokens.copy()
    for b in range(cfg.B):
        tokens1[b, new_sets[0][b]] = synth.replacement_rows(cfg, 0, new_sets[0].shape[1])[b]
    z1 = z.copy()
    s1, R1, A1 = orc.mar_step(blocks, mar, tokens1, known[1], cache, new_sets[1], new_sets[0], 3, z1,
                              full_decoder=False, **kw(cfg))
    x1 = decoder_input_all(cfg, blocks, mar, tokens1, known[1])
    out1 = np.zeros(tokens.shape)
    r1, Rr, Ar = orc.in_step_selection_step(dec, x1, ref_cache, new_sets[1], new_sets[0], 3, out1, n_heads=cfg.H,
                                            score_layer=sl, ln_eps=cfg.ln_eps)
    assert np.array_equal(R1, Rr) and np.array_equal(A1, Ar) and np.array_equal(s1, r1)
    for b in range(cfg.B):
        rows = A1[b]
        want = orc.layer_norm(out1[b, rows], mar["dec_norm_g"].astype(np.float64), mar["dec_norm_b"].astype(np.float64), cfg.ln_eps)
        assert np.allclose(z1[b, rows], want, atol=1e-11)
        rest = np.setdiff1d(np.arange(cfg.S), rows)
        assert np.array_equal(z1[b, rest], z[b, rest])                 # rows outside A keep their bytes


def test_refreshing_everything_equals_the_full_decoder():
    """Appendix A: with every candidate refreshed, the cache-aware decoder is exact."""
    cfg = cfg6()
    blocks, mar, tokens = setup(cfg, seed=1)
    new_sets, known = sets(cfg)
    ca, cb = (orc.KVCache(cfg.L, cfg.B, cfg.S, cfg.D) for _ in range(2))
    za, zb = np.zeros(tokens.shape), np.zeros(tokens.shape)
    for c, z in ((ca, za), (cb, zb)):
        orc.mar_step(blocks, mar, tokens, known[0], c, new_sets[0], None, 0, z, full_decoder=True, **kw(cfg))
    tokens1 = tokens.copy()
    for b in range(cfg.B):
        tokens1[b, new_sets[0][b]] = synth.replacement_rows(cfg, 0, new_sets[0].shape[1])[b]
    k_all = cfg.S - new_sets[1].shape[1] - new_sets[0].shape[1]
    orc.mar_step(blocks, mar, tokens1, known[1], ca, new_sets[1], new_sets[0], k_all, za, full_decoder=False, **kw(cfg))
    orc.mar_step(blocks, mar, tokens1, known[1], cb, new_sets[1], new_sets[0], 0, zb, full_decoder=True, **kw(cfg))
    assert np.allclose(za, zb, atol=1e-10)
    assert np.allclose(ca.K, cb.K, atol=1e-10) and np.allclose(ca.V, cb.V, atol=1e-10)


def test_generation_schedule_and_budget():
    cfg = cfg6()
    blocks, mar, tokens = setup(cfg)
    new_sets, known = sets(cfg)
    log, _ = orc.generate_mar(blocks, mar, tokens, new_sets, known, lambda t, n: synth.replacement_rows(cfg, t, n),
                              budget=10, period=3, **kw(cfg))
    assert [d["kind"] for d in log] == ["full", "in_step", "in_step", "full"]
    for t, d in enumerate(log):
        if d["kind"] == "in_step":
            nG, nN = new_sets[t].shape[1], new_sets[t - 1].shape[1]
            assert d["active"].shape[1] == max(10, nG + nN) or d["active"].shape[1] == nG + nN + d["refresh"].shape[1]
            assert d["refresh"].shape[1] == max(0, min(10 - nG - nN, cfg.S - nG - nN))
        assert np.isfinite(d["z"]).all()


def test_argument_checks():
    cfg = cfg6()
    blocks, mar, tokens = setup(cfg)
    new_sets, known = sets(cfg)
    cache = orc.KVCache(cfg.L, cfg.B, cfg.S, cfg.D)
    z = np.zeros(tokens.shape)
    with pytest.raises(RuntimeError):                                   # cache-aware decoder on an empty cache
        orc.mar_step(blocks, mar, tokens, known[1], cache, new_sets[1], new_sets[0], 2, z, full_decoder=False, **kw(cfg))
    with pytest.raises(ValueError):                                     # scoring block inside the encoder
        orc.mar_step(blocks, mar, tokens, known[0], cache, new_sets[0], None, 0, z, full_decoder=True,
                     **kw(cfg, score_layer=cfg.E - 1))
