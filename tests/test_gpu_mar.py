"""Parity of marche_mar_step (encoder over the known tokens, Eq. 1; decoder input with mask
embeddings, Eq. 2; cache-aware decoder under the schedule of Section 4.2 / 4.3) with the CPU
oracle, teacher-forced with the oracle's refresh sets, plus invariants and error behaviour."""
import numpy as np
import pytest
import torch

import synth
from oracle import marche_oracle as orc
from paper_2506_12035_b200.binding import MarcheError, upload_mar_weights
from paper_2506_12035_b200.generation import Generation
from helpers import assert_close, cache_to_oracle_layout, dev, idx_dev, make_model, max_abs

pytestmark = pytest.mark.gpu

CASES = {
    "tiny_f32": synth.CONFIGS["tiny"].replace(L=6, E=2),
    "tiny_bf16": synth.CONFIGS["tiny"].replace(L=6, E=2, dtype="bf16"),
    # MAR-B-shaped rows (D 768, 12 heads, S 320, 64 buffer tokens), cut down in depth, batch and steps
    "marb_slice": synth.CONFIGS["mar_b"].replace(L=5, E=2, B=4, T=6),
    # MAR-L-shaped rows at a batch that takes the CTA-pair GEMM and the tcgen05 attention
    "marl_slice": synth.CONFIGS["mar_l"].replace(L=5, E=2, B=8, T=5),
}


def build(cfg):
    blocks = synth.make_weights(cfg)
    mar = synth.make_mar_weights(cfg)
    tokens0 = synth.make_hidden(cfg)
    sets = synth.new_token_sets(cfg, synth.generation_orders(cfg))
    known = synth.known_token_sets(cfg, sets)
    m = make_model(cfg, blocks)
    m.set_mar_weights(upload_mar_weights(mar, cfg.dtype))
    rows = [dev(synth.replacement_rows(cfg, t, sets[t].shape[1])) for t in range(cfg.T)]
    return blocks, mar, tokens0, sets, known, m, Generation(m, sets, 0.0, rows)


@pytest.mark.parametrize("case", list(CASES))
def test_two_stage_generation_teacher_forced(case):
    cfg = CASES[case]
    budget = 24 if cfg.S < 100 else 64
    blocks, mar, tokens0, sets, known, m, gen = build(cfg)
    log, cache = orc.generate_mar(blocks, mar, tokens0, sets, known, lambda t, n: synth.replacement_rows(cfg, t, n),
                                  n_heads=cfg.H, n_enc=cfg.E, score_layer=cfg.score_layer, budget=budget, period=3,
                                  ln_eps=cfg.ln_eps)
    forced = [idx_dev(r["refresh"]) if r["kind"] == "in_step" and r["refresh"].shape[1] else None for r in log]
    glog = gen.run_mar(dev(tokens0), known, budget=budget, period=3, record=True, forced_refresh=forced)
    assert m.device_status() == 0
    mask = torch.empty(cfg.B * cfg.S, dtype=torch.uint8, device="cuda")
    for rec, g in zip(log, glog):
        A = rec["active"]
        assert g["n_active"] == A.shape[1]
        if rec["kind"] == "in_step":
            assert np.array_equal(g["active"], A)
        for b in range(cfg.B):
            # the decoder output is normalised (unit-size entries), so the absolute bound applies as is
            assert_close(g["z"][b, A[b]], rec["z"][b, A[b]], cfg.dtype, "%s step %d (%s)" % (case, rec["t"], rec["kind"]))
        unit = cfg.H * rec["new"].shape[1] / cfg.S
        assert max_abs(g["scores"], rec["scores"]) <= (5e-2 if cfg.dtype == "bf16" else 1e-4) * unit
        k = rec["refresh"].shape[1]
        if k:   # fed the oracle's scores, the device's selection is bit-exact
            out = torch.empty(cfg.B, k, dtype=torch.int32, device="cuda")
            m.select_refresh(dev(rec["scores"]), idx_dev(rec["new"]), idx_dev(rec["prev"]), k, out, mask)
            assert np.array_equal(out.cpu().numpy(), rec["refresh"])
    K, V = cache_to_oracle_layout(gen.cache)
    assert_close(K[cfg.E:], cache.K[cfg.E:], cfg.dtype, case + " decoder cache K")
    assert_close(V[cfg.E:], cache.V[cfg.E:], cfg.dtype, case + " decoder cache V")


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_invariants(dtype):
    """Masked rows of the input are never read; rows outside A keep their bytes; refreshing every
    candidate reproduces the full decoder; two runs give the same bits."""
    cfg = CASES["tiny_" + dtype]
    blocks, mar, tokens0, sets, known, m, gen = build(cfg)
    B, S = cfg.B, cfg.S
    tok = dev(tokens0)
    ws = gen.workspace
    z_full = torch.zeros(B, S, cfg.D, device="cuda")
    G0, G1 = gen.new_sets[0], gen.new_sets[1]
    kn0, kn1 = idx_dev(known[0]), idx_dev(known[1])

    m.init_cache(gen.cache)
    m.mar_step(True, tok, kn0, gen.cache, G0, None, 0, None, z_full, None, None, ws)
    poisoned = tok.clone()
    for b in range(B):
        masked = np.setdiff1d(np.arange(S), known[0][b])
        poisoned[b, torch.as_tensor(masked, device="cuda")] = float("nan")
    cache2 = m.alloc_cache()
    m.init_cache(cache2)
    z2 = torch.zeros_like(z_full)
    m.mar_step(True, poisoned, kn0, cache2, G0, None, 0, None, z2, None, None, ws)
    assert torch.isfinite(z2).all() and torch.equal(z2, z_full)                       # masked rows unread + same bits
    assert torch.equal(cache2[cfg.E:], gen.cache[cfg.E:])                             # decoder cache: same bits

    # step 1 two ways: cache-aware with every candidate refreshed == full decoder
    m.scatter_rows(gen.rows[0], G0, tok)
    n_gn = G1.shape[1] + G0.shape[1]
    k_all = S - n_gn
    refresh = torch.empty(B, k_all, dtype=torch.int32, device="cuda")
    active = torch.empty(B, S, dtype=torch.int32, device="cuda")
    z_a = z_full.clone()
    m.mar_step(False, tok, kn1, gen.cache, G1, G0, k_all, None, z_a, refresh, active, ws)
    z_b = torch.zeros_like(z_full)
    m.mar_step(True, tok, kn1, cache2, G1, G0, 0, None, z_b, None, None, ws)
    assert sorted(active[0].tolist()) == list(range(S))
    lim = 2e-2 if dtype == "bf16" else 1e-4
    assert max_abs(z_a.cpu().numpy(), z_b.cpu().numpy()) <= lim

    # a small active set leaves the other rows of z_out alone
    z_c = torch.full_like(z_full, 7.0)
    k = 5
    act = torch.empty(B, n_gn + k, dtype=torch.int32, device="cuda")
    m.mar_step(False, tok, kn1, gen.cache, G1, G0, k, None, z_c, refresh[:, :k].contiguous(), act, ws)
    zc = z_c.cpu().numpy()
    for b in range(B):
        rest = np.setdiff1d(np.arange(S), act[b].cpu().numpy())
        assert (zc[b, rest] == 7.0).all() and not (zc[b, act[b].cpu().numpy()] == 7.0).all()
    assert m.device_status() == 0


def test_argument_errors():
    cfg = CASES["tiny_f32"]
    blocks, mar, tokens0, sets, known, m, gen = build(cfg)
    tok, z = dev(tokens0), torch.zeros(cfg.B, cfg.S, cfg.D, device="cuda")
    kn = idx_dev(known[1])
    G0, G1 = gen.new_sets[0], gen.new_sets[1]
    m.init_cache(gen.cache)
    r = torch.empty(cfg.B, 4, dtype=torch.int32, device="cuda")
    a = torch.empty(cfg.B, cfg.S, dtype=torch.int32, device="cuda")
    with pytest.raises(MarcheError) as e:                      # cache-aware decoder before any full step
        m.mar_step(False, tok, kn, gen.cache, G1, G0, 4, None, z, r, a, gen.workspace)
    assert e.value.code == -4
    with pytest.raises(MarcheError) as e:                      # in place
        m.mar_step(True, tok, kn, gen.cache, G1, G0, 0, None, tok, None, None, gen.workspace)
    assert e.value.code == -1
    with pytest.raises(MarcheError) as e:                      # workspace too small
        m.mar_step(True, tok, kn, gen.cache, G1, G0, 0, None, z, None, None, gen.workspace[:1024])
    assert e.value.code == -3
    # a context without glue weights refuses the call
    m2 = make_model(cfg, blocks)
    with pytest.raises(MarcheError) as e:
        m2.mar_step(True, tok, kn, gen.cache, G1, G0, 0, None, z, None, None, gen.workspace)
    assert e.value.code == -1
    # scoring block inside the encoder
    m3 = make_model(cfg.replace(E=4), blocks)                  # default score layer E+1 = 5 = L-1: fine for full only
    m3.set_mar_weights(m.mar_weights)
    m3.mar_step(True, tok, kn, gen.cache, G1, G0, 0, None, z, None, None, gen.workspace)
    with pytest.raises(MarcheError) as e:                      # no cache-aware block left after the scoring block
        m3.mar_step(False, tok, kn, gen.cache, G1, G0, 4, None, z, r, a, gen.workspace)
    assert e.value.code == -1
    torch.cuda.synchronize()
    assert m.device_status() == 0
