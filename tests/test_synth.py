"""Checks of the seeded workload generators (inputs only, no method arithmetic)."""
import numpy as np
import torch

import synth


def test_cosine_schedule_counts():
    assert synth.mask_schedule(64, 8) == [2, 3, 6, 8, 10, 11, 12, 12]
    for n_img, T in ((256, 64), (1024, 64), (1024, 256)):
        c = synth.mask_schedule(n_img, T)
        assert len(c) == T and sum(c) == n_img and min(c) >= 1
    assert max(synth.mask_schedule(256, 64)) == 7 and max(synth.mask_schedule(1024, 64)) == 25


def test_orders_are_permutations_and_cfg_pairs_share():
    cfg = synth.CONFIGS["mar_b"].replace(B=8)
    o = synth.generation_orders(cfg)
    assert o.shape == (8, 256) and np.array_equal(o[:4], o[4:])
    for row in o:
        assert sorted(row.tolist()) == list(range(cfg.n_buffer, cfg.S))
    sets = synth.new_token_sets(cfg, o)
    assert np.array_equal(np.concatenate(sets, axis=1), o)


def test_bf16_rounding_matches_torch():
    rng = np.random.default_rng(0)
    a = (rng.standard_normal(100000) * np.exp(rng.uniform(-20, 20, 100000))).astype(np.float32)
    want = torch.from_numpy(a).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(synth.round_to_bf16(a), want)


def test_prefix_consistency_and_determinism():
    cfg = synth.CONFIGS["tiny"]
    assert np.array_equal(synth.make_hidden(cfg, batch=1)[0], synth.make_hidden(cfg)[0])
    w1, w2 = synth.make_weights(cfg, n_blocks=2), synth.make_weights(cfg)
    for k in synth.BLOCK_FIELDS:
        assert np.array_equal(w1[1][k], w2[1][k])
    r = synth.replacement_rows(cfg, 3, 5)
    assert np.array_equal(r[:1], synth.replacement_rows(cfg, 3, 5, batch=1))
    assert not np.array_equal(r, synth.replacement_rows(cfg, 4, 5))
    wb = synth.make_weights(synth.CONFIGS["mar_b"], n_blocks=1)[0]["w_qkv"]
    assert np.array_equal(wb, synth.round_to_bf16(wb)) and abs(wb.std() - 0.02) < 1e-3
