"""marche_select_refresh_static: the refresh selection for callers that may not allocate.

Some users of the library run where asking the device allocator for a scratch buffer is off
limits (memory planned up front, a serving loop that must not touch the allocator, a plug-in
that only receives its tensors).  For them the candidate mask sits in a fixed array inside the
library.  This file checks, through the C ABI, that the variant returns exactly what the
ordinary entry point returns (index work: bit-exact) on two calls in a row that use different
token sets, so that bytes left in the shared array by the first call would show up in the
second if they mattered; and that shapes beyond the built-in array are refused.

Collected last on purpose: a failure here cannot hide the result of any other test.
"""
import numpy as np
import pytest
import torch

import synth
from oracle import marche_oracle as orc
from paper_2506_12035_b200.binding import Marche, MarcheError, upload_weights

pytestmark = pytest.mark.gpu


def _model(B, S):
    cfg = synth.CONFIGS["tiny"].replace(L=1, E=0, D=128, H=2, F=128, S=S, B=B, n_buffer=0)
    return Marche.from_config(cfg, upload_weights(synth.make_weights(cfg), cfg.dtype))


def test_static_scratch_selection_matches_ordinary_entry_point():
    B, S = 8, 320
    m = _model(B, S)
    rng = np.random.default_rng(42)
    mask = torch.empty(B * S, dtype=torch.uint8, device="cuda")
    for call, (n_new, n_excl, k) in enumerate([(5, 7, 32), (2, 0, 40)]):        # two calls in a row
        scores = rng.integers(0, 6, (B, S)).astype(np.float32) / 4.0             # many ties
        perm = np.stack([rng.permutation(S) for _ in range(B)]).astype(np.int32)
        new = torch.as_tensor(perm[:, :n_new]).cuda().contiguous()
        excl = torch.as_tensor(perm[:, n_new:n_new + n_excl]).cuda().contiguous() if n_excl else None
        sc = torch.as_tensor(scores).cuda()
        want = torch.full((B, k), -1, dtype=torch.int32, device="cuda")
        got = torch.full((B, k), -2, dtype=torch.int32, device="cuda")
        m.select_refresh(sc, new, excl, k, want, mask)
        m.select_refresh_static(sc, new, excl, k, got)
        torch.cuda.synchronize()
        assert torch.equal(got, want), "call %d differs from marche_select_refresh" % call
        ref = orc.select_refresh(scores, perm[:, :n_new], perm[:, n_new:n_new + n_excl] if n_excl else None, k)
        assert np.array_equal(got.cpu().numpy(), ref)
    assert m.device_status() == 0


def test_static_scratch_rejects_shapes_beyond_its_size():
    B, S = 900, 320                                   # 288000 bytes of mask > 256 KiB
    m = _model(B, S)
    sc = torch.zeros(B, S, device="cuda")
    out = torch.full((B, 4), -7, dtype=torch.int32, device="cuda")
    with pytest.raises(MarcheError) as e:
        m.select_refresh_static(sc, None, None, 4, out)
    assert e.value.code == -3 and "288000" in str(e.value) and "262144" in str(e.value)
    torch.cuda.synchronize()
    assert (out == -7).all()                          # nothing was enqueued


def test_static_scratch_accepts_the_largest_shape_it_holds():
    B, S = 128, 2048                                  # exactly 262144 bytes of mask: the limit itself
    m = _model(B, S)
    rng = np.random.default_rng(7)
    scores = rng.integers(0, 50, (B, S)).astype(np.float32)
    perm = np.stack([rng.permutation(S)[:9] for _ in range(B)]).astype(np.int32)
    new, excl = torch.as_tensor(perm[:, :4]).cuda().contiguous(), torch.as_tensor(perm[:, 4:]).cuda().contiguous()
    sc = torch.as_tensor(scores).cuda()
    k = 205
    want = torch.full((B, k), -1, dtype=torch.int32, device="cuda")
    got = torch.full((B, k), -2, dtype=torch.int32, device="cuda")
    m.select_refresh(sc, new, excl, k, want, torch.empty(B * S, dtype=torch.uint8, device="cuda"))
    m.select_refresh_static(sc, new, excl, k, got)
    torch.cuda.synchronize()
    assert torch.equal(got, want)
    assert np.array_equal(got.cpu().numpy(), orc.select_refresh(scores, perm[:, :4], perm[:, 4:], k))
