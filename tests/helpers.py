"""Shared helpers of the GPU parity tests (marshalling between NumPy and the binding)."""
import numpy as np
import torch

import synth
from paper_2506_12035_b200.binding import Marche, upload_weights

# Acceptance bounds (max-abs, relative L2) against the fp64 oracle.
# "bf16" is the 16-bit context with fp16 projection operands (MARCHE_BF16_F16OP), "bf16b" the one with
# bf16 operands throughout (MARCHE_BF16); both face the same bound.
TOL = {"bf16": (3e-2, 1e-2), "bf16b": (3e-2, 1e-2), "f32": (1e-4, 1e-5)}


def make_model(cfg, blocks, operand="f16"):
    return Marche.from_config(cfg, upload_weights(blocks, cfg.dtype, operand=operand))


def dev(a, dtype=None):
    t = torch.as_tensor(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda().contiguous()


def idx_dev(a):
    return dev(np.asarray(a, dtype=np.int32))


def host(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def max_abs(a, b):
    return float(np.abs(np.asarray(a, dtype=np.float64) - np.asarray(b, dtype=np.float64)).max()) if np.size(a) else 0.0


def rel_l2(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    den = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / den) if den > 0 else float(np.linalg.norm(a - b))


def assert_close(got, want, dtype, what="", scale=1.0):
    ma, rl = TOL[dtype]
    m, r = max_abs(got, want), rel_l2(got, want)
    assert m <= ma * scale and r <= rl, "%s: max-abs %.3g (limit %.3g), rel-L2 %.3g (limit %.3g)" % (what, m, ma * scale, r, rl)


def cache_to_oracle_layout(cache_t):
    """device cache [L][2][B][S][D] -> (K, V) float64 [L][B][S][D]"""
    c = host(cache_t)
    return c[:, 0], c[:, 1]


def small_cfg(dtype, **kw):
    base = synth.CONFIGS["tiny"].replace(dtype=dtype)
    return base.replace(**kw) if kw else base
