"""Synthetic MAR-shaped workload generator.

Everything here is input construction: model shapes, N(0, 0.02) weights,
N(0, 1) hidden rows, per-image random generation orders and the cosine mask
schedule that says how many tokens each decoding step generates.  The paper's
experiments run trained MAR-B/L/H on ImageNet 256x256 (Section 5.1); neither
exists here, so these seeded tensors of the same shapes stand in for them.

All random numbers come from NumPy's counter-based Philox generator so the
same (seed, shape) always yields the same bytes on every machine.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List

import numpy as np

# Seeds of the recipe (one stream per kind of tensor).
SEED_WEIGHTS = 1234
SEED_HIDDEN = 2025
SEED_ORDERS = 7
SEED_ROWS = 99

# Per-block parameter names, in the order the C-ABI struct lists them.
BLOCK_FIELDS = (
    "ln1_g", "ln1_b", "w_qkv", "b_qkv", "w_o", "b_o",
    "ln2_g", "ln2_b", "w_fc1", "b_fc1", "w_fc2", "b_fc2",
)
MATRIX_FIELDS = ("w_qkv", "w_o", "w_fc1", "w_fc2")


@dataclasses.dataclass(frozen=True)
class MarConfig:
    """Shape of one MAR-like stack and of its decoding run.

    L blocks (E of them "encoder"), width D = H * dh, MLP width F, S tokens per
    sample of which the first n_buffer are buffer tokens, B batch rows (already
    doubled for classifier-free guidance when cfg_pairs is True), T decoding
    steps, compute dtype "f32" or "bf16", refresh ratio r.
    """

    name: str
    L: int
    E: int
    D: int
    H: int
    F: int
    S: int
    n_buffer: int
    B: int
    T: int
    dtype: str
    ratio: float = 0.10
    cfg_pairs: bool = True
    ln_eps: float = 1e-6

    @property
    def dh(self) -> int:
        return self.D // self.H

    @property
    def n_img(self) -> int:
        return self.S - self.n_buffer

    @property
    def score_layer(self) -> int:
        """Default scoring block: the second decoder block (0-based E + 1)."""
        return min(self.E + 1, self.L - 1)

    @property
    def n_images(self) -> int:
        return self.B // 2 if self.cfg_pairs else self.B

    def replace(self, **kw) -> "MarConfig":
        return dataclasses.replace(self, **kw)


CONFIGS: Dict[str, MarConfig] = {
    # 4 blocks, width 256, 8x8 grid + 4 buffer tokens, batch 2, fp32, 8 steps
    "tiny": MarConfig("tiny", L=4, E=2, D=256, H=4, F=1024, S=68, n_buffer=4, B=2, T=8,
                      dtype="f32", cfg_pairs=False),
    "mar_b": MarConfig("mar_b", L=24, E=12, D=768, H=12, F=3072, S=320, n_buffer=64, B=128, T=64,
                       dtype="bf16"),
    "mar_l": MarConfig("mar_l", L=32, E=16, D=1024, H=16, F=4096, S=320, n_buffer=64, B=128, T=64,
                       dtype="bf16"),
    "mar_h": MarConfig("mar_h", L=40, E=20, D=1280, H=16, F=5120, S=320, n_buffer=64, B=128, T=64,
                       dtype="bf16"),
    "hires": MarConfig("hires", L=32, E=16, D=1024, H=16, F=4096, S=1088, n_buffer=64, B=64, T=64,
                       dtype="bf16"),
}


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16-representable value (ties to even),
    returned as fp32.  Finite inputs only."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    r = (u + bias) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def mask_schedule(n_img: int, T: int) -> List[int]:
    """Number of tokens generated at each of the T steps (cosine schedule).

    The masked count after step t is floor(n_img * cos(pi/2 * (t+1)/T)), forced
    to drop by at least one per step and to stay >= 1 until the last step, which
    generates whatever is left.
    """
    counts: List[int] = []
    masked = n_img
    for t in range(T):
        if t == T - 1:
            nxt = 0
        else:
            nxt = int(math.floor(n_img * math.cos(math.pi / 2.0 * (t + 1) / T)))
            nxt = max(1, min(nxt, masked - 1))
        counts.append(masked - nxt)
        masked = nxt
    assert sum(counts) == n_img and all(c >= 1 for c in counts)
    return counts


def generation_orders(cfg: MarConfig, seed: int = SEED_ORDERS) -> np.ndarray:
    """int32 [B][n_img]: per sample a uniformly random order of the image-token
    positions [n_buffer, S).  With CFG pairs, rows b and b + B/2 share an order."""
    rng = np.random.Generator(np.random.Philox(seed))
    n_real = cfg.n_images
    base = np.stack([rng.permutation(cfg.n_img) for _ in range(n_real)]).astype(np.int32)
    base += np.int32(cfg.n_buffer)
    if cfg.cfg_pairs:
        return np.concatenate([base, base], axis=0)
    return base


def new_token_sets(cfg: MarConfig, orders: np.ndarray) -> List[np.ndarray]:
    """List over steps t of int32 [B][#G(t)]: the positions generated at step t
    (consecutive chunks of each sample's order)."""
    counts = mask_schedule(cfg.n_img, cfg.T)
    out, pos = [], 0
    for c in counts:
        out.append(np.ascontiguousarray(orders[:, pos:pos + c]))
        pos += c
    return out


def make_weights(cfg: MarConfig, seed: int = SEED_WEIGHTS, n_blocks: int | None = None
                 ) -> List[Dict[str, np.ndarray]]:
    """Per block: fp32 arrays.  Linear weights ([out][in]) and all biases
    ~ N(0, 0.02^2); LayerNorm gain 1 + N(0, 0.02^2), shift N(0, 0.02^2).
    For bf16 configs the four matrices are rounded once to bf16-representable values (the recipe's
    "weights rounded to bf16 on the host"); how a consumer stores them afterwards is its own business."""
    rng = np.random.Generator(np.random.Philox(seed))
    D, F = cfg.D, cfg.F
    shapes = {
        "ln1_g": (D,), "ln1_b": (D,), "w_qkv": (3 * D, D), "b_qkv": (3 * D,),
        "w_o": (D, D), "b_o": (D,), "ln2_g": (D,), "ln2_b": (D,),
        "w_fc1": (F, D), "b_fc1": (F,), "w_fc2": (D, F), "b_fc2": (D,),
    }
    blocks = []
    for _ in range(cfg.L if n_blocks is None else n_blocks):
        blk = {}
        for name in BLOCK_FIELDS:
            a = rng.standard_normal(shapes[name], dtype=np.float32) * np.float32(0.02)
            if name in ("ln1_g", "ln2_g"):
                a = a + np.float32(1.0)
            if cfg.dtype == "bf16" and name in MATRIX_FIELDS:
                a = round_to_bf16(a)
            blk[name] = np.ascontiguousarray(a, dtype=np.float32)
        blocks.append(blk)
    return blocks


def peaked_weights(blocks: List[Dict[str, np.ndarray]], cfg: MarConfig, gain: float = 16.0
                   ) -> List[Dict[str, np.ndarray]]:
    """Copy of `blocks` with the query and key rows of w_qkv scaled by `gain`,
    which turns the near-uniform attention of N(0, 0.02) weights into sharply
    peaked rows (power-of-two gain keeps bf16 representability)."""
    out = []
    for blk in blocks:
        nb = dict(blk)
        w = blk["w_qkv"].copy()
        w[: 2 * cfg.D] *= np.float32(gain)
        nb["w_qkv"] = w
        out.append(nb)
    return out


def make_hidden(cfg: MarConfig, seed: int = SEED_HIDDEN, batch: int | None = None) -> np.ndarray:
    """fp32 [B][S][D] ~ N(0, 1): the stack's input rows (token embeddings plus
    positional terms are opaque to the hot path)."""
    rng = np.random.Generator(np.random.Philox(seed))
    B = cfg.B if batch is None else batch
    return rng.standard_normal((B, cfg.S, cfg.D), dtype=np.float32)


def replacement_rows(cfg: MarConfig, t: int, n_rows: int, seed: int = SEED_ROWS,
                     batch: int | None = None) -> np.ndarray:
    """fp32 [B][n_rows][D] ~ N(0, 1): stand-in for the tokens the sampler would
    produce at step t; the driver writes them over hidden[b][G(t)]."""
    rng = np.random.Generator(np.random.Philox(key=seed, counter=[t, 0, 0, 0]))
    B = cfg.B if batch is None else batch
    return rng.standard_normal((B, n_rows, cfg.D), dtype=np.float32)


SEED_MAR = 4321
MAR_FIELDS = ("enc_norm_g", "enc_norm_b", "w_dec_embed", "b_dec_embed", "mask_token", "dec_pos",
              "dec_norm_g", "dec_norm_b")


def make_mar_weights(cfg: MarConfig, seed: int = SEED_MAR) -> Dict[str, np.ndarray]:
    """fp32 arrays of the two-stage model's glue: final encoder norm, encoder-to-decoder linear map
    ([out][in]), mask embedding [D], decoder positional embedding [S][D], final decoder norm.
    Norm gains 1 + N(0, 0.02^2); the embeddings N(0, 1) and N(0, 0.02^2) like the rest; for bf16
    configs the matrix is rounded to bf16-representable values."""
    rng = np.random.Generator(np.random.Philox(seed))
    D, S = cfg.D, cfg.S
    shapes = {"enc_norm_g": (D,), "enc_norm_b": (D,), "w_dec_embed": (D, D), "b_dec_embed": (D,),
              "mask_token": (D,), "dec_pos": (S, D), "dec_norm_g": (D,), "dec_norm_b": (D,)}
    out = {}
    for name in MAR_FIELDS:
        a = rng.standard_normal(shapes[name], dtype=np.float32)
        if name not in ("mask_token", "dec_pos"):
            a = a * np.float32(0.02)
        if name.endswith("_g"):
            a = a + np.float32(1.0)
        if name == "w_dec_embed":
            # one-over-sqrt(D) scale keeps the projected rows at unit size like the mask embedding
            a = a * np.float32(50.0 / math.sqrt(D))
            if cfg.dtype == "bf16":
                a = round_to_bf16(a)
        out[name] = np.ascontiguousarray(a, dtype=np.float32)
    return out


def known_token_sets(cfg: MarConfig, new_sets: List[np.ndarray]) -> List[np.ndarray]:
    """List over steps t of int32 [B][n_known(t)], ascending: the buffer positions plus every
    position generated before step t (the tokens that are not masked at step t)."""
    B = new_sets[0].shape[0]
    known = np.tile(np.arange(cfg.n_buffer, dtype=np.int32), (B, 1))
    out = []
    for G in new_sets:
        out.append(np.ascontiguousarray(np.sort(known, axis=1)))
        known = np.concatenate([known, G.astype(np.int32)], axis=1)
    return out
