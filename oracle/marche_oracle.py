"""CPU oracle for the MARche decoding step.  TEST INFRASTRUCTURE ONLY.

This file is the slow, plain statement of what one decoding step computes.
Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may
import it; the CUDA library never does, and it shares no code with that
library (no kernels, helpers, tables or pre/post-processing).  Inputs come
from the seeded generators of the `synth` package or from the tests.

Arithmetic: NumPy, IEEE double precision throughout (`real=np.float64`); the
paper does not fix a precision.  `real=np.float32` gives the single-precision
variant, which the tests show agrees with the double one far inside the
tolerance used for the bf16 CUDA path.  `@` (matrix product) and `exp`, `erf`
are used as library primitives; there is no tiling, fusion or reordering.

What is written out, and from where in the paper:

* `softmax_attention`      standard scaled dot-product attention, Eq. 5 in the
                           max-shifted form of Eq. 11 (Appendix A).
* `two_segment_attention`  Eq. 6-10 literally: logits over the active and the
                           cached segment, shared max, exponentials, one
                           normaliser, merged output (Appendix A.2, Algorithm 1
                           lines 6-8).  Used to pin `softmax_attention`.
* `marche_step`            Algorithm 1 lines 4-11 for a stack of pre-LN blocks:
                           Q, K, V for active rows only, cached K, V for the
                           rest, attention of active queries over all tokens,
                           feed-forward for active rows only, cache write-back
                           for active rows only.
* relevance scores         Section 4.2 / Figure 3: attention probability from
                           the generating tokens' queries to every token,
                           summed over heads (and over those queries) at one
                           chosen block.
* `select_refresh`         Section 4.2: the top-K tokens by relevance score.
* `full_step`              the same stack with every token active: the initial
                           full refresh of Section 4.3 and the full-recompute
                           MAR baseline of Section 3 (Motivation).
* `active_set`             Algorithm 1 line 4: A = G u R u N.
* `in_step_selection_step` the paper's own schedule of one step (Section 4.2, Figure 3): full
                           attention up to the scoring block, selection there, cache-aware
                           blocks after it; `generate_in_step` adds the fixed active budget
                           and the periodic full refresh of Section 4.3.
* `mar_encoder`, `mar_decoder_input`, `mar_step`, `generate_mar`
                           the two-stage shape of Section 3: Eq. 1 (encoder blocks on the known
                           tokens only, nothing cached) and Eq. 2 (decoder over the whole sequence,
                           mask embedding at masked positions), with the decoder scheduled as in
                           Section 4.2 / 4.3.  Pinned by: encoder == full pass over the compacted
                           sequence, masked rows never read, closed forms of the decoder input,
                           decoder == the pinned uniform-stack functions on the same input,
                           refresh-everything == full decoder.

Readings where the paper is silent (block internals, tie rule, refresh ratio)
are listed in the repository's design notes; each is marked "reading" below.

Pins (tests/, CPU only): equivalence of the step with every token active to the
full step (Appendix A), Eq. 6-10 == Eq. 5, idempotence on unchanged input,
block-0 cache exactness, untouched rows byte-identical, score checksum H * #G,
uniform-attention closed form, peaked (one-hot) attention, brute-force top-k,
permutation/sample independence, and textbook values for LayerNorm / GELU /
linear.  Numerical agreement with the authors' own implementation and any
image-quality figure is "parity unpinned": the paper prints no numeric example
and no weights exist here.
"""
from __future__ import annotations

import math
from typing import Dict, List, Optional, Sequence

import numpy as np
from scipy.special import erf as _erf

Block = Dict[str, np.ndarray]


# --------------------------------------------------------------------------
# Building blocks (reading: standard pre-LN transformer block; the paper's
# Algorithm 1 abbreviates the block as "FFN(z)").
# --------------------------------------------------------------------------

def layer_norm(x: np.ndarray, gamma: np.ndarray, beta: np.ndarray, eps: float) -> np.ndarray:
    """Row-wise LayerNorm over the last axis: (x - mean) / sqrt(var + eps) * gamma + beta,
    biased variance."""
    mu = x.mean(axis=-1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
    return (x - mu) / np.sqrt(var + eps) * gamma + beta


def gelu(x: np.ndarray) -> np.ndarray:
    """Exact GELU: x/2 * (1 + erf(x / sqrt 2))  (reading: erf flavour, not tanh)."""
    return 0.5 * x * (1.0 + _erf(x / math.sqrt(2.0)))


def linear(x: np.ndarray, W: np.ndarray, b: np.ndarray) -> np.ndarray:
    """y = x W^T + b with W stored [out][in]."""
    return x @ W.T + b


def softmax_attention(q: np.ndarray, K: np.ndarray, V: np.ndarray):
    """Eq. 5 / Eq. 11 for one head.

    q [n][d] queries, K [N][d], V [N][d] keys/values of ALL N tokens.
    Returns (z [n][d], p [n][N]) where p are the softmax weights
    exp(q.k_j / sqrt d) / sum_l exp(q.k_l / sqrt d)."""
    d = q.shape[-1]
    s = (q @ K.T) / math.sqrt(d)
    m = s.max(axis=-1, keepdims=True)
    e = np.exp(s - m)
    p = e / e.sum(axis=-1, keepdims=True)
    return p @ V, p


def two_segment_attention(q, K_A, V_A, K_C, V_C):
    """Eq. 6-10 for one head: attention over an active segment (K_A, V_A) and a
    cached segment (K_C, V_C) merged with one shared maximum and normaliser,
    without concatenating the segments.  Either segment may be empty."""
    d = q.shape[-1]
    s_A = (q @ K_A.T) / math.sqrt(d)                                   # Eq. 6
    s_C = (q @ K_C.T) / math.sqrt(d)
    neg = np.full((q.shape[0], 1), -np.inf, dtype=s_A.dtype)
    m_A = s_A.max(axis=-1, keepdims=True) if s_A.shape[1] else neg
    m_C = s_C.max(axis=-1, keepdims=True) if s_C.shape[1] else neg
    m = np.maximum(m_A, m_C)                                           # Eq. 7
    alpha_A = np.exp(s_A - m)                                          # Eq. 8
    alpha_C = np.exp(s_C - m)
    ell = alpha_A.sum(axis=-1, keepdims=True) + alpha_C.sum(axis=-1, keepdims=True)  # Eq. 9
    return (alpha_A @ V_A + alpha_C @ V_C) / ell                       # Eq. 10


# --------------------------------------------------------------------------
# State
# --------------------------------------------------------------------------

class KVCache:
    """Per block, per sample, per token: (K_i, V_i) from the last step in which
    token i was active (Algorithm 1 line 11).  Arrays are [L][B][S][D]."""

    def __init__(self, L: int, B: int, S: int, D: int, real=np.float64):
        self.K = np.zeros((L, B, S, D), dtype=real)
        self.V = np.zeros((L, B, S, D), dtype=real)
        self.filled = False

    def copy(self) -> "KVCache":
        c = KVCache.__new__(KVCache)
        c.K, c.V, c.filled = self.K.copy(), self.V.copy(), self.filled
        return c


# --------------------------------------------------------------------------
# Set bookkeeping and selection
# --------------------------------------------------------------------------

def active_set(G: np.ndarray, N: Optional[np.ndarray], R: Optional[np.ndarray]) -> np.ndarray:
    """Algorithm 1 line 4: A = G u N u R per sample, as int32 [B][#G+#N+#R] in
    that order (generating, caching, refreshing).  The three sets must be
    disjoint per sample."""
    parts = [np.asarray(G, dtype=np.int32)]
    for extra in (N, R):
        if extra is not None and extra.shape[1] > 0:
            parts.append(np.asarray(extra, dtype=np.int32))
    A = np.concatenate(parts, axis=1)
    for b in range(A.shape[0]):
        if len(set(A[b].tolist())) != A.shape[1]:
            raise ValueError("active sets overlap in sample %d" % b)
    return A


def refresh_count(refresh_ratio: float, S: int, n_candidates: int) -> int:
    """Reading: K = min(#candidates, floor(ratio * S + 1/2))."""
    return int(min(n_candidates, math.floor(float(refresh_ratio) * S + 0.5)))


def fixed_budget_refresh_count(budget: int, n_generating: int, n_caching: int) -> int:
    """Section 4.3: the active set is filled up to a fixed budget, so the number of
    refreshing tokens is what the generating and caching tokens leave over."""
    return max(0, int(budget) - int(n_generating) - int(n_caching))


def _mix32(seed: int, b: int, t: int) -> int:
    """Counter-based 32-bit hash of (seed, sample, token) for the random-selection ablation."""
    M = 0xFFFFFFFF
    x = (seed ^ (b * 0x9E3779B1) ^ (t * 0x85EBCA77)) & M
    x ^= x >> 16
    x = (x * 0x7FEB352D) & M
    x ^= x >> 15
    x = (x * 0x846CA68B) & M
    x ^= x >> 16
    return x


def select_refresh(scores: np.ndarray, new_idx: np.ndarray, exclude_idx: Optional[np.ndarray],
                   k: int, policy: str = "high", seed: int = 0) -> np.ndarray:
    """Section 4.2: the k candidate tokens with the highest relevance score.

    scores fp32 [B][S].  Candidates are all tokens not in new_idx[b] or
    exclude_idx[b].  Reading (the paper gives no tie rule): rank by score
    descending, then token index ascending; the result is int32 [B][k] in
    ascending index order.  Done by a full sort.  `policy` "low" / "random" are the selection
    ablations of Section 5.3 (lowest scores first; order by a hash of seed, sample and token)."""
    scores = np.asarray(scores, dtype=np.float32)
    B, S = scores.shape
    out = np.zeros((B, k), dtype=np.int32)
    for b in range(B):
        banned = set(np.asarray(new_idx[b]).tolist())
        if exclude_idx is not None:
            banned |= set(np.asarray(exclude_idx[b]).tolist())
        cand = [t for t in range(S) if t not in banned]
        if k > len(cand):
            raise ValueError("k exceeds the number of candidates")
        if policy == "high":            # the method: highest relevance first
            ranked = sorted(cand, key=lambda t: (-float(scores[b, t]), t))
        elif policy == "low":           # ablation (Section 5.3): lowest attention first
            ranked = sorted(cand, key=lambda t: (float(scores[b, t]) + 0.0, t))
        elif policy == "random":        # ablation: random candidates
            ranked = sorted(cand, key=lambda t: (_mix32(seed, b, t), t))
        else:
            raise ValueError("unknown policy")
        out[b] = np.array(sorted(ranked[:k]), dtype=np.int32)
    return out


# --------------------------------------------------------------------------
# The step
# --------------------------------------------------------------------------

def _block(X, blk, K_l, V_l, idx, n_heads, eps, scoring_rows):
    """One pre-LN block for one sample.

    X [nA][D] residual rows of the active tokens `idx`; K_l, V_l [S][D] this
    block's cache for the sample (updated in place at rows `idx`).  Returns the
    new X and, when `scoring_rows` (bool [nA]) is given, the per-token sum over
    heads and scoring queries of the attention probabilities."""
    D = X.shape[1]
    dh = D // n_heads
    U = layer_norm(X, blk["ln1_g"], blk["ln1_b"], eps)
    QKV = linear(U, blk["w_qkv"], blk["b_qkv"])            # Algorithm 1 line 5 (active rows only)
    Q, Kn, Vn = QKV[:, :D], QKV[:, D:2 * D], QKV[:, 2 * D:]
    K_l[idx] = Kn                                          # Algorithm 1 line 11; done first so that
    V_l[idx] = Vn                                          # the attention below sees fresh K_A, V_A
    O = np.empty_like(X)
    score = np.zeros(K_l.shape[0], dtype=X.dtype) if scoring_rows is not None else None
    for h in range(n_heads):
        c = slice(h * dh, (h + 1) * dh)
        z, p = softmax_attention(Q[:, c], K_l[:, c], V_l[:, c])   # lines 6-8 == Eq. 5 (Appendix A)
        O[:, c] = z
        if score is not None:
            score += p[scoring_rows].sum(axis=0)
    X = X + linear(O, blk["w_o"], blk["b_o"])
    U2 = layer_norm(X, blk["ln2_g"], blk["ln2_b"], eps)
    X = X + linear(gelu(linear(U2, blk["w_fc1"], blk["b_fc1"])), blk["w_fc2"], blk["b_fc2"])  # line 9
    return X, score


def marche_step(blocks: Sequence[Block], hidden: np.ndarray, cache: KVCache,
                active_idx: np.ndarray, new_idx: np.ndarray, exclude_idx: Optional[np.ndarray],
                refresh_ratio: float, hidden_out: np.ndarray, *, n_heads: int, score_layer: int,
                ln_eps: float = 1e-6, real=np.float64, require_filled: bool = True,
                layer_scores: Optional[Dict[int, np.ndarray]] = None):
    """One cache-aware decoding step (Algorithm 1), every sample independently.

    hidden fp32 [B][S][D]; active_idx int32 [B][nA]; new_idx int32 [B][nG]
    (subset of active_idx: the generating tokens, whose queries score);
    exclude_idx int32 [B][nX] or None.  Rows `active_idx` of `hidden_out`
    ([B][S][D], modified in place) receive the stack output; every other row of
    `hidden_out` and of the cache keeps its bytes.
    `layer_scores`, when given, is a dict whose keys are block indices; each value is replaced by
    that block's relevance scores fp32 [B][S] (same definition as at score_layer; for the top-K
    overlap statistics across layers of Section 5.3).
    Returns (scores fp32 [B][S], refresh_idx int32 [B][k])."""
    if require_filled and not cache.filled:
        raise RuntimeError("cache-aware step before any full step")
    B, S, D = hidden.shape
    L = len(blocks)
    blocks = [{k: np.asarray(v, dtype=real) for k, v in blk.items()} for blk in blocks]
    scores = np.zeros((B, S), dtype=real)
    extra = {l: np.zeros((B, S), dtype=real) for l in (layer_scores or {})}
    for b in range(B):
        idx = np.asarray(active_idx[b], dtype=np.int64)
        if len(set(idx.tolist())) != len(idx) or idx.min() < 0 or idx.max() >= S:
            raise ValueError("active_idx must be unique and in range")
        new = set(np.asarray(new_idx[b]).tolist())
        if not new <= set(idx.tolist()):
            raise ValueError("new_idx must be a subset of active_idx")
        scoring_rows = np.array([int(t) in new for t in idx], dtype=bool)
        X = hidden[b, idx].astype(real)
        for l in range(L):
            wanted = l == score_layer or (layer_scores is not None and l in layer_scores)
            X, sc = _block(X, blocks[l], cache.K[l, b], cache.V[l, b], idx, n_heads, ln_eps,
                           scoring_rows if wanted else None)
            if sc is not None and l == score_layer:
                scores[b] = sc
            if sc is not None and layer_scores is not None and l in layer_scores:
                extra[l][b] = sc
        hidden_out[b, idx] = X.astype(hidden_out.dtype)
    scores32 = scores.astype(np.float32)
    for l in extra:
        layer_scores[l] = extra[l].astype(np.float32)
    n_new = new_idx.shape[1]
    n_excl = 0 if exclude_idx is None else exclude_idx.shape[1]
    k = refresh_count(refresh_ratio, S, S - n_new - n_excl)
    return scores32, select_refresh(scores32, new_idx, exclude_idx, k)


def full_step(blocks, hidden, cache: KVCache, new_idx, exclude_idx, refresh_ratio, hidden_out, *,
              n_heads, score_layer, ln_eps=1e-6, real=np.float64, layer_scores=None):
    """Every token active: fills the cache (initial full refresh, Section 4.3) and
    is the full-recompute baseline (every token recomputed at every step)."""
    B, S, _ = hidden.shape
    all_idx = np.tile(np.arange(S, dtype=np.int32), (B, 1))
    out = marche_step(blocks, hidden, cache, all_idx, new_idx, exclude_idx, refresh_ratio, hidden_out,
                      n_heads=n_heads, score_layer=score_layer, ln_eps=ln_eps, real=real,
                      require_filled=False, layer_scores=layer_scores)
    cache.filled = True
    return out


def in_step_selection_step(blocks: Sequence[Block], hidden: np.ndarray, cache: KVCache, new_idx: np.ndarray,
                           prev_idx: Optional[np.ndarray], n_refresh: int, hidden_out: np.ndarray, *,
                           n_heads: int, score_layer: int, ln_eps: float = 1e-6, real=np.float64,
                           forced_refresh: Optional[np.ndarray] = None):
    """One decoding step under the paper's own schedule (Section 4.2, Figure 3; Section 4.3):

    blocks 0 .. score_layer run full attention on every token ("the active tokens are not yet
    finalized"), the relevance scores are taken from the generating tokens' queries at block
    score_layer, the n_refresh highest-scoring tokens outside G u N become the refreshing tokens R,
    and the blocks after score_layer run cache-aware attention on A = G u N u R.
    new_idx = G [B][nG], prev_idx = N [B][nN] (the tokens generated in the previous step) or None.
    `forced_refresh` [B][n_refresh], when given, is used as R instead of the selection (the
    selection is still returned).  Rows A of hidden_out receive the stack output.
    Returns (scores fp32 [B][S], refresh_idx int32 [B][n_refresh], active_idx int32 [B][nA])."""
    if not cache.filled:
        raise RuntimeError("step before any full step")
    B, S, D = hidden.shape
    L = len(blocks)
    if not (0 <= score_layer < L - 1):
        raise ValueError("score_layer must leave at least one cache-aware block")
    blocks = [{k: np.asarray(v, dtype=real) for k, v in blk.items()} for blk in blocks]
    all_idx = np.arange(S, dtype=np.int64)
    scores = np.zeros((B, S), dtype=real)
    X_full = []
    for b in range(B):
        new = set(np.asarray(new_idx[b]).tolist())
        scoring_rows = np.array([t in new for t in range(S)], dtype=bool)
        X = hidden[b].astype(real)
        for l in range(score_layer + 1):
            X, sc = _block(X, blocks[l], cache.K[l, b], cache.V[l, b], all_idx, n_heads, ln_eps,
                           scoring_rows if l == score_layer else None)
            if sc is not None:
                scores[b] = sc
        X_full.append(X)
    scores32 = scores.astype(np.float32)
    refresh = select_refresh(scores32, new_idx, prev_idx, n_refresh)
    R = refresh if forced_refresh is None else np.asarray(forced_refresh, dtype=np.int32)
    A = active_set(new_idx, prev_idx, R)
    for b in range(B):
        idx = A[b].astype(np.int64)
        X = X_full[b][idx]
        for l in range(score_layer + 1, L):
            X, _ = _block(X, blocks[l], cache.K[l, b], cache.V[l, b], idx, n_heads, ln_eps, None)
        hidden_out[b, idx] = X.astype(hidden_out.dtype)
    return scores32, refresh, A


def generate_in_step(blocks, hidden0: np.ndarray, new_sets: List[np.ndarray], replacement, *, n_heads: int,
                     score_layer: int, budget: int = 64, period: int = 3, ln_eps: float = 1e-6, real=np.float64):
    """The paper's schedule over a whole generation (Section 4.3): the first step and every
    `period`-th step refresh the whole cache with a full step; the others use
    in_step_selection_step with a fixed active budget, K = budget - #G - #N (clipped to the
    number of candidates).  Returns per-step dicts and the final cache."""
    B, S, D = hidden0.shape
    hidden = hidden0.copy()
    hidden_out = np.zeros_like(hidden0)
    cache = KVCache(len(blocks), B, S, D, real=real)
    empty = np.zeros((B, 0), dtype=np.int32)
    log = []
    kw = dict(n_heads=n_heads, score_layer=score_layer, ln_eps=ln_eps, real=real)
    for t, G in enumerate(new_sets):
        N = new_sets[t - 1] if t > 0 else empty
        if t % period == 0:
            A = np.tile(np.arange(S, dtype=np.int32), (B, 1))
            scores, _ = full_step(blocks, hidden, cache, G, None, 0.0, hidden_out, **kw)
            R = empty
            kind = "full"
        else:
            k = min(fixed_budget_refresh_count(budget, G.shape[1], N.shape[1]), S - G.shape[1] - N.shape[1])
            scores, R, A = in_step_selection_step(blocks, hidden, cache, G, N, k, hidden_out, **kw)
            kind = "in_step"
        log.append(dict(t=t, kind=kind, active=A, new=G, prev=N, scores=scores, refresh=R,
                        hidden_out=hidden_out.copy()))
        rows = replacement(t, G.shape[1])
        for b in range(B):
            hidden[b, G[b]] = rows[b]
    return log, cache


# --------------------------------------------------------------------------
# T-step synthetic generation driver (set bookkeeping of Section 3 and 4.1;
# the sampler of Eq. 3 is replaced by caller-supplied rows).
# --------------------------------------------------------------------------

def generate(blocks, hidden0: np.ndarray, new_sets: List[np.ndarray], replacement, refresh_ratio: float,
             *, n_heads: int, score_layer: int, ln_eps: float = 1e-6, mode: str = "marche",
             real=np.float64, forced_refresh: Optional[List[np.ndarray]] = None):
    """Run len(new_sets) decoding steps.

    Step 0 is a full step (the cache is empty).  Step t >= 1 is cache-aware with
    A(t) = G(t) u G(t-1) u R(t), where R(t) was selected at step t-1 with
    G(t) excluded from the candidates; mode="full" runs a full step every time.
    After step t, rows G(t) of the stack input are overwritten by
    replacement(t, #G(t)) -> fp32 [B][#G(t)][D].  `forced_refresh[t]`, when
    given, replaces the refresh set selected for step t+1 (teacher forcing).
    Returns a list of per-step dicts with the sets used and the outputs."""
    B, S, D = hidden0.shape
    hidden = hidden0.copy()
    hidden_out = np.zeros_like(hidden0)
    cache = KVCache(len(blocks), B, S, D, real=real)
    empty = np.zeros((B, 0), dtype=np.int32)
    R = empty
    log = []
    T = len(new_sets)
    for t in range(T):
        G = new_sets[t]
        X = new_sets[t + 1] if t + 1 < T else empty
        kw = dict(n_heads=n_heads, score_layer=score_layer, ln_eps=ln_eps, real=real)
        if t == 0 or mode == "full":
            A = np.tile(np.arange(S, dtype=np.int32), (B, 1))
            scores, R_next = full_step(blocks, hidden, cache, G, X, refresh_ratio, hidden_out, **kw)
        else:
            A = active_set(G, new_sets[t - 1], R)
            scores, R_next = marche_step(blocks, hidden, cache, A, G, X, refresh_ratio, hidden_out, **kw)
        if forced_refresh is not None:
            R_next = forced_refresh[t]
        log.append(dict(t=t, active=A, new=G, exclude=X, scores=scores, refresh=R_next,
                        hidden_in=hidden.copy(), hidden_out=hidden_out.copy()))
        rows = replacement(t, G.shape[1])
        for b in range(B):
            hidden[b, G[b]] = rows[b]
        R = R_next
    return log, cache


# --------------------------------------------------------------------------
# MAR's two-stage shape (Section 3, Eq. 1 and Eq. 2): an encoder over the known
# tokens only, then a decoder over the whole sequence with mask embeddings.
# --------------------------------------------------------------------------

def mar_encoder(blocks: Sequence[Block], tokens_b: np.ndarray, known: np.ndarray, *, n_heads: int,
                ln_eps: float) -> np.ndarray:
    """Eq. 1 for one sample: the encoder blocks on the rows `known` of tokens_b [S][D] alone.
    Keys and values are those of the known tokens of this very step; nothing is cached
    (reading: the paper speaks of cached projections only for decoder layers).
    Returns the encoder output rows [n_known][D] before the encoder's final norm."""
    X = tokens_b[known]
    n = len(known)
    own = np.arange(n, dtype=np.int64)
    for blk in blocks:
        K_l = np.zeros((n, X.shape[1]), dtype=X.dtype)
        V_l = np.zeros_like(K_l)
        X, _ = _block(X, blk, K_l, V_l, own, n_heads, ln_eps, None)
    return X


def mar_decoder_input(h_enc: np.ndarray, known: np.ndarray, S: int, mar: Dict[str, np.ndarray],
                      ln_eps: float) -> np.ndarray:
    """The decoder's input of Eq. 2 for one sample, [S][D]: at a known position the encoder
    output, normalised and projected to the decoder (reading: MAR's final encoder norm and its
    encoder-to-decoder linear map), at a masked position the learned mask embedding; the
    decoder's positional embedding is added to every position."""
    X = np.tile(mar["mask_token"], (S, 1))
    X[known] = linear(layer_norm(h_enc, mar["enc_norm_g"], mar["enc_norm_b"], ln_eps),
                      mar["w_dec_embed"], mar["b_dec_embed"])
    return X + mar["dec_pos"]


def mar_step(blocks: Sequence[Block], mar: Dict[str, np.ndarray], tokens: np.ndarray, known_idx: np.ndarray,
             cache: KVCache, new_idx: np.ndarray, prev_idx: Optional[np.ndarray], n_refresh: int,
             z_out: np.ndarray, *, n_heads: int, n_enc: int, score_layer: int, full_decoder: bool,
             ln_eps: float = 1e-6, real=np.float64, forced_refresh: Optional[np.ndarray] = None):
    """One decoding step of the two-stage model (Eq. 1, Eq. 2) with the cache-aware decoder.

    blocks[:n_enc] are the encoder, blocks[n_enc:] the decoder; cache rows of the encoder
    blocks are not used.  tokens [B][S][D] holds the embedded known tokens (rows outside
    known_idx are ignored); known_idx int32 [B][n_known] ascending.
    full_decoder: every decoder block on every token (first step, periodic full refresh of
    Section 4.3).  Otherwise the schedule of Section 4.2: decoder blocks up to score_layer on
    every token, top-n_refresh selection there with G and N excluded, A = G u N u R afterwards.
    Rows A (all rows when full_decoder) of z_out [B][S][D] receive the decoder output after
    the decoder's final norm.
    Returns (scores fp32 [B][S], refresh_idx int32 [B][n_refresh], active_idx int32 [B][nA])."""
    B, S, D = tokens.shape
    L = len(blocks)
    if not (n_enc <= score_layer < L):
        raise ValueError("score_layer must be a decoder block")
    if not full_decoder and (not cache.filled or score_layer >= L - 1):
        raise RuntimeError("cache-aware decoder needs a filled cache and a block after score_layer")
    blocks = [{k: np.asarray(v, dtype=real) for k, v in blk.items()} for blk in blocks]
    mar = {k: np.asarray(v, dtype=real) for k, v in mar.items()}
    all_idx = np.arange(S, dtype=np.int64)
    last_full = L - 1 if full_decoder else score_layer
    scores = np.zeros((B, S), dtype=real)
    X_full = []
    for b in range(B):
        known = np.asarray(known_idx[b], dtype=np.int64)
        h_enc = mar_encoder(blocks[:n_enc], tokens[b].astype(real), known, n_heads=n_heads, ln_eps=ln_eps)
        X = mar_decoder_input(h_enc, known, S, mar, ln_eps)
        new = set(np.asarray(new_idx[b]).tolist())
        scoring_rows = np.array([t in new for t in range(S)], dtype=bool)
        for l in range(n_enc, last_full + 1):
            X, sc = _block(X, blocks[l], cache.K[l, b], cache.V[l, b], all_idx, n_heads, ln_eps,
                           scoring_rows if l == score_layer else None)
            if sc is not None:
                scores[b] = sc
        X_full.append(X)
    scores32 = scores.astype(np.float32)
    refresh = select_refresh(scores32, new_idx, prev_idx, n_refresh)
    if full_decoder:
        cache.filled = True
        A = np.tile(np.arange(S, dtype=np.int32), (B, 1))
        for b in range(B):
            z_out[b] = layer_norm(X_full[b], mar["dec_norm_g"], mar["dec_norm_b"], ln_eps).astype(z_out.dtype)
        return scores32, refresh, A
    R = refresh if forced_refresh is None else np.asarray(forced_refresh, dtype=np.int32)
    A = active_set(new_idx, prev_idx, R)
    for b in range(B):
        idx = A[b].astype(np.int64)
        X = X_full[b][idx]
        for l in range(score_layer + 1, L):
            X, _ = _block(X, blocks[l], cache.K[l, b], cache.V[l, b], idx, n_heads, ln_eps, None)
        z_out[b, idx] = layer_norm(X, mar["dec_norm_g"], mar["dec_norm_b"], ln_eps).astype(z_out.dtype)
    return scores32, refresh, A


def generate_mar(blocks, mar, tokens0: np.ndarray, new_sets: List[np.ndarray], known_sets: List[np.ndarray],
                 replacement, *, n_heads: int, n_enc: int, score_layer: int, budget: int = 64, period: int = 3,
                 ln_eps: float = 1e-6, real=np.float64):
    """A whole generation of the two-stage model under the schedule of Section 4.3: the decoder is
    fully refreshed at the first and at every `period`-th step, otherwise it runs the in-step
    selection with the fixed active budget K = budget - #G - #N.  After step t, rows G(t) of the
    token embeddings are overwritten by replacement(t, #G(t)) and count as known from then on."""
    B, S, D = tokens0.shape
    tokens = tokens0.copy()
    z = np.zeros_like(tokens0)
    cache = KVCache(len(blocks), B, S, D, real=real)
    empty = np.zeros((B, 0), dtype=np.int32)
    log = []
    for t, G in enumerate(new_sets):
        N = new_sets[t - 1] if t > 0 else empty
        full = t % period == 0
        k = 0 if full else min(fixed_budget_refresh_count(budget, G.shape[1], N.shape[1]),
                               S - G.shape[1] - N.shape[1])
        scores, R, A = mar_step(blocks, mar, tokens, known_sets[t], cache, G, N, k, z, n_heads=n_heads,
                                n_enc=n_enc, score_layer=score_layer, full_decoder=full, ln_eps=ln_eps, real=real)
        log.append(dict(t=t, kind="full" if full else "in_step", active=A, new=G, prev=N, scores=scores,
                        refresh=R, z=z.copy()))
        rows = replacement(t, G.shape[1])
        for b in range(B):
            tokens[b, G[b]] = rows[b]
    return log, cache
