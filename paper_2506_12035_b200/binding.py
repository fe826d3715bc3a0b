"""ctypes binding of libmarche.so: one Python method per C-ABI entry point.

Argument marshalling only - every step of the hot path runs inside the
library's CUDA kernels.  PyTorch tensors provide device memory and streams.
There is no fallback: if the shared library is missing or a call fails, an
exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmarche.so")

MARCHE_F32, MARCHE_BF16, MARCHE_BF16_F16OP = 0, 1, 2
ATTENTION_AUTO, ATTENTION_MMA, ATTENTION_TCGEN05, ATTENTION_TCGEN05_TWO_PASS = 0, 1, 2, 3
GEMM_AUTO, GEMM_SINGLE, GEMM_PAIR = 0, 1, 2
EPI_BIAS, EPI_BIAS_RESIDUAL, EPI_BIAS_GELU = 0, 1, 2
ERRORS = {-1: "EINVAL", -2: "ESHAPE", -3: "EWORKSPACE", -4: "ECACHE", -5: "EINDEX", -6: "ECUDA", -7: "ETIMEOUT"}

BLOCK_FIELDS = ("ln1_g", "ln1_b", "w_qkv", "b_qkv", "w_o", "b_o",
                "ln2_g", "ln2_b", "w_fc1", "b_fc1", "w_fc2", "b_fc2")
MATRIX_FIELDS = ("w_qkv", "w_o", "w_fc1", "w_fc2")


class MarcheConfig(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_blocks", "n_enc_blocks", "width", "n_heads", "head_dim", "mlp_dim",
                                         "seq_len", "n_buffer", "batch", "dtype", "score_layer")] + [("ln_eps", C.c_float)]


class MarcheBlockWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in BLOCK_FIELDS]


MAR_FIELDS = ("enc_norm_g", "enc_norm_b", "w_dec_embed", "b_dec_embed", "mask_token", "dec_pos",
              "dec_norm_g", "dec_norm_b")


class MarcheMarWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in MAR_FIELDS]


class MarcheTuning(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("stream_k", "fuse_qkv_scatter", "attention_kernel", "attention_tc_min_rows",
                                         "two_segment_attention", "gemm_kernel", "tail_split", "tile_n", "pdl")]


class MarcheError(RuntimeError):
    def __init__(self, code: int, detail: str = ""):
        self.code = code
        super().__init__("libmarche: %s (%d) %s" % (ERRORS.get(code, "?"), code, detail))


_vp, _i, _f, _sz = C.c_void_p, C.c_int, C.c_float, C.c_size_t
_SIGNATURES = {
    "marche_create": (C.c_int, [C.POINTER(MarcheConfig), C.POINTER(MarcheBlockWeights), C.POINTER(_vp)]),
    "marche_destroy": (None, [_vp]),
    "marche_cache_bytes": (_sz, [_vp]),
    "marche_workspace_bytes": (_sz, [_vp, _i]),
    "marche_init_cache": (C.c_int, [_vp, _vp, _sz, _vp]),
    "marche_step": (C.c_int, [_vp, _vp, _vp, _vp, _i, _vp, _i, _vp, _i, _f, _vp, _vp, C.POINTER(C.c_int), _vp, _sz, _vp]),
    "marche_full_step": (C.c_int, [_vp, _vp, _vp, _vp, _i, _vp, _i, _f, _vp, _vp, C.POINTER(C.c_int), _vp, _sz, _vp]),
    "marche_step_in_step_selection": (C.c_int, [_vp, _vp, _vp, _vp, _i, _vp, _i, _i, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "marche_set_mar_weights": (C.c_int, [_vp, C.POINTER(MarcheMarWeights)]),
    "marche_mar_step": (C.c_int, [_vp, _i, _vp, _vp, _i, _vp, _vp, _i, _vp, _i, _i, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "marche_select_refresh": (C.c_int, [_vp, _vp, _vp, _i, _vp, _i, _i, _vp, _vp, _vp]),
    "marche_select_refresh_policy": (C.c_int, [_vp, _vp, _vp, _i, _vp, _i, _i, _i, C.c_uint32, _vp, _vp, _vp]),
    "marche_select_refresh_static": (C.c_int, [_vp, _vp, _vp, _i, _vp, _i, _i, _vp, _vp]),
    "marche_get_scores": (C.c_int, [_vp, _vp, _vp, _vp]),
    "marche_set_score_layers": (C.c_int, [_vp, C.POINTER(C.c_int32), _i]),
    "marche_get_layer_scores": (C.c_int, [_vp, _vp, _i, _vp, _vp]),
    "marche_build_active": (C.c_int, [_vp, _vp, _i, _vp, _i, _vp, _i, _vp, _vp]),
    "marche_scatter_rows": (C.c_int, [_vp, _vp, _vp, _i, _vp, _vp]),
    "marche_validate_indices": (C.c_int, [_vp, _vp, _i, _vp, _i, _vp, _i, _vp]),
    "marche_gather_layernorm": (C.c_int, [_vp, _vp, _i, _vp, _i, _vp, _vp, _vp, _vp, _vp]),
    "marche_linear": (C.c_int, [_vp, _vp, _i, _i, _vp, _vp, _i, _i, _i, _vp, _vp]),
    "marche_scatter_kv": (C.c_int, [_vp, _vp, _vp, _i, _vp, _i, _vp, _vp]),
    "marche_attention": (C.c_int, [_vp, _vp, _i, _i, _vp, _vp, _vp, _vp, _vp]),
    "marche_attention_two_segment": (C.c_int, [_vp, _vp, _i, _i, _vp, _vp, _vp, _vp, _vp, _vp]),
    "marche_gather_rows": (C.c_int, [_vp, _vp, _vp, _i, _vp, _vp]),
    "marche_staging_bytes": (_sz, [_vp, _i]),
    "marche_step_host": (C.c_int, [_vp, _i, _vp, _vp, _vp, _vp, _i, _vp, _i, _vp, _i, _vp, _i, _f, _vp, _vp, _vp, _vp,
                                   C.POINTER(C.c_int), _i, _vp, _sz, _vp, _sz, _vp]),
    "marche_launch_count": (C.c_ulonglong, [_vp]),
    "marche_profile_begin": (C.c_int, [_vp]),
    "marche_profile_end": (C.c_int, [_vp, _vp, C.POINTER(C.c_float), C.POINTER(C.c_int)]),
    "marche_kernel_class_name": (C.c_char_p, [C.c_int]),
    "marche_strerror": (C.c_char_p, [C.c_int]),
    "marche_last_error": (C.c_char_p, [_vp]),
    "marche_device_status": (C.c_int, [_vp]),
    "marche_clear_device_status": (None, [_vp]),
    "marche_get_tuning": (C.c_int, [_vp, C.POINTER(MarcheTuning)]),
    "marche_set_tuning": (C.c_int, [_vp, C.POINTER(MarcheTuning)]),
    "marche_check_status": (C.c_int, [_vp, _vp]),
    "marche_debug_bounded_wait": (C.c_int, [_vp, C.c_longlong, _vp]),
    "marche_debug_skip_classes": (C.c_int, [_vp, C.c_uint]),
    "marche_debug_repeat_classes": (C.c_int, [_vp, C.c_uint]),
}
EXPORTED_SYMBOLS = tuple(_SIGNATURES)

_lib = None


def load_library() -> C.CDLL:
    """Loads libmarche.so (built in-tree by paper_2506_12035_b200.build); raises if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                "%s not found: build it with `python -m paper_2506_12035_b200.build` (no fallback exists)" % LIB_PATH)
        lib = C.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device-resident contiguous tensor required"
    return t.data_ptr()


def _stream(stream: Optional[torch.cuda.Stream]) -> Optional[int]:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream or None


def _operand_dtype(dtype: str, operand: str) -> torch.dtype:
    if dtype != "bf16":
        return torch.float32
    if operand not in ("f16", "bf16"):
        raise ValueError("operand must be 'f16' or 'bf16'")
    return torch.float16 if operand == "f16" else torch.bfloat16


def _as_operand(t: torch.Tensor, mt: torch.dtype, name: str, device) -> torch.Tensor:
    out = t.to(device=device, dtype=mt).contiguous()
    if mt == torch.float16 and not bool(torch.isfinite(out).all()):
        raise ValueError("%s does not fit IEEE fp16 (|value| > 65504); use operand='bf16'" % name)
    return out


def upload_weights(blocks: Sequence[Dict], dtype: str, device="cuda", operand: str = "f16") -> List[Dict[str, torch.Tensor]]:
    """Copies per-block parameter arrays (NumPy or torch, fp32) to the device: the four matrices
    in the projections' operand type (16-bit contexts: fp16 for operand "f16", bf16 for "bf16";
    fp32 otherwise), LayerNorm parameters and biases in fp32."""
    mt = _operand_dtype(dtype, operand)
    out = []
    for blk in blocks:
        d = {}
        for name in BLOCK_FIELDS:
            t = torch.as_tensor(blk[name])
            d[name] = _as_operand(t, mt, name, device) if name in MATRIX_FIELDS else \
                t.to(device=device, dtype=torch.float32).contiguous()
        out.append(d)
    return out


def upload_mar_weights(mar: Dict, dtype: str, device="cuda", operand: str = "f16") -> Dict[str, torch.Tensor]:
    """Copies the two-stage model's glue parameters to the device (the encoder-to-decoder matrix
    as a projection operand, everything else fp32)."""
    mt = _operand_dtype(dtype, operand)
    return {name: (_as_operand(torch.as_tensor(mar[name]), mt, name, device) if name == "w_dec_embed" else
                   torch.as_tensor(mar[name]).to(device=device, dtype=torch.float32).contiguous())
            for name in MAR_FIELDS}


class Marche:
    """One model shape on the current CUDA device.  Methods carry the names of the C
    calls without the `marche_` prefix and take torch CUDA tensors.  dtype "f32" or "bf16"; for
    "bf16" the projections' operand type is taken from the weight matrices handed over (fp16 ->
    MARCHE_BF16_F16OP, bf16 -> MARCHE_BF16)."""

    def __init__(self, *, L: int, E: int, D: int, H: int, F: int, S: int, B: int, dtype: str,
                 weights: Sequence[Dict[str, torch.Tensor]], n_buffer: int = 0, score_layer: int = -1,
                 ln_eps: float = 1e-6):
        if not torch.cuda.is_available():
            raise RuntimeError("libmarche needs a CUDA device; there is no CPU path")
        self.lib = load_library()
        self.L, self.E, self.D, self.H, self.F, self.S, self.B = L, E, D, H, F, S, B
        self.dtype = dtype
        self.torch_dtype = torch.bfloat16 if dtype == "bf16" else torch.float32      # q/k/v, K/V cache
        self.operand_dtype = weights[0]["w_qkv"].dtype if dtype == "bf16" else torch.float32   # projection operands
        assert self.operand_dtype in ((torch.float16, torch.bfloat16) if dtype == "bf16" else (torch.float32,))
        code = MARCHE_F32 if dtype != "bf16" else (MARCHE_BF16 if self.operand_dtype == torch.bfloat16 else MARCHE_BF16_F16OP)
        self.weights = list(weights)          # keeps the device tensors alive
        assert len(self.weights) == L
        cfg = MarcheConfig(L, E, D, H, D // H, F, S, n_buffer, B, code, score_layer, ln_eps)
        arr = (MarcheBlockWeights * L)()
        for l, blk in enumerate(self.weights):
            for name in BLOCK_FIELDS:
                t = blk[name]
                want = self.operand_dtype if name in MATRIX_FIELDS else torch.float32
                assert t.is_cuda and t.is_contiguous() and t.dtype == want, name
                setattr(arr[l], name, t.data_ptr())
        h = C.c_void_p()
        self._check(self.lib.marche_create(C.byref(cfg), arr, C.byref(h)), None)
        self.h = h

    @classmethod
    def from_config(cls, cfg, weights, **kw) -> "Marche":
        """cfg: any object with attributes L, E, D, H, F, S, B, n_buffer, dtype, ln_eps."""
        return cls(L=cfg.L, E=cfg.E, D=cfg.D, H=cfg.H, F=cfg.F, S=cfg.S, B=cfg.B, dtype=cfg.dtype, weights=weights,
                   n_buffer=cfg.n_buffer, ln_eps=cfg.ln_eps, **kw)

    def __del__(self):
        h = getattr(self, "h", None)
        if h:
            self.lib.marche_destroy(h)
            self.h = None

    def _check(self, rc: int, h="self"):
        if rc != 0:
            detail = ""
            if h == "self" and rc in (-1, -6):
                detail = self.lib.marche_last_error(self.h).decode()
            raise MarcheError(rc, detail)

    # ------------------------------------------------------------- sizes and buffers
    def cache_bytes(self) -> int:
        return self.lib.marche_cache_bytes(self.h)

    def workspace_bytes(self, max_active: int) -> int:
        return self.lib.marche_workspace_bytes(self.h, max_active)

    def alloc_cache(self) -> torch.Tensor:
        return torch.empty(self.L, 2, self.B, self.S, self.D, dtype=self.torch_dtype, device="cuda")

    def alloc_workspace(self, max_active: int) -> torch.Tensor:
        return torch.empty(self.workspace_bytes(max_active), dtype=torch.uint8, device="cuda")

    # ------------------------------------------------------------- C calls
    def init_cache(self, kv_cache, stream=None):
        self._check(self.lib.marche_init_cache(self.h, _ptr(kv_cache), kv_cache.numel() * kv_cache.element_size(),
                                               _stream(stream)))

    def step(self, hidden, kv_cache, active_idx, new_idx, exclude_idx, refresh_ratio, hidden_out, refresh_idx,
             workspace, stream=None) -> int:
        k = C.c_int(0)
        self._check(self.lib.marche_step(
            self.h, _ptr(hidden), _ptr(kv_cache), _ptr(active_idx), active_idx.shape[1],
            _ptr(new_idx), 0 if new_idx is None else new_idx.shape[1],
            _ptr(exclude_idx), 0 if exclude_idx is None else exclude_idx.shape[1],
            refresh_ratio, _ptr(hidden_out), _ptr(refresh_idx), C.byref(k), _ptr(workspace), workspace.numel(),
            _stream(stream)))
        return k.value

    def full_step(self, hidden, kv_cache, new_idx, exclude_idx, refresh_ratio, hidden_out, refresh_idx, workspace,
                  stream=None) -> int:
        k = C.c_int(0)
        self._check(self.lib.marche_full_step(
            self.h, _ptr(hidden), _ptr(kv_cache),
            _ptr(new_idx), 0 if new_idx is None else new_idx.shape[1],
            _ptr(exclude_idx), 0 if exclude_idx is None else exclude_idx.shape[1],
            refresh_ratio, _ptr(hidden_out), _ptr(refresh_idx), C.byref(k), _ptr(workspace), workspace.numel(),
            _stream(stream)))
        return k.value

    def step_in_step_selection(self, hidden, kv_cache, new_idx, prev_idx, n_refresh, forced_refresh, hidden_out,
                               refresh_idx, active_idx, workspace, stream=None):
        self._check(self.lib.marche_step_in_step_selection(
            self.h, _ptr(hidden), _ptr(kv_cache), _ptr(new_idx), 0 if new_idx is None else new_idx.shape[1],
            _ptr(prev_idx), 0 if prev_idx is None else prev_idx.shape[1], n_refresh, _ptr(forced_refresh),
            _ptr(hidden_out), _ptr(refresh_idx), _ptr(active_idx), _ptr(workspace), workspace.numel(), _stream(stream)))

    def set_mar_weights(self, mar: Dict[str, torch.Tensor]):
        w = MarcheMarWeights()
        for name in MAR_FIELDS:
            t = mar[name]
            want = self.operand_dtype if name == "w_dec_embed" else torch.float32
            assert t.is_cuda and t.is_contiguous() and t.dtype == want, name
            setattr(w, name, t.data_ptr())
        self.mar_weights = dict(mar)          # keeps the device tensors alive
        self._check(self.lib.marche_set_mar_weights(self.h, C.byref(w)))

    def mar_step(self, full_decoder, tokens, known_idx, kv_cache, new_idx, prev_idx, n_refresh, forced_refresh, z_out,
                 refresh_idx, active_idx, workspace, stream=None):
        self._check(self.lib.marche_mar_step(
            self.h, 1 if full_decoder else 0, _ptr(tokens), _ptr(known_idx), known_idx.shape[1], _ptr(kv_cache),
            _ptr(new_idx), 0 if new_idx is None else new_idx.shape[1],
            _ptr(prev_idx), 0 if prev_idx is None else prev_idx.shape[1], n_refresh, _ptr(forced_refresh),
            _ptr(z_out), _ptr(refresh_idx), _ptr(active_idx), _ptr(workspace), workspace.numel(), _stream(stream)))

    def select_refresh(self, scores, new_idx, exclude_idx, k, refresh_idx, mask_scratch, stream=None):
        self._check(self.lib.marche_select_refresh(
            self.h, _ptr(scores), _ptr(new_idx), 0 if new_idx is None else new_idx.shape[1],
            _ptr(exclude_idx), 0 if exclude_idx is None else exclude_idx.shape[1], k, _ptr(refresh_idx),
            _ptr(mask_scratch), _stream(stream)))

    def select_refresh_policy(self, scores, new_idx, exclude_idx, k, policy, seed, refresh_idx, mask_scratch,
                              stream=None):
        """policy 0 = highest scores (the method), 1 = lowest scores, 2 = random (hash of seed, sample, token)."""
        self._check(self.lib.marche_select_refresh_policy(
            self.h, _ptr(scores), _ptr(new_idx), 0 if new_idx is None else new_idx.shape[1],
            _ptr(exclude_idx), 0 if exclude_idx is None else exclude_idx.shape[1], k, policy, seed, _ptr(refresh_idx),
            _ptr(mask_scratch), _stream(stream)))

    def select_refresh_static(self, scores, new_idx, exclude_idx, k, refresh_idx, stream=None):
        """select_refresh without a caller-supplied scratch buffer: the candidate mask lives in a
        fixed 256 KiB array inside the library (B*S must fit).  Nothing is allocated."""
        rc = self.lib.marche_select_refresh_static(
            self.h, _ptr(scores), _ptr(new_idx), 0 if new_idx is None else new_idx.shape[1],
            _ptr(exclude_idx), 0 if exclude_idx is None else exclude_idx.shape[1], k, _ptr(refresh_idx),
            _stream(stream))
        if rc == -3:
            raise MarcheError(rc, self.lib.marche_last_error(self.h).decode())
        self._check(rc)

    def get_scores(self, workspace, scores_out, stream=None):
        self._check(self.lib.marche_get_scores(self.h, _ptr(workspace), _ptr(scores_out), _stream(stream)))

    def set_score_layers(self, layers: Sequence[int]):
        arr = (C.c_int32 * max(len(layers), 1))(*layers)
        self._check(self.lib.marche_set_score_layers(self.h, arr, len(layers)))

    def get_layer_scores(self, workspace, layer: int, scores_out, stream=None):
        self._check(self.lib.marche_get_layer_scores(self.h, _ptr(workspace), layer, _ptr(scores_out), _stream(stream)))

    def build_active(self, new_idx, prev_idx, refresh_idx, n_refresh, active_idx, stream=None):
        self._check(self.lib.marche_build_active(
            self.h, _ptr(new_idx), 0 if new_idx is None else new_idx.shape[1],
            _ptr(prev_idx), 0 if prev_idx is None else prev_idx.shape[1],
            _ptr(refresh_idx) if n_refresh else None, n_refresh, _ptr(active_idx), _stream(stream)))

    def scatter_rows(self, rows, idx, dst, stream=None):
        self._check(self.lib.marche_scatter_rows(self.h, _ptr(rows), _ptr(idx), idx.shape[1], _ptr(dst),
                                                 _stream(stream)))

    def validate_indices(self, active_idx, new_idx, exclude_idx, stream=None):
        self._check(self.lib.marche_validate_indices(
            self.h, _ptr(active_idx), 0 if active_idx is None else active_idx.shape[1],
            _ptr(new_idx), 0 if new_idx is None else new_idx.shape[1],
            _ptr(exclude_idx), 0 if exclude_idx is None else exclude_idx.shape[1], _stream(stream)))

    def gather_layernorm(self, src, idx, n, gamma, beta, x_out, u_out, stream=None):
        self._check(self.lib.marche_gather_layernorm(self.h, _ptr(src), src.shape[1], _ptr(idx), n, _ptr(gamma),
                                                     _ptr(beta), _ptr(x_out), _ptr(u_out), _stream(stream)))

    def linear(self, a, w, bias, epilogue, out, M=None, lda=None, stream=None):
        N, K = w.shape
        M = a.shape[0] if M is None else M
        lda = a.stride(0) if lda is None else lda
        self._check(self.lib.marche_linear(self.h, a.data_ptr(), lda, M, _ptr(w), _ptr(bias), N, K, epilogue,
                                           _ptr(out), _stream(stream)))

    def scatter_kv(self, k, v, ld_kv, idx, n, cache_layer, stream=None):
        self._check(self.lib.marche_scatter_kv(self.h, k.data_ptr(), v.data_ptr(), ld_kv, _ptr(idx), n,
                                               _ptr(cache_layer), _stream(stream)))

    def attention(self, q, ld_q, n, cache_layer, is_new, score_partial, o, stream=None):
        self._check(self.lib.marche_attention(self.h, q.data_ptr(), ld_q, n, _ptr(cache_layer), _ptr(is_new),
                                              _ptr(score_partial), _ptr(o), _stream(stream)))

    def attention_two_segment(self, qkv, ld, n, active_idx, cache_layer, is_new, score_partial, o, stream=None):
        self._check(self.lib.marche_attention_two_segment(self.h, qkv.data_ptr(), ld, n, _ptr(active_idx),
                                                          _ptr(cache_layer), _ptr(is_new), _ptr(score_partial), _ptr(o),
                                                          _stream(stream)))

    def gather_rows(self, src, idx, rows_out, stream=None):
        self._check(self.lib.marche_gather_rows(self.h, _ptr(src), _ptr(idx), idx.shape[1], _ptr(rows_out),
                                                _stream(stream)))

    def staging_bytes(self, max_new: int) -> int:
        return self.lib.marche_staging_bytes(self.h, max_new)

    def step_host(self, full, hidden, kv_cache, h_prev_rows, h_prev_idx, h_new_idx, h_excl_idx, refresh_in,
                  n_refresh_in, refresh_ratio, hidden_out, refresh_out, h_out_rows, h_refresh_out, max_new, staging,
                  workspace, stream=None) -> int:
        """Host tensors (h_*) are CPU tensors, pinned for asynchronous copies; the rest are CUDA tensors."""
        def hp(t):
            return None if t is None else t.data_ptr()
        k = C.c_int(0)
        self._check(self.lib.marche_step_host(
            self.h, 1 if full else 0, _ptr(hidden), _ptr(kv_cache), hp(h_prev_rows), hp(h_prev_idx),
            0 if h_prev_idx is None else h_prev_idx.shape[1], hp(h_new_idx), 0 if h_new_idx is None else h_new_idx.shape[1],
            hp(h_excl_idx), 0 if h_excl_idx is None else h_excl_idx.shape[1], _ptr(refresh_in) if n_refresh_in else None,
            n_refresh_in, refresh_ratio, _ptr(hidden_out), _ptr(refresh_out), hp(h_out_rows), hp(h_refresh_out),
            C.byref(k), max_new, _ptr(staging), staging.numel(), _ptr(workspace), workspace.numel(), _stream(stream)))
        return k.value

    def launch_count(self) -> int:
        return int(self.lib.marche_launch_count(self.h))

    def profile_begin(self):
        self._check(self.lib.marche_profile_begin(self.h))

    def profile_end(self, stream=None):
        """-> {class name: (milliseconds, launches)} for the calls since profile_begin."""
        n = 11
        ms = (C.c_float * n)()
        cnt = (C.c_int * n)()
        self._check(self.lib.marche_profile_end(self.h, _stream(stream), ms, cnt))
        return {self.lib.marche_kernel_class_name(i).decode(): (float(ms[i]), int(cnt[i])) for i in range(n)}

    def get_tuning(self) -> Dict[str, int]:
        t = MarcheTuning()
        self._check(self.lib.marche_get_tuning(self.h, C.byref(t)))
        return {n: int(getattr(t, n)) for n, _ in MarcheTuning._fields_}

    def set_tuning(self, **fields):
        """Changes the named switches (see marche_tuning in the header); the others keep their values."""
        t = MarcheTuning()
        self._check(self.lib.marche_get_tuning(self.h, C.byref(t)))
        for n, v in fields.items():
            if n not in dict(MarcheTuning._fields_):
                raise KeyError(n)
            setattr(t, n, int(v))
        self._check(self.lib.marche_set_tuning(self.h, C.byref(t)))

    def check_status(self, stream=None):
        """Synchronises and raises MarcheError(ETIMEOUT) if a kernel gave up a bounded wait."""
        self._check(self.lib.marche_check_status(self.h, _stream(stream)))

    def debug_bounded_wait(self, limit_cycles: int, stream=None):
        self._check(self.lib.marche_debug_bounded_wait(self.h, limit_cycles, _stream(stream)))

    KERNEL_CLASSES = ("step_flags", "gather_layernorm", "gemm_qkv", "scatter_kv", "attention", "gemm_out_proj",
                      "gemm_fc1_gelu", "gemm_fc2", "scatter_rows", "topk", "other")

    def debug_skip_classes(self, names: Sequence[str] = ()):
        """Measurement hook: the named kernel classes are not launched until called again with ()."""
        mask = 0
        for n in names:
            mask |= 1 << self.KERNEL_CLASSES.index(n)
        self._check(self.lib.marche_debug_skip_classes(self.h, mask))

    def debug_repeat_classes(self, names: Sequence[str] = ()):
        """Measurement hook: every launch of the named kernel classes is issued twice until called again with ()."""
        mask = 0
        for n in names:
            mask |= 1 << self.KERNEL_CLASSES.index(n)
        self._check(self.lib.marche_debug_repeat_classes(self.h, mask))

    def device_status(self) -> int:
        return self.lib.marche_device_status(self.h)

    def clear_device_status(self):
        self.lib.marche_clear_device_status(self.h)
