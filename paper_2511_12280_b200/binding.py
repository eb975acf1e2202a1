"""ctypes binding of libd3tom.so: the same names as the C ABI (include/d3tom.h),
argument marshalling only.  Every step of the path runs in the CUDA kernels of
the library; there is no Python or CPU fallback, and a missing library or a
non-zero status raises.

Tensors are torch CUDA tensors used purely as device memory; work is enqueued on
torch's current stream unless a stream is given.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libd3tom.so")

BF16, FP32 = 0, 1
AGG_SUM, AGG_MEAN = 0, 1
OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = -1, -2, -3, -4, -5


class Limits(C.Structure):
    _fields_ = [("max_total_tokens", C.c_int), ("max_batch", C.c_int), ("heads", C.c_int), ("head_dim", C.c_int),
                ("max_deciders", C.c_int), ("max_visual_per_request", C.c_int)]


class D3tomError(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__("%s failed: %s (%d)" % (what, status_string(status), status))
        self.status = status


_lib = None
_P, _I, _F = C.c_void_p, C.c_int, C.c_float

_SIGNATURES = {
    "d3tom_create": (_I, [C.POINTER(_P), _I, C.POINTER(Limits)]),
    "d3tom_destroy": (_I, [_P]),
    "d3tom_status_string": (C.c_char_p, [_I]),
    "d3tom_last_cuda_error": (_I, [_P]),
    "d3tom_device_status": (_I, [_P, C.POINTER(_I)]),
    "d3tom_reset_device_status": (_I, [_P]),
    "d3tom_selftest_wait_timeout": (_I, [_P, C.c_int64, _P]),
    "d3tom_workspace_bytes": (C.c_int64, [_P]),
    "d3tom_set_reference_kernels": (_I, [_P, _I]),
    "d3tom_set_launch_overlap": (_I, [_I]),
    "d3tom_set_pair_tiles": (_I, [_I]),
    "d3tom_set_single_tile_attention": (_I, [_I]),
    "d3tom_keep_count": (_I, [_I, C.c_double]),
    "d3tom_schedule_alpha": (_I, [_I, _I, C.c_double, C.c_double, _I, C.POINTER(C.c_double)]),
    "d3tom_attn_importance": (_I, [_P, _I, _P, _P, _P, _P, _P, _P, _P, _I, _I, _I, _I, _I, _F, _P, _P, _P, _P]),
    "d3tom_attn_importance_static": (_I, [_I, _I, _I, _P, _P, _P, _P, _P, _P, _P, _I, _I, _I, _I, _I, _F, _P, _P, _P, _P,
                                          _P]),
    "d3tom_select": (_I, [_P, _P, _P, _P, _P, _I, _I, _P, _P, _P]),
    "d3tom_merge": (_I, [_P, _I, _I, _P, _P, _P, _P, _P, _P, _I, _I, _I, _I, _I, _I, _P, _P, _P, _P, _P, _P, _P]),
    "d3tom_merge_kv": (_I, [_P, _I, _I, _P, _P, _P, _P, _P, _P, _P, _I, _I, _I, _I, _I, _I, _P, _P, _P, _P, _P, _P, _P, _P]),
    "d3tom_attn_varlen": (_I, [_P, _I, _P, _P, _P, _P, _I, _I, _I, _F, _P, _P]),
    "d3tom_proj_qkv": (_I, [_P, _I, _P, _P, _I, _I, _P, _P, _P, _P]),
    "d3tom_linear": (_I, [_P, _I, _P, _P, _P, _I, _I, _I, _P, _P]),
    "d3tom_ffn": (_I, [_P, _I, _P, _P, _P, _P, _I, _I, _I, _P, _P, _P]),
}


def load():
    """Load the shared library (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libd3tom.so is missing: build it with `python -m paper_2511_12280_b200.build`")
        lib = C.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


def exported_symbols():
    return sorted(_SIGNATURES)


def status_string(status: int) -> str:
    return load().d3tom_status_string(status).decode()


def _check(status: int, what: str):
    if status != OK:
        raise D3tomError(status, what)


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device, contiguous tensors only"
    return C.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float32:
        return FP32
    raise TypeError("storage type must be bf16 or fp32")


# ------------------------------------------------------------------ host helpers
def d3tom_keep_count(n_visual: int, keep_ratio: float) -> int:
    return load().d3tom_keep_count(int(n_visual), float(keep_ratio))


def d3tom_set_launch_overlap(on: bool):
    """Profiling aid: with on = False kernels start only after their predecessor has finished (separable per-kernel
    device times); the default lets a kernel's blocks become resident while its predecessor drains."""
    _check(load().d3tom_set_launch_overlap(int(on)), "d3tom_set_launch_overlap")


def d3tom_set_pair_tiles(width: int):
    """Tile shape of the dense layers: -1 chosen per shape (default), 0 single-CTA tiles only, 256 forces
    256 x 256 tiles computed by CTA pairs wherever the layer's width allows."""
    _check(load().d3tom_set_pair_tiles(int(width)), "d3tom_set_pair_tiles")


def d3tom_set_single_tile_attention(mode: int):
    """Attention kernel choice: -1 per launch (default), 0 two query tiles per CTA, 1 one query tile per CTA with three
    score buffers wherever supported (bf16, head_dim 128, no importance)."""
    _check(load().d3tom_set_single_tile_attention(int(mode)), "d3tom_set_single_tile_attention")


def d3tom_schedule_alpha(step: int, T: int, a_min: float, a_max: float, reversed_: bool = False) -> float:
    out = C.c_double()
    _check(load().d3tom_schedule_alpha(step, T, a_min, a_max, int(reversed_), C.byref(out)), "d3tom_schedule_alpha")
    return out.value


def d3tom_attn_importance_static(heads, head_dim, q, k, v, cu_seqlens, n_visual, decider_pos, cu_deciders, B,
                                 total_tokens, max_seqlen, max_visual, n_deciders_total, softmax_scale, attn_out,
                                 importance, cu_vis, device_status_out=None, stream=None):
    """d3tom_attn_importance for callers that may not allocate device memory: no context, the
    scratch is a fixed array inside the library (see include/d3tom.h for its size limits).
    Runs on the current device; calls on one device must not overlap."""
    _check(load().d3tom_attn_importance_static(_dt(q), heads, head_dim, _ptr(q), _ptr(k), _ptr(v), _ptr(cu_seqlens),
                                               _ptr(n_visual), _ptr(decider_pos), _ptr(cu_deciders), B, total_tokens,
                                               max_seqlen, max_visual, n_deciders_total, softmax_scale,
                                               _ptr(attn_out), _ptr(importance), _ptr(cu_vis),
                                               _ptr(device_status_out), _stream(stream)),
           "d3tom_attn_importance_static")


class Context:
    """Owns a d3tom_ctx (scratch sized from the limits)."""

    def __init__(self, max_total_tokens, max_batch, heads, head_dim, max_deciders, max_visual_per_request, device=0):
        self._h = C.c_void_p()
        self.limits = Limits(max_total_tokens, max_batch, heads, head_dim, max_deciders, max_visual_per_request)
        self.device = device
        _check(load().d3tom_create(C.byref(self._h), device, C.byref(self.limits)), "d3tom_create")

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            load().d3tom_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def workspace_bytes(self) -> int:
        return load().d3tom_workspace_bytes(self._h)

    def set_reference_kernels(self, on: bool):
        _check(load().d3tom_set_reference_kernels(self._h, int(on)), "d3tom_set_reference_kernels")

    def device_status(self) -> int:
        out = C.c_int()
        _check(load().d3tom_device_status(self._h, C.byref(out)), "d3tom_device_status")
        return out.value

    def reset_device_status(self):
        _check(load().d3tom_reset_device_status(self._h), "d3tom_reset_device_status")

    def selftest_wait_timeout(self, limit_ns: int, stream=None):
        """Enqueues the one-block kernel whose wait cannot end; afterwards device_status() is ERR_TIMEOUT."""
        _check(load().d3tom_selftest_wait_timeout(self._h, int(limit_ns), _stream(stream)), "d3tom_selftest_wait_timeout")

    # -------------------------------------------------------------- the four calls (+ projection)
    def d3tom_attn_importance(self, q, k, v, cu_seqlens, n_visual, decider_pos, cu_deciders, B, total_tokens,
                              max_seqlen, max_visual, n_deciders_total, softmax_scale, attn_out, importance, cu_vis,
                              stream=None):
        _check(load().d3tom_attn_importance(self._h, _dt(q), _ptr(q), _ptr(k), _ptr(v), _ptr(cu_seqlens),
                                            _ptr(n_visual), _ptr(decider_pos), _ptr(cu_deciders), B, total_tokens,
                                            max_seqlen, max_visual, n_deciders_total, softmax_scale, _ptr(attn_out),
                                            _ptr(importance), _ptr(cu_vis), _stream(stream)), "d3tom_attn_importance")

    def d3tom_select(self, importance, cu_vis, keep_count, cu_kept, B, max_visual, kept_idx, keep_mask, stream=None):
        _check(load().d3tom_select(self._h, _ptr(importance), _ptr(cu_vis), _ptr(keep_count), _ptr(cu_kept), B,
                                   max_visual, _ptr(kept_idx), _ptr(keep_mask), _stream(stream)), "d3tom_select")

    def d3tom_merge(self, mode, hidden, cu_seqlens, n_visual, cu_vis, kept_idx, cu_kept, B, D, total_tokens,
                    total_out, max_visual, max_kept, hidden_out, cu_seqlens_out, assign, member_count, src_of_dst,
                    sim_debug=None, stream=None):
        _check(load().d3tom_merge(self._h, _dt(hidden), mode, _ptr(hidden), _ptr(cu_seqlens), _ptr(n_visual),
                                  _ptr(cu_vis), _ptr(kept_idx), _ptr(cu_kept), B, D, total_tokens, total_out,
                                  max_visual, max_kept, _ptr(hidden_out), _ptr(cu_seqlens_out), _ptr(assign),
                                  _ptr(member_count), _ptr(src_of_dst), _ptr(sim_debug), _stream(stream)),
               "d3tom_merge")

    def d3tom_merge_kv(self, mode, k_cache, v_cache, cu_seqlens, n_visual, cu_vis, kept_idx, cu_kept, B, D, total_tokens,
                       total_out, max_visual, max_kept, k_out, v_out, cu_seqlens_out, assign, member_count, src_of_dst,
                       sim_debug=None, stream=None):
        _check(load().d3tom_merge_kv(self._h, _dt(k_cache), mode, _ptr(k_cache), _ptr(v_cache), _ptr(cu_seqlens),
                                     _ptr(n_visual), _ptr(cu_vis), _ptr(kept_idx), _ptr(cu_kept), B, D, total_tokens,
                                     total_out, max_visual, max_kept, _ptr(k_out), _ptr(v_out), _ptr(cu_seqlens_out),
                                     _ptr(assign), _ptr(member_count), _ptr(src_of_dst), _ptr(sim_debug),
                                     _stream(stream)), "d3tom_merge_kv")

    def d3tom_attn_varlen(self, q, k, v, cu_seqlens, B, total_tokens, max_seqlen, softmax_scale, out, stream=None):
        _check(load().d3tom_attn_varlen(self._h, _dt(q), _ptr(q), _ptr(k), _ptr(v), _ptr(cu_seqlens), B,
                                        total_tokens, max_seqlen, softmax_scale, _ptr(out), _stream(stream)),
               "d3tom_attn_varlen")

    def d3tom_proj_qkv(self, x, w_qkv, total, D, q, k, v, stream=None):
        _check(load().d3tom_proj_qkv(self._h, _dt(x), _ptr(x), _ptr(w_qkv), total, D, _ptr(q), _ptr(k), _ptr(v),
                                     _stream(stream)), "d3tom_proj_qkv")

    def d3tom_linear(self, x, w, residual, rows, K, N, out, stream=None):
        _check(load().d3tom_linear(self._h, _dt(x), _ptr(x), _ptr(w), _ptr(residual) if residual is not None else None,
                                   rows, K, N, _ptr(out), _stream(stream)), "d3tom_linear")

    def d3tom_ffn(self, x, w_gate_up, w_down, residual, rows, D, m, act, out, stream=None):
        _check(load().d3tom_ffn(self._h, _dt(x), _ptr(x), _ptr(w_gate_up), _ptr(w_down),
                                _ptr(residual) if residual is not None else None, rows, D, m, _ptr(act), _ptr(out),
                                _stream(stream)), "d3tom_ffn")
