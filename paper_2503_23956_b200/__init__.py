"""Thin ctypes binding of libaircache.so, the sm_100a CUDA library of the AirCache hot path.

Argument marshalling only: every function below forwards to the C entry point of the same name
(include/aircache.h) with raw device pointers taken from torch tensors.  All arithmetic of the
method runs in the CUDA kernels; there is no CPU or PyTorch fallback, and loading fails loudly
when the library has not been built (``python -m paper_2503_23956_b200.build``).
"""
from __future__ import annotations

import ctypes as C
import math
import os

import torch

from .build import LIB, build_library  # noqa: F401  (re-exported for the build entry)

OK = 0
ERR_INVALID_ARG = -1
ERR_UNSUPPORTED = -2
ERR_ALIGNMENT = -3
ERR_WORKSPACE_TOO_SMALL = -4
ERR_CAPACITY = -5
ERR_CUDA = -6
ERR_TIMEOUT = -7
ERR_STATIC_SCRATCH = -8
ERR_INCONSISTENT = -9


class AirCacheError(RuntimeError):
    def __init__(self, fn: str, code: int):
        self.code = code
        msg = lib().aircache_strerror(code).decode()
        extra = f" (cudaError {lib().aircache_last_cuda_error()})" if code == ERR_CUDA else ""
        super().__init__(f"{fn}: {msg}{extra} [{code}]")


class Shape(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "batch", "n_q_heads", "n_kv_heads", "head_dim", "n_visual",
                                           "n_text", "window", "slack")] + [("scale", C.c_float),
                                                                            ("per_kv_head", C.c_int32)]


class Full(C.Structure):
    _fields_ = [("k", C.c_void_p), ("v", C.c_void_p), ("stride_layer", C.c_int64), ("stride_batch", C.c_int64),
                ("stride_head", C.c_int64), ("stride_token", C.c_int64)]


class Ragged(C.Structure):
    _fields_ = [("k", C.c_void_p), ("v", C.c_void_p), ("offsets", C.c_void_p), ("lens", C.c_void_p),
                ("total_rows", C.c_int64), ("first_row", C.c_int64)]


_lib = None

_SIGNATURES = {
    "aircache_version": (C.c_int, []),
    "aircache_strerror": (C.c_char_p, [C.c_int]),
    "aircache_last_cuda_error": (C.c_int, []),
    "aircache_kept_per_sequence": (C.c_int64, [C.POINTER(Shape), C.c_double]),
    "aircache_total_rows": (C.c_int64, [C.POINTER(Shape), C.c_double]),
    "aircache_workspace_bytes": (C.c_int64, [C.POINTER(Shape)]),
    "aircache_score": (C.c_int, [C.POINTER(Shape), C.POINTER(Full), C.c_void_p, C.c_float, C.c_void_p, C.c_void_p,
                                 C.c_void_p, C.c_int64, C.c_void_p]),
    "aircache_score_layers": (C.c_int, [C.POINTER(Shape), C.POINTER(Full), C.c_void_p, C.c_float, C.c_int32, C.c_int32,
                                        C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p]),
    "aircache_budget": (C.c_int, [C.POINTER(Shape), C.c_void_p, C.c_double, C.c_int32, C.c_void_p, C.c_void_p,
                                  C.c_void_p, C.POINTER(Ragged), C.c_void_p, C.c_int64, C.c_void_p]),
    "aircache_compact": (C.c_int, [C.POINTER(Shape), C.POINTER(Full), C.c_void_p, C.c_void_p, C.c_double,
                                   C.POINTER(Ragged), C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p]),
    "aircache_decode_attn": (C.c_int, [C.POINTER(Shape), C.POINTER(Ragged), C.c_void_p, C.c_void_p, C.c_void_p,
                                       C.c_int64, C.c_void_p]),
    "aircache_decode_step": (C.c_int, [C.POINTER(Shape), C.POINTER(Ragged), C.c_void_p, C.c_void_p, C.c_void_p,
                                       C.c_int32, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p]),
    "aircache_decode_attn_static": (C.c_int, [C.POINTER(Shape), C.POINTER(Ragged), C.c_void_p, C.c_void_p,
                                              C.c_void_p]),
    "aircache_append": (C.c_int, [C.POINTER(Shape), C.POINTER(Ragged), C.c_void_p, C.c_void_p, C.c_int32,
                                  C.c_void_p]),
    "aircache_reset_status": (C.c_int, [C.c_void_p, C.c_int64, C.c_void_p]),
    "aircache_check_status": (C.c_int, [C.c_void_p, C.c_int64, C.c_void_p]),
    "aircache_selftest_wait_timeout": (C.c_int, [C.c_void_p, C.c_int64, C.c_void_p]),
    "aircache_host_range_is_mapped": (C.c_int, [C.c_void_p, C.c_int64]),
    "aircache_pipeline_host": (C.c_int, [C.POINTER(Shape), C.POINTER(Full), C.c_int64, C.c_void_p, C.c_void_p,
                                         C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_float,
                                         C.c_double, C.c_int32, C.c_void_p, C.c_void_p, C.POINTER(Ragged),
                                         C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p]),
}


def lib() -> C.CDLL:
    """The loaded library.  Raises when libaircache.so has not been built: there is no fallback."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB):
            raise RuntimeError(f"{LIB} is missing: build it with `python -m paper_2503_23956_b200.build` "
                               "(the AirCache path has no CPU or PyTorch fallback)")
        handle = C.CDLL(LIB)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype = res
            fn.argtypes = args
        _lib = handle
    return _lib


def exported_symbols() -> list[str]:
    return list(_SIGNATURES)


# ------------------------------------------------------------------------------------------------
# marshalling helpers
# ------------------------------------------------------------------------------------------------
def _ptr(t) -> int | None:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream) -> int | None:
    if stream is None:
        stream = torch.cuda.current_stream()
    if isinstance(stream, int):
        return stream or None
    return stream.cuda_stream or None


def _check(fn: str, rc: int) -> None:
    if rc != OK:
        raise AirCacheError(fn, rc)


def shape(n_layers, batch, n_q_heads, n_kv_heads, head_dim, n_visual, n_text, window, slack=0, scale=None,
          per_kv_head=0) -> Shape:
    if scale is None:
        scale = 1.0 / math.sqrt(head_dim)   # rounded to fp32 by ctypes
    return Shape(n_layers, batch, n_q_heads, n_kv_heads, head_dim, n_visual, n_text, window, slack, scale,
                 int(per_kv_head))


def full_view(k: torch.Tensor, v: torch.Tensor) -> Full:
    """View of two bf16 tensors whose logical dims are [L, B, Hkv, N, d] (any strides, d contiguous)."""
    assert k.dtype == torch.bfloat16 and v.dtype == torch.bfloat16 and k.dim() == 5
    assert k.shape == v.shape and k.stride() == v.stride() and k.stride(4) == 1
    sl, sb, sh, st, _ = k.stride()
    return Full(k.data_ptr(), v.data_ptr(), sl, sb, sh, st)


def ragged_view(k, v, offsets, lens, total_rows: int, first_row: int = 0) -> Ragged:
    """`offsets` / `lens` may be tensors or raw addresses (a stretch of shared arrays, see aircache_ragged_t)."""
    return Ragged(_ptr(k), _ptr(v), _ptr(offsets), _ptr(lens), total_rows, first_row)


# ------------------------------------------------------------------------------------------------
# the C ABI, same names
# ------------------------------------------------------------------------------------------------
def aircache_version() -> int:
    return lib().aircache_version()


def aircache_strerror(code: int) -> str:
    return lib().aircache_strerror(code).decode()


def aircache_kept_per_sequence(sh: Shape, ratio: float) -> int:
    return int(lib().aircache_kept_per_sequence(C.byref(sh), ratio))


def aircache_total_rows(sh: Shape, ratio: float) -> int:
    return int(lib().aircache_total_rows(C.byref(sh), ratio))


def aircache_workspace_bytes(sh: Shape) -> int:
    return int(lib().aircache_workspace_bytes(C.byref(sh)))


def aircache_score(sh, full, q_window, alpha, scores, elite_mask, workspace, stream=None, check=True) -> int:
    rc = lib().aircache_score(C.byref(sh), C.byref(full), _ptr(q_window), alpha, _ptr(scores), _ptr(elite_mask),
                              _ptr(workspace), _nbytes(workspace), _stream(stream))
    if check:
        _check("aircache_score", rc)
    return rc


def aircache_score_layers(sh, full, q_window, alpha, layer_begin, layer_count, scores, elite_mask, workspace,
                          stream=None, check=True) -> int:
    rc = lib().aircache_score_layers(C.byref(sh), C.byref(full), _ptr(q_window), alpha, layer_begin, layer_count,
                                     _ptr(scores), _ptr(elite_mask), _ptr(workspace), _nbytes(workspace),
                                     _stream(stream))
    if check:
        _check("aircache_score_layers", rc)
    return rc


def aircache_budget(sh, scores, ratio, mode, budgets, strength, skewness, layout, workspace, stream=None,
                    check=True) -> int:
    rc = lib().aircache_budget(C.byref(sh), _ptr(scores), ratio, mode, _ptr(budgets), _ptr(strength),
                               _ptr(skewness), C.byref(layout), _ptr(workspace), _nbytes(workspace), _stream(stream))
    if check:
        _check("aircache_budget", rc)
    return rc


def aircache_compact(sh, full, scores, budgets, ratio, out, kept_idx, workspace, stream=None, check=True) -> int:
    rc = lib().aircache_compact(C.byref(sh), C.byref(full), _ptr(scores), _ptr(budgets), ratio, C.byref(out),
                                _ptr(kept_idx), _ptr(workspace), _nbytes(workspace), _stream(stream))
    if check:
        _check("aircache_compact", rc)
    return rc


def aircache_decode_attn(sh, cache, q, out, workspace, stream=None, check=True) -> int:
    rc = lib().aircache_decode_attn(C.byref(sh), C.byref(cache), _ptr(q), _ptr(out), _ptr(workspace),
                                    _nbytes(workspace), _stream(stream))
    if check:
        _check("aircache_decode_attn", rc)
    return rc


def aircache_decode_step(sh, cache, q, k_new, v_new, appended, out, workspace, stream=None, check=True) -> int:
    rc = lib().aircache_decode_step(C.byref(sh), C.byref(cache), _ptr(q), _ptr(k_new), _ptr(v_new), appended,
                                    _ptr(out), _ptr(workspace), _nbytes(workspace), _stream(stream))
    if check:
        _check("aircache_decode_step", rc)
    return rc


def aircache_decode_attn_static(sh, cache, q, out, stream=None, check=True) -> int:
    """aircache_decode_attn without a workspace: scratch comes from an array built into the library."""
    rc = lib().aircache_decode_attn_static(C.byref(sh), C.byref(cache), _ptr(q), _ptr(out), _stream(stream))
    if check:
        _check("aircache_decode_attn_static", rc)
    return rc


def aircache_append(sh, cache, k_new, v_new, appended, stream=None, check=True) -> int:
    rc = lib().aircache_append(C.byref(sh), C.byref(cache), _ptr(k_new), _ptr(v_new), appended, _stream(stream))
    if check:
        _check("aircache_append", rc)
    return rc


def aircache_reset_status(workspace, stream=None, check=True) -> int:
    rc = lib().aircache_reset_status(_ptr(workspace), _nbytes(workspace), _stream(stream))
    if check:
        _check("aircache_reset_status", rc)
    return rc


def aircache_check_status(workspace, stream=None, check=True) -> int:
    rc = lib().aircache_check_status(_ptr(workspace), _nbytes(workspace), _stream(stream))
    if check:
        _check("aircache_check_status", rc)
    return rc


def aircache_selftest_wait_timeout(workspace, stream=None, check=True) -> int:
    rc = lib().aircache_selftest_wait_timeout(_ptr(workspace), _nbytes(workspace), _stream(stream))
    if check:
        _check("aircache_selftest_wait_timeout", rc)
    return rc


def aircache_host_range_is_mapped(host_tensor) -> bool:
    """True if kernels can read the tensor's host memory in place (page-locked and mapped)."""
    return bool(lib().aircache_host_range_is_mapped(_ptr(host_tensor), _nbytes(host_tensor)))


def aircache_pipeline_host(sh, h_full, full_elems, d_full_k, d_full_v, h_q_window, d_q_window, h_q_steps, d_q_steps,
                           n_steps, alpha, ratio, mode, d_scores, d_budgets, d_cache, d_out, h_out, h_budgets,
                           workspace, stream=None, check=True) -> int:
    rc = lib().aircache_pipeline_host(C.byref(sh), C.byref(h_full), full_elems, _ptr(d_full_k), _ptr(d_full_v),
                                      _ptr(h_q_window), _ptr(d_q_window), _ptr(h_q_steps), _ptr(d_q_steps), n_steps,
                                      alpha, ratio, mode, _ptr(d_scores), _ptr(d_budgets), C.byref(d_cache),
                                      _ptr(d_out), _ptr(h_out), _ptr(h_budgets), _ptr(workspace),
                                      _nbytes(workspace), _stream(stream))
    if check:
        _check("aircache_pipeline_host", rc)
    return rc


def _nbytes(t) -> int:
    if t is None or isinstance(t, int):
        return 0
    return t.numel() * t.element_size()
