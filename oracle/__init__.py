"""ctypes front-end of the AirCache CPU oracle (oracle/aircache_oracle.c).

TEST INFRASTRUCTURE, NOT THE PRODUCT: only the tests, the smoke check and the
benchmark's CPU-baseline leg may import this package.  It shares nothing with the
CUDA library; it never imports the product package and is never imported by it.

Every wrapper takes and returns numpy arrays; bf16 tensors travel as uint16 bit
patterns (``tensor.view(torch.int16).numpy().view(np.uint16)`` on the torch side).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "aircache_oracle.c")
_LIB = os.path.join(_HERE, "libaircache_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C, fp contraction off, OpenMP over work items)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Dims(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "batch", "n_q_heads", "n_kv_heads", "head_dim",
                                           "n_visual", "n_text", "window")]


@dataclass(frozen=True)
class Dims:
    n_layers: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    n_visual: int
    n_text: int
    window: int

    def c(self) -> _Dims:
        return _Dims(self.n_layers, self.batch, self.n_q_heads, self.n_kv_heads, self.head_dim,
                     self.n_visual, self.n_text, self.window)


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_total_kept.restype = C.c_int64
        _lib.oracle_total_kept.argtypes = [C.c_int32, C.c_int32, C.c_double]
    return _lib


def _p(a: np.ndarray | None):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _u16(a) -> np.ndarray:
    a = np.asarray(a)
    assert a.dtype == np.uint16, a.dtype
    return a


def _strides_elems(a: np.ndarray) -> tuple[int, ...]:
    return tuple(s // a.itemsize for s in a.strides)


def full_cache_strides(k: np.ndarray) -> tuple[int, int, int, int]:
    """Element strides (layer, batch, head, token) of a logical [L, B, Hkv, N, d] uint16 view."""
    assert k.ndim == 5 and k.strides[-1] == k.itemsize
    s = _strides_elems(k)
    return s[0], s[1], s[2], s[3]


def _mask_shape(dims: Dims):
    """Elite masks: one 64-bit word per query head, two when the window has more than 64 candidates."""
    words = (dims.window + 63) // 64
    return (dims.n_layers, dims.batch, dims.n_q_heads) + ((words,) if words > 1 else ())


def score(dims: Dims, k: np.ndarray, q_window: np.ndarray, scale: float, alpha: float,
          want_logits: bool = False):
    """Eq. 4-8.  k: uint16 logical [L,B,Hkv,N,d] (any strides, d contiguous); q_window: uint16 [L,B,W,Hq,d].

    Returns dict(scores f32 [L,B,Nv], elite_mask u64 [L,B,Hq], text_mass f64 [L,B,Hq][, elite_logits])."""
    k = _u16(k)
    q_window = np.ascontiguousarray(_u16(q_window))
    L, B, Hq, W = dims.n_layers, dims.batch, dims.n_q_heads, dims.window
    assert k.shape == (L, B, dims.n_kv_heads, dims.n_visual + dims.n_text, dims.head_dim), k.shape
    assert q_window.shape == (L, B, W, Hq, dims.head_dim), q_window.shape
    sl, sb, sh, st = full_cache_strides(k)
    scores = np.empty((L, B, dims.n_visual), np.float32)
    mask = np.empty(_mask_shape(dims), np.uint64)
    tmass = np.empty((L, B, Hq), np.float64)
    logits = np.empty((L, B, Hq, W), np.float32) if want_logits else None
    d = dims.c()
    rc = lib().oracle_score(C.byref(d), _p(k), C.c_int64(sl), C.c_int64(sb), C.c_int64(sh), C.c_int64(st),
                            _p(q_window), C.c_float(scale), C.c_float(alpha), _p(scores), _p(mask), _p(tmass),
                            _p(logits))
    if rc:
        raise ValueError(f"oracle_score: {rc}")
    out = dict(scores=scores, elite_mask=mask, text_mass=tmass)
    if want_logits:
        out["elite_logits"] = logits
    return out


def score_groups(dims: Dims, k: np.ndarray, q_window: np.ndarray, scale: float, alpha: float):
    """Eq. 4-8 with the importance kept apart per KV group -> dict(scores f32 [L,B,Hkv,Nv], elite_mask u64 [L,B,Hq])."""
    k = _u16(k)
    q_window = np.ascontiguousarray(_u16(q_window))
    L, B, Hq, W = dims.n_layers, dims.batch, dims.n_q_heads, dims.window
    assert k.shape == (L, B, dims.n_kv_heads, dims.n_visual + dims.n_text, dims.head_dim), k.shape
    assert q_window.shape == (L, B, W, Hq, dims.head_dim), q_window.shape
    sl, sb, sh, st = full_cache_strides(k)
    scores = np.empty((L, B, dims.n_kv_heads, dims.n_visual), np.float32)
    mask = np.empty(_mask_shape(dims), np.uint64)
    d = dims.c()
    rc = lib().oracle_score_groups(C.byref(d), _p(k), C.c_int64(sl), C.c_int64(sb), C.c_int64(sh), C.c_int64(st),
                                   _p(q_window), C.c_float(scale), C.c_float(alpha), _p(scores), _p(mask))
    if rc:
        raise ValueError(f"oracle_score_groups: {rc}")
    return dict(scores=scores, elite_mask=mask)


def allocate_groups(strength: np.ndarray, skewness: np.ndarray, n_visual: int, ratio: float, mode: int = 0):
    """Eq. 11 over the (layer, KV head) cells of each sequence.  strength/skewness f64 [L,B,Hkv] -> budgets i32."""
    strength = np.ascontiguousarray(strength, np.float64)
    skewness = np.ascontiguousarray(skewness, np.float64)
    L, B, Hkv = strength.shape
    budgets = np.zeros((L, B, Hkv), np.int32)
    rc = lib().oracle_allocate_groups(_p(strength), _p(skewness), C.c_int32(L), C.c_int32(B), C.c_int32(Hkv),
                                      C.c_int32(n_visual), C.c_double(ratio), C.c_int32(mode), _p(budgets))
    if rc:
        raise ValueError(f"oracle_allocate_groups: {rc}")
    return budgets


def compact_groups(dims: Dims, slack: int, k: np.ndarray, v: np.ndarray, scores: np.ndarray, budgets: np.ndarray):
    """Per-KV-group select + gather -> dict(k, v uint16 [rows,1,d], offsets i64 [cells+1], lens i32 [cells], kept_idx)."""
    k, v = _u16(k), _u16(v)
    assert k.shape == v.shape and k.strides == v.strides
    L, B, Hkv = dims.n_layers, dims.batch, dims.n_kv_heads
    cells = L * B * Hkv
    scores = np.ascontiguousarray(scores, np.float32).reshape(cells, dims.n_visual)
    budgets = np.ascontiguousarray(budgets, np.int32).reshape(cells)
    rows = int(budgets.sum()) + cells * (dims.n_text + slack)
    k_out = np.zeros((rows, 1, dims.head_dim), np.uint16)
    v_out = np.zeros_like(k_out)
    offsets = np.empty(cells + 1, np.int64)
    lens = np.empty(cells, np.int32)
    kept = np.empty(max(int(budgets.sum()), 1), np.int32)
    sl, sb, sh, st = full_cache_strides(k)
    d = dims.c()
    rc = lib().oracle_compact_groups(C.byref(d), C.c_int32(slack), _p(k), _p(v), C.c_int64(sl), C.c_int64(sb),
                                     C.c_int64(sh), C.c_int64(st), _p(scores), _p(budgets), _p(k_out), _p(v_out),
                                     _p(offsets), _p(lens), _p(kept))
    if rc:
        raise ValueError(f"oracle_compact_groups: {rc}")
    return dict(k=k_out, v=v_out, offsets=offsets, lens=lens, kept_idx=kept[:int(budgets.sum())])


def group_decode_dims(dims: Dims) -> Dims:
    """The per-KV-group cache seen by decode(): every cell is a region with one KV head and G query heads."""
    return Dims(dims.n_layers * dims.batch * dims.n_kv_heads, 1, dims.n_q_heads // dims.n_kv_heads, 1,
                dims.head_dim, dims.n_visual, dims.n_text, dims.window)


def moments(scores: np.ndarray):
    """Eq. 9-10 on fp32 scores [..., Nv] -> (strength f64 [...], skewness f64 [...])."""
    scores = np.ascontiguousarray(scores, np.float32)
    nv = scores.shape[-1]
    lead = scores.shape[:-1]
    n = int(np.prod(lead)) if lead else 1
    st = np.empty(n, np.float64)
    sk = np.empty(n, np.float64)
    rc = lib().oracle_moments(_p(scores), C.c_int64(n), C.c_int32(nv), _p(st), _p(sk))
    if rc:
        raise ValueError(f"oracle_moments: {rc}")
    return st.reshape(lead), sk.reshape(lead)


def total_kept(n_visual: int, n_layers: int, ratio: float) -> int:
    return int(lib().oracle_total_kept(n_visual, n_layers, C.c_double(ratio)))


def allocate(strength: np.ndarray, skewness: np.ndarray, n_visual: int, ratio: float, mode: int = 0):
    """Eq. 11 + integer budgets.  strength/skewness f64 [L,B] -> budgets i32 [L,B]."""
    strength = np.ascontiguousarray(strength, np.float64)
    skewness = np.ascontiguousarray(skewness, np.float64)
    L, B = strength.shape
    budgets = np.zeros((L, B), np.int32)
    rc = lib().oracle_allocate(_p(strength), _p(skewness), C.c_int32(L), C.c_int32(B), C.c_int32(n_visual),
                               C.c_double(ratio), C.c_int32(mode), _p(budgets))
    if rc:
        raise ValueError(f"oracle_allocate: {rc}")
    return budgets


def select(scores: np.ndarray, n_keep: int) -> np.ndarray:
    """Top-n_keep of one fp32 score vector, ties -> lower index, ascending indices."""
    scores = np.ascontiguousarray(scores, np.float32)
    kept = np.empty(max(n_keep, 1), np.int32)
    rc = lib().oracle_select(_p(scores), C.c_int32(scores.shape[0]), C.c_int32(n_keep), _p(kept))
    if rc:
        raise ValueError(f"oracle_select: {rc}")
    return kept[:n_keep]


def compact(dims: Dims, slack: int, k: np.ndarray, v: np.ndarray, scores: np.ndarray, budgets: np.ndarray):
    """Select + gather.  Returns dict(k, v uint16 [rows,Hkv,d], offsets i64 [L*B+1], lens i32 [L*B], kept_idx i32)."""
    k, v = _u16(k), _u16(v)
    assert k.shape == v.shape and k.strides == v.strides
    L, B = dims.n_layers, dims.batch
    scores = np.ascontiguousarray(scores, np.float32).reshape(L, B, dims.n_visual)
    budgets = np.ascontiguousarray(budgets, np.int32).reshape(L, B)
    rows = int(budgets.sum()) + L * B * (dims.n_text + slack)
    k_out = np.zeros((rows, dims.n_kv_heads, dims.head_dim), np.uint16)
    v_out = np.zeros_like(k_out)
    offsets = np.empty(L * B + 1, np.int64)
    lens = np.empty(L * B, np.int32)
    kept = np.empty(max(int(budgets.sum()), 1), np.int32)
    sl, sb, sh, st = full_cache_strides(k)
    d = dims.c()
    rc = lib().oracle_compact(C.byref(d), C.c_int32(slack), _p(k), _p(v), C.c_int64(sl), C.c_int64(sb),
                              C.c_int64(sh), C.c_int64(st), _p(scores), _p(budgets), _p(k_out), _p(v_out),
                              _p(offsets), _p(lens), _p(kept))
    if rc:
        raise ValueError(f"oracle_compact: {rc}")
    return dict(k=k_out, v=v_out, offsets=offsets, lens=lens, kept_idx=kept[:int(budgets.sum())])


def decode(dims: Dims, k_c: np.ndarray, v_c: np.ndarray, offsets: np.ndarray, lens: np.ndarray,
           q: np.ndarray, scale: float) -> np.ndarray:
    """Single-token attention over the ragged cache.  q uint16 [L,B,Hq,d] -> out f32 [L,B,Hq,d]."""
    k_c, v_c = np.ascontiguousarray(_u16(k_c)), np.ascontiguousarray(_u16(v_c))
    q = np.ascontiguousarray(_u16(q))
    offsets = np.ascontiguousarray(offsets, np.int64)
    lens = np.ascontiguousarray(lens, np.int32)
    out = np.empty(q.shape, np.float32)
    d = dims.c()
    rc = lib().oracle_decode(C.byref(d), _p(k_c), _p(v_c), _p(offsets), _p(lens), _p(q), C.c_float(scale),
                             _p(out))
    if rc:
        raise ValueError(f"oracle_decode: {rc}")
    return out


def num_threads() -> int:
    return int(lib().oracle_num_threads())
