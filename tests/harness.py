"""Shared plumbing of the GPU parity tests: runs the CUDA path through the binding and the CPU oracle
on the same seeded inputs.  The two sides share only the input generators of `workloads`."""
from __future__ import annotations

import numpy as np
import torch

import paper_2503_23956_b200 as ac
from paper_2503_23956_b200.session import Session
from workloads import full_cache, window_queries
from workloads.synth import to_u16


def shape_of(wl, **kw):
    d = dict(n_layers=wl.n_layers, batch=wl.batch, n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads,
             head_dim=wl.head_dim, n_visual=wl.n_visual, n_text=wl.n_text, window=wl.window, slack=wl.slack,
             scale=wl.scale)
    d.update(kw)
    return ac.shape(**d)


def oracle_dims(oracle, wl, **kw):
    d = dict(n_layers=wl.n_layers, batch=wl.batch, n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads,
             head_dim=wl.head_dim, n_visual=wl.n_visual, n_text=wl.n_text, window=wl.window)
    d.update(kw)
    return oracle.Dims(**d)


def logical(t: torch.Tensor) -> torch.Tensor:
    """Token-major [L,B,N,Hkv,d] storage -> logical [L,B,Hkv,N,d] view (no copy)."""
    return t.permute(0, 1, 3, 2, 4)


def u16(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor (any device, any strides) -> numpy uint16 with the same logical shape and strides on CPU."""
    t = t.detach()
    if t.device.type != "cpu":
        base = torch.empty_strided(t.shape, t.stride(), dtype=t.dtype)
        base.copy_(t)
        t = base
    return to_u16(t)


class GpuPath(Session):
    """Device buffers of one workload and the four stages as methods (thin calls into the C ABI)."""

    def __init__(self, wl, ratio=None, device="cuda:0", slack=None, per_kv_head=0):
        self.wl = wl
        self.slack = wl.slack if slack is None else slack
        super().__init__(shape_of(wl, slack=self.slack, per_kv_head=per_kv_head), wl.ratio if ratio is None else ratio,
                         wl.alpha, device)


def gen_inputs(wl, device):
    k = full_cache(wl, "k", device)
    v = full_cache(wl, "v", device)
    qw = window_queries(wl, device)
    return k, v, qw


def rel_row_err(a: np.ndarray, b: np.ndarray) -> float:
    """max over rows of max_i |a_i - b_i| / max_i |b_i| (rows = last axis)."""
    a = a.reshape(-1, a.shape[-1]).astype(np.float64)
    b = b.reshape(-1, b.shape[-1]).astype(np.float64)
    den = np.abs(b).max(axis=1)
    den = np.where(den > 0, den, 1.0)
    return float((np.abs(a - b).max(axis=1) / den).max())


def rel_elem_err(a: np.ndarray, b: np.ndarray) -> float:
    a = a.astype(np.float64)
    b = b.astype(np.float64)
    return float((np.abs(a - b) / np.maximum(np.abs(b), 1e-30)).max())
