"""Shared plumbing of the GPU parity tests: runs the CUDA path through the binding and the CPU oracle
on the same seeded inputs.  The two sides share only the input generators of `workloads`."""
from __future__ import annotations

import numpy as np
import torch

import paper_2503_23956_b200 as ac
from workloads import decode_queries, full_cache, window_queries
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


class GpuPath:
    """Device buffers of one workload and the four stages as methods (thin calls into the C ABI)."""

    def __init__(self, wl, ratio=None, device="cuda:0", slack=None):
        self.wl = wl
        self.dev = torch.device(device)
        self.ratio = wl.ratio if ratio is None else ratio
        self.slack = wl.slack if slack is None else slack
        self.sh = shape_of(wl, slack=self.slack)
        LB = wl.n_layers * wl.batch
        self.ws = torch.empty(ac.aircache_workspace_bytes(self.sh), dtype=torch.uint8, device=self.dev)
        ac.aircache_reset_status(self.ws)
        self.scores = torch.empty((wl.n_layers, wl.batch, wl.n_visual), dtype=torch.float32, device=self.dev)
        self.mask = torch.zeros((wl.n_layers, wl.batch, wl.n_q_heads), dtype=torch.int64, device=self.dev)
        self.budgets = torch.empty((wl.n_layers, wl.batch), dtype=torch.int32, device=self.dev)
        self.strength = torch.empty((wl.n_layers, wl.batch), dtype=torch.float64, device=self.dev)
        self.skew = torch.empty((wl.n_layers, wl.batch), dtype=torch.float64, device=self.dev)
        self.rows = ac.aircache_total_rows(self.sh, self.ratio)
        self.kept_n = wl.batch * ac.aircache_kept_per_sequence(self.sh, self.ratio)
        self.k_c = torch.empty((self.rows, wl.n_kv_heads, wl.head_dim), dtype=torch.bfloat16, device=self.dev)
        self.v_c = torch.empty_like(self.k_c)
        self.offsets = torch.zeros(LB + 1, dtype=torch.int64, device=self.dev)
        self.lens = torch.zeros(LB, dtype=torch.int32, device=self.dev)
        self.kept = torch.empty(max(self.kept_n, 1), dtype=torch.int32, device=self.dev)
        self.cache = ac.ragged_view(self.k_c, self.v_c, self.offsets, self.lens, self.rows)
        self.out = torch.empty((wl.n_layers, wl.batch, wl.n_q_heads, wl.head_dim), dtype=torch.float32,
                               device=self.dev)

    def set_full(self, k_log: torch.Tensor, v_log: torch.Tensor):
        """k_log, v_log: device bf16 tensors with logical dims [L,B,Hkv,N,d]."""
        self.k_full, self.v_full = k_log, v_log
        self.full = ac.full_view(k_log, v_log)

    def score(self, qw, alpha=None):
        ac.aircache_score(self.sh, self.full, qw, self.wl.alpha if alpha is None else alpha, self.scores, self.mask,
                          self.ws)

    def budget(self, scores=None, mode=0):
        ac.aircache_budget(self.sh, self.scores if scores is None else scores, self.ratio, mode, self.budgets,
                           self.strength, self.skew, self.cache, self.ws)

    def compact(self, scores=None, budgets=None, want_kept=True):
        ac.aircache_compact(self.sh, self.full, self.scores if scores is None else scores,
                            self.budgets if budgets is None else budgets, self.ratio, self.cache,
                            self.kept if want_kept else None, self.ws)

    def decode(self, q, out=None):
        ac.aircache_decode_attn(self.sh, self.cache, q, self.out if out is None else out, self.ws)

    def status(self):
        return ac.aircache_check_status(self.ws, check=False)


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
