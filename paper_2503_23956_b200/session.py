"""Device buffers of one problem shape plus the stages as one-line calls into the C ABI.

Allocation only: torch provides the device memory and the current stream, every stage runs in
libaircache.so.  Used by the benchmark, the smoke check and the tests."""
from __future__ import annotations

import torch

from . import (Shape, aircache_budget, aircache_check_status, aircache_compact, aircache_decode_attn,
               aircache_kept_per_sequence, aircache_reset_status, aircache_score, aircache_total_rows,
               aircache_workspace_bytes, full_view, ragged_view)


class Session:
    def __init__(self, sh: Shape, ratio: float, alpha: float = 0.9, device="cuda:0"):
        self.sh, self.ratio, self.alpha = sh, ratio, alpha
        self.dev = torch.device(device)
        L, B, Hq, Hkv, d, Nv = sh.n_layers, sh.batch, sh.n_q_heads, sh.n_kv_heads, sh.head_dim, sh.n_visual
        cells = Hkv if sh.per_kv_head else 1      # units with a budget of their own per (layer, sequence)
        row_heads = 1 if sh.per_kv_head else Hkv  # KV heads stored in one row of the compressed cache
        LB = L * B * cells
        per = (cells,) if sh.per_kv_head else ()
        with torch.cuda.device(self.dev):
            self.ws = torch.empty(aircache_workspace_bytes(sh), dtype=torch.uint8, device=self.dev)
            aircache_reset_status(self.ws)
        self.scores = torch.empty((L, B) + per + (Nv,), dtype=torch.float32, device=self.dev)
        words = (sh.window + 63) // 64
        self.mask = torch.zeros((L, B, Hq) + ((words,) if words > 1 else ()), dtype=torch.int64, device=self.dev)
        self.budgets = torch.empty((L, B) + per, dtype=torch.int32, device=self.dev)
        self.strength = torch.empty((L, B) + per, dtype=torch.float64, device=self.dev)
        self.skew = torch.empty((L, B) + per, dtype=torch.float64, device=self.dev)
        self.rows = aircache_total_rows(sh, ratio)
        self.kept_n = B * aircache_kept_per_sequence(sh, ratio)
        self.k_c = torch.empty((self.rows, row_heads, d), dtype=torch.bfloat16, device=self.dev)
        self.v_c = torch.empty_like(self.k_c)
        self.offsets = torch.zeros(LB + 1, dtype=torch.int64, device=self.dev)
        self.lens = torch.zeros(LB, dtype=torch.int32, device=self.dev)
        self.kept = torch.empty(max(self.kept_n, 1), dtype=torch.int32, device=self.dev)
        self.cache = ragged_view(self.k_c, self.v_c, self.offsets, self.lens, self.rows)
        self.out = torch.empty((L, B, Hq, d), dtype=torch.float32, device=self.dev)
        self.full = None

    def set_full(self, k_log: torch.Tensor, v_log: torch.Tensor):
        """k_log, v_log: device bf16 tensors with logical dims [L, B, Hkv, N, d] (any strides, d contiguous)."""
        self.k_full, self.v_full = k_log, v_log
        self.full = full_view(k_log, v_log)

    def score(self, qw, alpha=None, stream=None):
        aircache_score(self.sh, self.full, qw, self.alpha if alpha is None else alpha, self.scores, self.mask,
                       self.ws, stream)

    def budget(self, scores=None, mode=0, stream=None):
        aircache_budget(self.sh, self.scores if scores is None else scores, self.ratio, mode, self.budgets,
                        self.strength, self.skew, self.cache, self.ws, stream)

    def compact(self, scores=None, budgets=None, want_kept=True, stream=None):
        aircache_compact(self.sh, self.full, self.scores if scores is None else scores,
                         self.budgets if budgets is None else budgets, self.ratio, self.cache,
                         self.kept if want_kept else None, self.ws, stream)

    def decode(self, q, out=None, stream=None):
        aircache_decode_attn(self.sh, self.cache, q, self.out if out is None else out, self.ws, stream)

    def status(self) -> int:
        return aircache_check_status(self.ws, check=False)
