"""Counter-based synthetic K/V/Q generator shaped like the paper's LVLM workloads.

Recipe (per layer l, sequence b, KV head g):
  * K, V, window queries and decode queries are standard normal, quantised to 65536 quantile
    levels that are exactly representable in bf16: value = table[hash(key, index) >> 16].
  * "Planted relevance": a random 5 % of the visual tokens get K[g, i] += a_lb * u_lbg and every
    window query of the heads in group g gets += q_gain * u_lbg, where u_lbg is a unit vector,
    a_lb ~ U(0.5, 4) differs per layer (so the skewness of the importance scores differs per
    layer) and q_gain = sqrt(head_dim).  For video-shaped workloads the planted tokens are
    drawn only from a few "hot" frames chosen per sequence.
  * Optional (text_amp_hi > 0, off in the five configurations): the text keys of the candidate window get
    += t_lb * u_lbg with t_lb ~ U(0, text_amp_hi) per layer, so that the window's own text keys take a share
    of the softmax that differs by layer (and with it the allocation strength of the layers).
  * Small random objects (a_lb, u_lbg, planted sets, hot frames) come from numpy's PCG64
    seeded with (seed, sequence, tag); they are computed on the host and uploaded.
All fp32 arithmetic on the large tensors is one addition of two fp32 numbers followed by a
round-to-nearest-even conversion to bf16, identical on CPU and GPU.
"""
from __future__ import annotations

import math
import zlib
from dataclasses import dataclass, replace

import numpy as np
import torch

_M32 = 0xFFFFFFFF
BASE_SEED = 20250331


@dataclass(frozen=True)
class Workload:
    name: str
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    batch: int
    n_visual: int
    n_text: int
    ratio: float
    steps: int
    window: int = 16
    slack: int = 0
    alpha: float = 0.9            # relevance threshold of the elite window (the method's, not the generator's)
    plant_frac: float = 0.05
    amp_lo: float = 0.5           # planting amplitude a_lb ~ U(amp_lo, amp_hi)
    amp_hi: float = 4.0
    n_frames: int = 0             # > 0: video-shaped, n_visual = n_frames * tokens per frame
    hot_frames: int = 3
    text_amp_hi: float = 0.0      # > 0: the text keys of the candidate window get + t_lb * u_lbg, t_lb ~ U(0, text_amp_hi)
    seed: int = BASE_SEED

    @property
    def n_tokens(self) -> int:
        return self.n_visual + self.n_text

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def scale(self) -> float:
        return float(np.float32(1.0 / math.sqrt(self.head_dim)))

    @property
    def q_gain(self) -> float:
        return float(np.float32(math.sqrt(self.head_dim)))

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


_7B = dict(n_layers=28, n_q_heads=28, n_kv_heads=4, head_dim=128)
CONFIGS = {
    # tiny synthetic LVLM cache: the correctness workhorse
    "c1": Workload("c1_tiny", 4, 8, 2, 64, batch=1, n_visual=576, n_text=64, ratio=0.10, steps=16),
    # Qwen2-7B-shaped decoder with one high-resolution image
    "c2": Workload("c2_7b_image", **_7B, batch=1, n_visual=7290, n_text=128, ratio=0.10, steps=128),
    # batch sweep (use .with_(batch=...)): independent seeds per sequence
    "c3": Workload("c3_7b_batch", **_7B, batch=64, n_visual=2916, n_text=256, ratio=0.10, steps=256),
    # video-shaped: 32 frames x 196 tokens, relevance concentrated in 3 frames
    "c4": Workload("c4_7b_video", **_7B, batch=4, n_visual=6272, n_text=512, ratio=0.10, steps=512, n_frames=32),
    # Qwen2-72B-shaped long-context stress
    "c5": Workload("c5_72b_long", 80, 64, 8, 128, batch=8, n_visual=7290, n_text=2048, ratio=0.05, steps=1024),
}

_TABLE = None


def normal_table() -> torch.Tensor:
    """65536 standard-normal quantiles, rounded to bf16-representable fp32 values (CPU tensor)."""
    global _TABLE
    if _TABLE is None:
        p = (torch.arange(65536, dtype=torch.float64) + 0.5) / 65536.0
        z = torch.special.ndtri(p)
        _TABLE = z.to(torch.float32).to(torch.bfloat16).to(torch.float32).contiguous()
    return _TABLE


_TABLE_DEV: dict = {}


def _table_on(device) -> torch.Tensor:
    device = torch.device(device)
    key = (device.type, device.index)
    if key not in _TABLE_DEV:
        _TABLE_DEV[key] = normal_table().to(device)
    return _TABLE_DEV[key]


def _mix32_py(x: int) -> int:
    x &= _M32
    x ^= x >> 16
    x = (x * 0x7FEB352D) & _M32
    x ^= x >> 15
    x = (x * 0x2C1B3C6D) & _M32
    x ^= x >> 16
    return x


def _mix32(x: torch.Tensor) -> torch.Tensor:
    """Integer mixer on int64 lanes holding values < 2**32 (all products stay below 2**63)."""
    x = x ^ (x >> 16)
    x = (x * 0x7FEB352D) & _M32
    x = x ^ (x >> 15)
    x = (x * 0x2C1B3C6D) & _M32
    x = x ^ (x >> 16)
    return x


def _stream_key(seed: int, tag: str, *ids: int) -> int:
    k = _mix32_py(seed ^ zlib.crc32(tag.encode()))
    for i in ids:
        k = _mix32_py(k ^ _mix32_py(int(i) + 0x632BE5AB))
    return k


def _normal_slab(key: int, start: int, count: int, device) -> torch.Tensor:
    """`count` table-quantised normals for element indices start..start+count-1 of stream `key` (fp32)."""
    idx = torch.arange(start, start + count, dtype=torch.int64, device=device)
    h = _mix32(((idx & _M32) * 0x3C6EF372 & _M32) ^ key)
    h = _mix32(h ^ (idx >> 32) ^ 0x1B873593)
    return _table_on(device)[h >> 16]


def _rng(wl: Workload, b: int, tag: str) -> np.random.Generator:
    return np.random.default_rng(np.random.SeedSequence([wl.seed, zlib.crc32(wl.name.encode()), b,
                                                         zlib.crc32(tag.encode())]))


@dataclass
class Plan:
    """Host-side small random objects of one workload."""
    amp: np.ndarray          # f32 [L, B]            planting amplitude a_lb
    u: np.ndarray            # f32 [L, B, Hkv, d]    unit directions
    planted: np.ndarray      # bool [L, B, Nv]       planted visual tokens
    hot: np.ndarray | None   # i64 [B, hot_frames]   hot frames (video-shaped only)
    text_amp: np.ndarray | None = None   # f32 [L, B]  amplitude t_lb on the window's text keys (text_amp_hi > 0 only)


_PLANS: dict = {}


def plan(wl: Workload) -> Plan:
    if wl in _PLANS:
        return _PLANS[wl]
    L, B, Hkv, d, Nv = wl.n_layers, wl.batch, wl.n_kv_heads, wl.head_dim, wl.n_visual
    amp = np.empty((L, B), np.float32)
    u = np.empty((L, B, Hkv, d), np.float32)
    planted = np.zeros((L, B, Nv), bool)
    hot = np.empty((B, wl.hot_frames), np.int64) if wl.n_frames else None
    n_plant = int(math.floor(wl.plant_frac * Nv))
    for b in range(B):
        amp[:, b] = _rng(wl, b, "amp").uniform(wl.amp_lo, wl.amp_hi, size=L).astype(np.float32)
        dirs = _rng(wl, b, "dir").standard_normal((L, Hkv, d))
        dirs /= np.linalg.norm(dirs, axis=-1, keepdims=True)
        u[:, b] = dirs.astype(np.float32)
        if wl.n_frames:
            per = Nv // wl.n_frames
            hot[b] = np.sort(_rng(wl, b, "frames").choice(wl.n_frames, wl.hot_frames, replace=False))
            pool = np.concatenate([np.arange(f * per, (f + 1) * per) for f in hot[b]])
        else:
            pool = np.arange(Nv)
        g = _rng(wl, b, "plant")
        for l in range(L):
            planted[l, b, g.choice(pool, n_plant, replace=False)] = True
    text_amp = None
    if wl.text_amp_hi > 0:
        # the window's text keys pull attention mass away from the visual tokens, by a different amount in every
        # layer: the visual share of the softmax (the allocation strength of Eq. 9) then differs by layer
        text_amp = np.stack([_rng(wl, b, "textamp").uniform(0.0, wl.text_amp_hi, size=L) for b in range(B)],
                            axis=1).astype(np.float32)
    p = Plan(amp, u, planted, hot, text_amp)
    _PLANS[wl] = p
    return p


def full_cache(wl: Workload, which: str, device="cpu", layers=None, seqs=None) -> torch.Tensor:
    """bf16 [L', B', N, Hkv, d] (token-major) slice of the full K ('k') or V ('v') cache."""
    assert which in ("k", "v")
    layers = list(range(wl.n_layers)) if layers is None else list(layers)
    seqs = list(range(wl.batch)) if seqs is None else list(seqs)
    N, Hkv, d, Nv = wl.n_tokens, wl.n_kv_heads, wl.head_dim, wl.n_visual
    out = torch.empty((len(layers), len(seqs), N, Hkv, d), dtype=torch.bfloat16, device=device)
    pl = plan(wl) if which == "k" else None
    for li, l in enumerate(layers):
        for bi, b in enumerate(seqs):
            z = _normal_slab(_stream_key(wl.seed, wl.name + which, l, b), 0, N * Hkv * d, device).view(N, Hkv, d)
            if which == "k":
                add = torch.from_numpy(pl.amp[l, b] * pl.u[l, b]).to(device)             # f32 [Hkv, d]
                mask = torch.from_numpy(pl.planted[l, b]).to(device)                     # bool [Nv]
                zv = z[:Nv]
                z[:Nv] = torch.where(mask[:, None, None], zv + add[None], zv)
                if pl.text_amp is not None:
                    z[N - wl.window:] += torch.from_numpy(pl.text_amp[l, b] * pl.u[l, b]).to(device)[None]
            out[li, bi] = z.to(torch.bfloat16)
    return out


def window_queries(wl: Workload, device="cpu", layers=None, seqs=None) -> torch.Tensor:
    """bf16 [L', B', W, Hq, d]: queries of the last W text tokens (the observation-window candidates)."""
    layers = list(range(wl.n_layers)) if layers is None else list(layers)
    seqs = list(range(wl.batch)) if seqs is None else list(seqs)
    W, Hq, d, G = wl.window, wl.n_q_heads, wl.head_dim, wl.group
    out = torch.empty((len(layers), len(seqs), W, Hq, d), dtype=torch.bfloat16, device=device)
    pl = plan(wl)
    gain = np.float32(wl.q_gain)
    for li, l in enumerate(layers):
        for bi, b in enumerate(seqs):
            z = _normal_slab(_stream_key(wl.seed, wl.name + "qwin", l, b), 0, W * Hq * d, device).view(W, Hq, d)
            add = torch.from_numpy(np.repeat(gain * pl.u[l, b], G, axis=0)).to(device)   # f32 [Hq, d]
            out[li, bi] = (z + add[None]).to(torch.bfloat16)
    return out


def decode_queries(wl: Workload, step: int, device="cpu", layers=None, seqs=None) -> torch.Tensor:
    """bf16 [L', B', Hq, d]: the query token of decode step `step` (plain standard normal)."""
    layers = list(range(wl.n_layers)) if layers is None else list(layers)
    seqs = list(range(wl.batch)) if seqs is None else list(seqs)
    Hq, d = wl.n_q_heads, wl.head_dim
    out = torch.empty((len(layers), len(seqs), Hq, d), dtype=torch.bfloat16, device=device)
    for li, l in enumerate(layers):
        for bi, b in enumerate(seqs):
            z = _normal_slab(_stream_key(wl.seed, wl.name + "qdec", l, b, step), 0, Hq * d, device)
            out[li, bi] = z.view(Hq, d).to(torch.bfloat16)
    return out


def to_u16(t: torch.Tensor) -> np.ndarray:
    """bf16 torch tensor (CPU) -> numpy uint16 view of the same bits and strides."""
    assert t.dtype == torch.bfloat16 and t.device.type == "cpu"
    return t.view(torch.int16).numpy().view(np.uint16)
