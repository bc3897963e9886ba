#!/usr/bin/env python
"""Benchmark of the AirCache compress-then-decode hot path on B200.

One *step* is one pass of the whole path over one batch of synthetic requests: for every resident request
batch the compression (aircache_score -> aircache_budget -> aircache_compact over all layers), then
`decode_steps` rounds of single-token decode attention (aircache_decode_attn over all layers) with a fresh query
per round.  `rotate` independent request batches (different seeds) are resident and are served round-robin, so
that consecutive decode launches never find their cache in L2.

The default workload is the largest one at 10 % visual retention: config 3 (7B shapes, 2916 visual + 256 text
tokens per sequence) at batch 64, 2 GB of compressed cache per decode launch, 256 decode rounds.

  value           tokens / s over the whole step (compression included), inputs resident in HBM
  decode_tok_s    tokens / s over the decode region of the step alone
  compress_us_per_layer   (score + budget + compact) / layers, per request batch
  roofline        decode attention: algorithmic bytes (every valid K' and V' row once, q and output) per
                  call / average duration of a call inside the timed region
  roofline_compact, roofline_score   the same for aircache_compact and aircache_score
  e2e             the same metric through aircache_pipeline_host: pinned host inputs, host outputs
  cpu_baseline    the CPU oracle timed on this host (rank 0, N = 1 only)
  allocation_ablation   budget vectors of the four allocation rules (mode flag) and their JS divergence
  workloads       every other configuration and sweep point (config 2 at 50 / 25 / 10 / 5 % retention - at 10 %
                  also with the cache resident in L2 and without CUDA graphs -, config 3 at batch 1 / 8 / 32,
                  config 4, config 5) with its full number of decode rounds, measured briefly after the main
                  run at N = 1: stage times, the three rooflines, clocks

`python bench.py --impl reference` times the CPU oracle instead (there is no other implementation of the
paper's method to run).  Under torchrun every rank runs the same workload on its own GPU with its own seeds
(no data-path collective: requests are independent); times are device times, maximum over ranks.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

METRIC = "decode_tok_s_at_10pct_visual_kv"
UNIT = "tok/s"
L2_BYTES = 126 * 2 ** 20
Q_RING, O_RING = 16, 8

# dram__bytes_read.sum + dram__bytes_write.sum of one decode_kernel launch from an ncu capture (config 3 at
# batch 16, the largest case the capture rules allow; traffic grows in proportion to the rows, so it is scaled
# to the launch that was timed).  Valid only for the kernel source it was taken on (sha1 of csrc/decode.cu,
# first 12 hex); null otherwise.
NCU_TRAFFIC = {"workload": "c3", "decode_cu_sha1": "275867bb0ec6", "bytes_per_valid_row": 2101.25}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default="c3:64", help="c1 | c2 | c3 | c4 | c5, optionally :batch and @ratio")
    ap.add_argument("--ratio", type=float, default=None)
    ap.add_argument("--alpha", type=float, default=None, help="relevance threshold of Eq. 5 (default 0.9; 0 = dense window)")
    ap.add_argument("--rotate", type=int, default=0, help="resident requests (0 = enough to exceed 2x L2)")
    ap.add_argument("--decode-steps", type=int, default=0, help="decode rounds per step (0 = the workload's)")
    ap.add_argument("--no-graph", action="store_true", help="launch through the C ABI every time (no CUDA graph)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--extra", default="c2,c2@0.5,c2@0.25,c2@0.05,c3:1,c3:8,c3:32,c4,c5",
                    help="comma list of further workloads measured briefly at N = 1 (stage times and rooflines); "
                         "\"none\" to skip")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    return ap.parse_args()


def pick_workload(spec: str, ratio, alpha=None):
    from workloads import CONFIGS
    spec, _, at = spec.partition("@")
    name, _, arg = spec.partition(":")
    wl = CONFIGS[name]
    if arg:
        wl = wl.with_(batch=int(arg))
    if at:
        wl = wl.with_(ratio=float(at))
    if ratio is not None:
        wl = wl.with_(ratio=ratio)
    if alpha is not None:
        wl = wl.with_(alpha=alpha)
    return wl


def shape_of(ac, wl, per_kv_head=0):
    return ac.shape(wl.n_layers, wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.n_visual, wl.n_text,
                    wl.window, wl.slack, wl.scale, per_kv_head)


def logical(t):
    return t.permute(0, 1, 3, 2, 4)


# --------------------------------------------------------------------------------------------------
# distributed plumbing (one process per GPU; gloo on CPU in the tests)
# --------------------------------------------------------------------------------------------------
def dist_info():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def reduce_over_ranks(local_ms: float, local_units: float, device, dist=None):
    """(max over ranks of the time, sum over ranks of the units).  Works with any backend."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return local_ms, local_units
    t = torch.tensor([local_ms], dtype=torch.float64, device=device)
    u = torch.tensor([local_units], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


# --------------------------------------------------------------------------------------------------
# clocks
# --------------------------------------------------------------------------------------------------
class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.proc = None
        self.gpu = gpu_index
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={gpu_index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "25"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for nm, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# --------------------------------------------------------------------------------------------------
# the CUDA arm
# --------------------------------------------------------------------------------------------------
def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


def decode_cu_sha1():
    p = os.path.join(ROOT, "paper_2503_23956_b200", "csrc", "decode.cu")
    return hashlib.sha1(open(p, "rb").read()).hexdigest()[:12]


def measure(ac, wl, n_dec, rotate, steps, warmup, use_graph, dev, rank, dist, append=False, per_kv_head=0):
    """Times `steps` steps of the whole path on `rotate` resident request batches of workload `wl`.
    Returns (local numbers, the sessions) -- the caller reduces over ranks."""
    from paper_2503_23956_b200.session import Session
    from workloads import decode_queries, full_cache, window_queries

    if append:
        wl = wl.with_(slack=n_dec)   # room for one appended token per decode round (Eq. 2)
    sh = shape_of(ac, wl, per_kv_head)
    reqs = []
    for i in range(rotate):
        w = wl.with_(seed=wl.seed + 1000 * rank + i)
        s = Session(sh, wl.ratio, wl.alpha, dev)
        if append:
            gen = torch.Generator(device=dev).manual_seed(wl.seed + 7 * i)
            shape_new = (n_dec, wl.n_layers * wl.batch, wl.n_kv_heads, wl.head_dim)
            s.k_new = torch.randn(shape_new, generator=gen, device=dev).to(torch.bfloat16)
            s.v_new = torch.randn(shape_new, generator=gen, device=dev).to(torch.bfloat16)
        k, v = full_cache(w, "k", dev), full_cache(w, "v", dev)
        s.set_full(logical(k), logical(v))
        s.qw = window_queries(w, dev)
        # the decode rounds cycle through Q_RING distinct query sets and O_RING output buffers (what a round
        # reads and writes besides the cache is a few KB per region)
        s.q_steps = torch.stack([decode_queries(w, t, dev) for t in range(min(n_dec, Q_RING))]).contiguous()
        s.out_steps = torch.empty((min(n_dec, O_RING),) + tuple(s.out.shape), dtype=torch.float32, device=dev)
        reqs.append(s)
    torch.cuda.synchronize()
    stream = torch.cuda.Stream(device=dev)

    def stage_score():
        for s in reqs:
            s.score(s.qw, stream=stream)

    def stage_budget():
        for s in reqs:
            s.budget(stream=stream)

    def stage_compact():
        for s in reqs:
            s.compact(want_kept=False, stream=stream)

    def stage_decode():
        for t in range(n_dec):
            for s in reqs:
                q, out = s.q_steps[t % Q_RING], s.out_steps[t % O_RING]
                if append:
                    ac.aircache_decode_step(s.sh, s.cache, q, s.k_new[t], s.v_new[t], t, out, s.ws, stream)
                else:
                    s.decode(q, out=out, stream=stream)

    stages = [("score", stage_score), ("budget", stage_budget), ("compact", stage_compact), ("decode", stage_decode)]
    graphs = {}
    with torch.cuda.stream(stream):
        for _, fn in stages[:3]:
            fn()       # one eager pass: the compressed caches exist before the decode graph is captured
        stream.synchronize()
        if use_graph:
            for name, fn in stages:
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=stream):
                    fn()
                graphs[name] = g

    def run_step(ev):
        ev[0].record(stream)
        for i, (name, fn) in enumerate(stages):
            if graphs:
                graphs[name].replay()
            else:
                fn()
            ev[i + 1].record(stream)

    def new_events():
        return [torch.cuda.Event(enable_timing=True) for _ in range(5)]

    with torch.cuda.stream(stream):
        for _ in range(warmup):
            run_step(new_events())
        stream.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        sampler = ClockSampler(dev.index or 0)
        evs = [new_events() for _ in range(steps)]
        for e in evs:
            run_step(e)
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        clocks = sampler.stop()
    for s in reqs:
        if s.status() != 0:
            raise RuntimeError("a device-side wait timed out")
    total_ms = evs[0][0].elapsed_time(evs[-1][4])
    stage_ms = {name: sum(e[i].elapsed_time(e[i + 1]) for e in evs) / steps for i, (name, _) in enumerate(stages)}
    valid_rows = sum(int(s.lens.sum().item()) for s in reqs) / rotate
    return dict(total_ms=total_ms, stage_ms=stage_ms, clocks=clocks, valid_rows=valid_rows, graph=bool(graphs)), reqs


def rooflines(ac, wl, m, rotate, n_dec, traffic=None):
    """Rooflines of decode attention, compaction and scoring from one measurement (algorithmic bytes /
    measured time).  Algorithmic bytes: decode - every valid K' and V' row once, the queries and the fp32
    outputs; compaction - every row of the compressed cache read and written once, plus the kept indices;
    scoring - every visual key once (the second pass of Eq. 7 is meant to find them in L2) plus the scores."""
    sh = shape_of(ac, wl)
    row_bytes = wl.n_kv_heads * wl.head_dim * 2
    T = ac.aircache_kept_per_sequence(sh, wl.ratio)
    LB = wl.n_layers * wl.batch
    q_out_bytes = LB * wl.n_q_heads * wl.head_dim * 6
    alg_bytes = 2 * row_bytes * m["valid_rows"] + q_out_bytes
    call_us = m["stage_ms"]["decode"] * 1e3 / (rotate * n_dec)
    peak, peak_kind = measured_peaks()

    def roof(kernel, nbytes, us, **more):
        gbs = nbytes / (us * 1e-6) / 1e9
        return {"kernel": kernel, "bound": "hbm", "achieved": gbs, "peak": peak, "peak_kind": f"of {peak_kind}",
                "unit": "GB/s", "frac": gbs / peak, "frac_of_8TBs_nominal": gbs / 8000.0, **more,
                "bytes_per_call": nbytes, "us_per_call": us}

    dec = roof("decode_kernel (one launch per aircache_decode_attn call)", alg_bytes, call_us, traffic=traffic)
    compact_bytes = 2 * alg_bytes - 2 * q_out_bytes + 4 * wl.batch * T     # read + write of every row, indices
    comp = roof("select_kernel + gather_kernel per aircache_compact call", compact_bytes,
                m["stage_ms"]["compact"] * 1e3 / rotate)
    score_bytes = LB * wl.n_visual * (row_bytes + 4)
    score = roof("elite_kernel + onepass_kernel + group_sum_kernel per aircache_score call", score_bytes,
                 m["stage_ms"]["score"] * 1e3 / rotate)
    return dec, comp, score


def default_rotate(ac, wl):
    sh = shape_of(ac, wl)
    T = ac.aircache_kept_per_sequence(sh, wl.ratio)
    cache_bytes = 2 * wl.n_kv_heads * wl.head_dim * 2 * wl.batch * (T + wl.n_layers * wl.n_text)
    return min(16, max(2, -(-2 * L2_BYTES // cache_bytes))), cache_bytes


def kernels_per_step(wl, rotate, n_dec):
    """Launches of this library's kernels in one step: elite + one-pass scoring + sum over the KV groups; budget;
    select + gather; one decode kernel per call.  (alpha = 0 and sequences too long for the one-pass kernel
    launch differently; no bench workload is either.)"""
    score = 3
    return rotate * (score + 1 + 2 + n_dec)


def config_of(ac, wl, n_dec, rotate, graph=True):
    """The `config` object of the JSON line (the reference arm reports the same one)."""
    _, cache_bytes = default_rotate(ac, wl)
    return {"workload": describe(wl), "decode_steps": n_dec, "resident_requests": rotate,
            "l2": f"inputs larger than L2: {rotate} independent request batches served round-robin, "
                  f"{rotate * cache_bytes / 2 ** 20:.0f} MiB of compressed cache cycled per decode round",
            "launch": "CUDA graph replay of the C-ABI calls" if graph else "direct C-ABI calls",
            "attention_only": True}


def decode_only(ac, reqs, n_dec, reps, dev, graph):
    """Average time (us) of one aircache_decode_attn call over the sessions `reqs` served round-robin, the
    compressed caches as they stand: `reps` timed passes of n_dec rounds after one untimed pass."""
    stream = torch.cuda.Stream(device=dev)

    def rounds():
        for t in range(n_dec):
            for s in reqs:
                s.decode(s.q_steps[t % Q_RING], out=s.out_steps[t % O_RING], stream=stream)

    with torch.cuda.stream(stream):
        g = None
        if graph:
            rounds()
            stream.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                rounds()
        run = g.replay if g is not None else rounds
        for _ in range(2):
            run()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(reps):
            run()
        e1.record(stream)
        stream.synchronize()
    return e0.elapsed_time(e1) * 1e3 / (reps * n_dec * len(reqs))


def workload_report(ac, spec, dev, rank, use_graph):
    """One further workload, measured briefly: stage times, the three rooflines, clocks."""
    w2 = pick_workload(spec, None)
    r2, _ = default_rotate(ac, w2)
    d2 = w2.steps
    m2, q2 = measure(ac, w2, d2, r2, 3, 3, use_graph, dev, rank, None)
    dec2, comp2, score2 = rooflines(ac, w2, m2, r2, d2)
    rep = {"workload": describe(w2), "decode_steps": d2, "resident_requests": r2,
           "decode_tok_s": r2 * d2 * w2.batch / (m2["stage_ms"]["decode"] * 1e-3),
           "compress_us_per_layer": (m2["stage_ms"]["score"] + m2["stage_ms"]["budget"] +
                                     m2["stage_ms"]["compact"]) * 1e3 / (r2 * w2.n_layers),
           "stage_us_per_request": {k: v * 1e3 / r2 for k, v in m2["stage_ms"].items()},
           "roofline": dec2, "roofline_compact": comp2, "roofline_score": score2, "clocks": m2["clocks"]}
    if 2 * m2["valid_rows"] * w2.n_kv_heads * w2.head_dim * 2 < L2_BYTES // 2:
        # The compressed cache of one request fits in L2: the same launch with its cache resident there (one
        # request, nothing rotated in between) next to the rotated, HBM-fed number above; and the per-call
        # time without CUDA graphs (tensor maps encoded and the launch configured on every call).
        warm_us = decode_only(ac, q2[:1], min(d2, 64), 5, dev, use_graph)
        rep["decode_l2_resident"] = {"us_per_call": warm_us, "cold_us_per_call": dec2["us_per_call"],
                                     "note": "one resident request: its compressed cache stays in L2 between calls"}
        rep["decode_no_graph_us_per_call"] = decode_only(ac, q2, min(d2, 64), 3, dev, False)
    del q2
    return rep


def per_kv_head_report(ac, spec, dev, rank, use_graph):
    """The same workload with a budget and a kept set per (layer, sequence, KV head) (aircache_shape_t.per_kv_head):
    stage times, decode time per call, and how far the KV heads' budget vectors over the layers lie from the
    shared one (Jensen-Shannon divergence, bits)."""
    wl = pick_workload(spec, None)
    rot, _ = default_rotate(ac, wl)
    d = min(wl.steps, 64)
    m, q = measure(ac, wl, d, rot, 3, 3, use_graph, dev, rank, None, per_kv_head=1)
    s = q[0]
    bud = s.budgets[:, 0].cpu().numpy().astype(np.float64)          # [L, Hkv], sequence 0
    shared = bud.sum(axis=1)

    def js(a, b):
        pa, pb = a / max(a.sum(), 1.0), b / max(b.sum(), 1.0)
        mid = 0.5 * (pa + pb)
        kl = lambda x, y: float(np.sum(x[x > 0] * np.log2(x[x > 0] / y[x > 0])))
        return 0.5 * kl(pa, mid) + 0.5 * kl(pb, mid)

    rep = {"workload": describe(wl) + " per_kv_head=1", "decode_steps": d, "resident_requests": rot,
           "stage_us_per_request": {k: v * 1e3 / rot for k, v in m["stage_ms"].items()},
           "decode_us_per_call": m["stage_ms"]["decode"] * 1e3 / (rot * d),
           "budgets_sequence0_layer_by_kv_head": bud.astype(int).tolist(),
           "js_divergence_bits_of_each_kv_head_vs_their_sum": [js(bud[:, g], shared) for g in range(bud.shape[1])]}
    del q
    return rep


def per_layer_scoring(ac, spec, dev):
    """Algorithm 1's first loop the way an engine runs it: after each layer's keys have been written (here: copied
    into place, which leaves them in L2 as a prefill kernel would) aircache_score_layers scores that layer -
    against one aircache_score call over the finished cache.  Same scores up to rounding."""
    from paper_2503_23956_b200.session import Session
    from workloads import full_cache, window_queries
    wl = pick_workload(spec, None)
    sh = shape_of(ac, wl)
    s = Session(sh, wl.ratio, wl.alpha, dev)
    k = full_cache(wl, "k", dev)
    staging = k.clone()
    s.set_full(logical(k), logical(k))
    qw = window_queries(wl, dev)

    stream = torch.cuda.Stream(device=dev)

    def timed(fn, reps=5):
        """Average time (us) of fn's work, replayed as a CUDA graph of its C-ABI calls and copies."""
        with torch.cuda.stream(stream):
            fn()
            stream.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                fn()
            g.replay()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(reps):
                g.replay()
            e1.record(stream)
            stream.synchronize()
        return e0.elapsed_time(e1) * 1e3 / reps

    def one_call():
        s.score(qw, stream=stream)

    def layer_by_layer(with_copy=True):
        for l in range(wl.n_layers):
            if with_copy:
                k[l].copy_(staging[l])
            ac.aircache_score_layers(sh, s.full, qw, wl.alpha, l, 1, s.scores, s.mask, s.ws, stream)

    def copies_only():
        for l in range(wl.n_layers):
            k[l].copy_(staging[l])

    with torch.cuda.stream(stream):
        one_call()
        want = s.scores.clone()
        layer_by_layer()
        stream.synchronize()
    same = float(((want - s.scores).abs() / want.abs().clamp_min(1e-30)).max().item())
    t_one, t_copy, t_both = timed(one_call), timed(copies_only), timed(layer_by_layer)
    return {"workload": describe(wl), "one_call_us": t_one, "layer_by_layer_after_the_layers_write_us": t_both - t_copy,
            "layer_writes_alone_us": t_copy, "max_rel_difference": same,
            "key_mb_per_layer": wl.batch * wl.n_visual * wl.n_kv_heads * wl.head_dim * 2 / 1e6,
            "note": "CUDA graph replay in all cases; a layer's keys fit in L2"}


def window_sweep(ac, spec, dev, windows=(16, 64, 128)):
    """aircache_score with the candidate window W = the last 16 / 64 / all 128 text tokens of the workload (the
    paper's own window is all of them), at the paper's threshold and with every candidate kept (alpha = 0: the
    continuous-window variants of its ablation, computed by the tcgen05 kernels)."""
    from paper_2503_23956_b200.session import Session
    from workloads import full_cache, window_queries
    wl0 = pick_workload(spec, None)
    k = full_cache(wl0, "k", dev)
    out = {}
    for W in windows:
        if W > wl0.n_text:
            continue
        wl = wl0.with_(window=W)
        s = Session(shape_of(ac, wl), wl.ratio, wl.alpha, dev)
        s.set_full(logical(k), logical(k))
        qw = window_queries(wl, dev)
        row = {}
        for alpha in (wl.alpha, 0.0):
            for _ in range(3):
                s.score(qw, alpha=alpha)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(10):
                s.score(qw, alpha=alpha)
            e1.record()
            torch.cuda.synchronize()
            bits = s.mask.cpu().numpy().view(np.uint8)
            rows = float(np.unpackbits(bits).sum()) / (wl.n_layers * wl.batch * wl.n_kv_heads)
            row[f"alpha_{alpha:g}"] = {"score_us": e0.elapsed_time(e1) * 1e2, "elite_rows_per_kv_group": rows}
        out[f"W{W}"] = row
        del s
    return {"workload": describe(wl0), "windows": out, "note": "direct C-ABI calls, one resident request"}


def run_cuda(args):
    import paper_2503_23956_b200 as ac

    rank, local_rank, world = dist_info()
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the AirCache path has no CPU fallback")
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    ac.lib()  # fail loudly if the library is missing

    wl = pick_workload(args.workload, args.ratio, args.alpha)
    n_dec = args.decode_steps or wl.steps
    sh = shape_of(ac, wl)
    rotate, cache_bytes = default_rotate(ac, wl)
    rotate = args.rotate or rotate
    warmup = max(args.warmup, 3)
    m, reqs = measure(ac, wl, n_dec, rotate, args.steps, warmup, not args.no_graph, dev, rank, dist)
    stage_ms = m["stage_ms"]
    tokens_per_step = rotate * n_dec * wl.batch
    total_ms_all, tokens_all = reduce_over_ranks(m["total_ms"], tokens_per_step * args.steps, dev, dist)
    decode_ms_all, _ = reduce_over_ranks(stage_ms["decode"], 0, dev, dist)
    traffic = None
    if NCU_TRAFFIC["bytes_per_valid_row"] and NCU_TRAFFIC["decode_cu_sha1"] == decode_cu_sha1() \
            and args.workload.startswith(NCU_TRAFFIC["workload"]):
        traffic = NCU_TRAFFIC["bytes_per_valid_row"] * m["valid_rows"]
    roof_dec, roof_comp, roof_score = rooflines(ac, wl, m, rotate, n_dec, traffic)

    result = {
        "metric": METRIC, "value": tokens_all / (total_ms_all * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": warmup, "ms_per_step": total_ms_all / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": config_of(ac, wl, n_dec, rotate, m["graph"]),
        "decode_tok_s": world * tokens_per_step / (decode_ms_all * 1e-3),
        "compress_us_per_layer": (stage_ms["score"] + stage_ms["budget"] + stage_ms["compact"]) * 1e3
                                 / (rotate * wl.n_layers),
        "stage_us_per_request": {k: v * 1e3 / rotate for k, v in stage_ms.items()},
        "roofline": roof_dec,
        "roofline_compact": roof_comp,
        "roofline_score": roof_score,
        "clocks": m["clocks"],
        "gpu_launches": args.steps * kernels_per_step(wl, rotate, n_dec),
    }
    if rank == 0 and not args.no_e2e:
        result["e2e"] = run_e2e(ac, wl, sh, reqs[0], n_dec, dev, min(args.steps, 3))
    del reqs
    torch.cuda.empty_cache()
    if rank == 0 and world == 1 and args.extra not in ("", "none"):
        result["allocation_ablation"] = allocation_ablation(ac, dev)

    # every other configuration and sweep point, briefly
    if rank == 0 and world == 1 and args.extra not in ("", "none"):
        extra = {}
        for spec in args.extra.split(","):
            try:
                extra[spec] = workload_report(ac, spec, dev, rank, not args.no_graph)
            except torch.cuda.OutOfMemoryError as e:
                # a further workload that does not fit this GPU's free memory does not take the main line down
                extra[spec] = {"skipped": f"out of device memory: {str(e)[:120]}"}
            torch.cuda.empty_cache()
        result["workloads"] = extra
        # config 2: the dense window (alpha = 0, tcgen05) and the decode rounds with the append of Eq. 2 fused in
        # (the cache grows over the rounds: lens change with every launch)
        w2 = pick_workload("c2", None)
        r2, _ = default_rotate(ac, w2)
        d3 = min(w2.steps, 64)
        m3, q3 = measure(ac, w2, d3, r2, 3, 3, not args.no_graph, dev, rank, None, append=True)
        result["decode_with_append"] = {
            "workload": describe(w2), "decode_steps": d3, "tok_s": r2 * d3 * w2.batch / (m3["stage_ms"]["decode"] * 1e-3),
            "us_per_round": m3["stage_ms"]["decode"] * 1e3 / (r2 * d3),
            "note": "aircache_decode_step (Eq. 2 append fused into the attention launch) per round and request"}
        result["score_dense_window"] = dense_window_score(w2, q3[0])
        del q3
        torch.cuda.empty_cache()
        result["window_sweep"] = window_sweep(ac, "c2", dev)
        torch.cuda.empty_cache()
        result["per_kv_head"] = per_kv_head_report(ac, "c2", dev, rank, not args.no_graph)
        torch.cuda.empty_cache()
        result["score_layer_by_layer"] = per_layer_scoring(ac, "c4", dev)
        torch.cuda.empty_cache()
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        result["cpu_baseline"] = cpu_baseline(wl, n_dec)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(result))


def dense_window_score(wl, s, reps=10):
    """aircache_score with alpha = 0 (every window query is an elite row: Eq. 7 becomes a dense
    [G*W x N_v] contraction per KV head, computed by the tcgen05 kernels), timed on one resident request."""
    for _ in range(3):
        s.score(s.qw, alpha=0.0)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        s.score(s.qw, alpha=0.0)
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / reps
    rows = wl.group * wl.window
    flops = 2 * 2.0 * rows * wl.n_visual * wl.head_dim * wl.n_kv_heads * wl.n_layers * wl.batch   # two passes
    return {"alpha": 0.0, "rows_per_kv_group": rows, "us_per_request": us, "tflops": flops / (us * 1e-6) / 1e12,
            "key_bytes": wl.n_visual * wl.n_kv_heads * wl.head_dim * 2 * wl.n_layers * wl.batch,
            "note": "both passes of Eq. 7 on tcgen05; FLOPs count the unpadded rows, keys are read once per pass"}


def allocation_ablation(ac, dev, spec="c2", text_amp_hi=8.0):
    """The allocation variants of the paper's ablation (strength + skewness, strength only, skewness only,
    uniform) as budget vectors over the layers of sequence 0, from aircache_budget's mode flag, and the
    Jensen-Shannon divergence (bits) of every variant's distribution of the budget over the layers from the
    combined rule's.  Run on a variant of the workload whose candidate-window text keys take a share of the
    softmax that differs by layer (generator option text_amp_hi): on the plain configurations the visual tokens
    hold nearly all of the mass in every layer and the strength term has nothing to tell apart."""
    from paper_2503_23956_b200.session import Session
    from workloads import full_cache, window_queries
    wl = pick_workload(spec, None).with_(text_amp_hi=text_amp_hi)
    s = Session(shape_of(ac, wl), wl.ratio, wl.alpha, dev)
    k = full_cache(wl, "k", dev)
    s.set_full(logical(k), logical(k))
    s.score(window_queries(wl, dev))
    LB = wl.n_layers * wl.batch
    budgets = torch.empty_like(s.budgets)
    strength = torch.empty_like(s.strength)
    layout = ac.ragged_view(None, None, torch.empty(LB + 1, dtype=torch.int64, device=s.dev),
                            torch.empty(LB, dtype=torch.int32, device=s.dev), 0)
    names = ["strength_and_skewness", "strength_only", "skewness_only", "uniform"]
    vec = {}
    for mode, name in enumerate(names):
        ac.aircache_budget(s.sh, s.scores, s.ratio, mode, budgets, strength, None, layout, s.ws)
        vec[name] = budgets[:, 0].cpu().numpy().astype(np.float64)

    def js(a, b):
        pa, pb = a / max(a.sum(), 1.0), b / max(b.sum(), 1.0)
        m = 0.5 * (pa + pb)

        def kl(x, y):
            nz = x > 0
            return float(np.sum(x[nz] * np.log2(x[nz] / y[nz])))
        return 0.5 * kl(pa, m) + 0.5 * kl(pb, m)

    ref = vec[names[0]]
    st = strength[:, 0].cpu().numpy()
    return {"workload": describe(wl) + f" text_amp_hi={text_amp_hi:g}",
            "strength_per_layer_sequence0": [round(float(x), 4) for x in st],
            "budgets_per_layer_sequence0": {n: [int(x) for x in v] for n, v in vec.items()},
            "js_divergence_bits_vs_combined": {n: js(vec[n], ref) for n in names[1:]}}


def describe(wl):
    return (f"{wl.name} r={wl.ratio:g} B={wl.batch} L={wl.n_layers} Hq={wl.n_q_heads} Hkv={wl.n_kv_heads} "
            f"d={wl.head_dim} Nv={wl.n_visual} Nt={wl.n_text} W={wl.window}")


def run_e2e(ac, wl, sh, s, n_dec, dev, steps):
    """Same metric through aircache_pipeline_host: every step uploads the full K cache and the queries from
    pinned host memory, reads the surviving V rows from pinned host memory in place, runs the whole path and
    downloads the attention outputs and the budgets."""
    stream = torch.cuda.current_stream(dev)
    k_tm = s.k_full.permute(0, 1, 3, 2, 4)      # back to the token-major storage order
    v_tm = s.v_full.permute(0, 1, 3, 2, 4)
    assert k_tm.is_contiguous()
    def pinned_copy(t):
        h = torch.empty(t.shape, dtype=t.dtype, pin_memory=True)
        h.copy_(t)
        return h

    h_k, h_v = pinned_copy(k_tm), pinned_copy(v_tm)
    h_full = ac.full_view(logical(h_k), logical(h_v))
    d_k, d_v = torch.empty_like(k_tm), torch.empty_like(v_tm)
    q_all = s.q_steps[torch.arange(n_dec, device=dev) % s.q_steps.shape[0]]      # [n_dec, L, B, Hq, d]
    h_qw, h_q = pinned_copy(s.qw), pinned_copy(q_all)
    d_qw, d_q = torch.empty_like(s.qw), torch.empty_like(q_all)
    del q_all
    d_out = torch.empty((n_dec,) + tuple(s.out.shape), dtype=torch.float32, device=dev)
    h_out = torch.empty(d_out.shape, dtype=torch.float32, pin_memory=True)
    h_bud = torch.empty(s.budgets.shape, dtype=torch.int32, pin_memory=True)

    def once():
        ac.aircache_pipeline_host(sh, h_full, h_k.numel(), d_k, d_v, h_qw, d_qw, h_q, d_q, n_dec, wl.alpha,
                                  wl.ratio, 0, s.scores, s.budgets, s.cache, d_out, h_out, h_bud, s.ws, stream)

    once()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(steps):
        once()      # synchronises internally after the device-to-host copies
    dt = (time.perf_counter() - t0) / steps
    # K whole; of V (page-locked, read in place by the gather kernel) only the rows of the compressed cache
    v_in_place = ac.aircache_host_range_is_mapped(h_v)
    v_bytes = int(s.lens.sum().item()) * wl.n_kv_heads * wl.head_dim * 2 if v_in_place else h_v.numel() * 2
    h2d = h_k.numel() * 2 + v_bytes + h_qw.numel() * 2 + h_q.numel() * 2
    d2h = h_out.numel() * 4 + h_bud.numel() * 4
    return {"value": n_dec * wl.batch / dt, "unit": UNIT, "ms_per_step": dt * 1e3, "requests_per_step": 1,
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "api": "aircache_pipeline_host",
            "v_read_in_place": bool(v_in_place)}


# --------------------------------------------------------------------------------------------------
# the CPU oracle, timed as it stands (cpu_baseline leg and --impl reference)
# --------------------------------------------------------------------------------------------------
class OracleSample:
    """A bounded sample of the workload for the CPU oracle: `max_seqs` sequences (all layers) and `dec_rounds`
    decode rounds over their compressed caches.  Inputs are generated once; run() times the oracle."""

    def __init__(self, wl, max_seqs=1, dec_rounds=16):
        import oracle
        from workloads import decode_queries, full_cache, window_queries
        from workloads.synth import to_u16
        oracle.build()
        self.oracle, self.wl = oracle, wl
        self.seqs = list(range(min(max_seqs, wl.batch)))
        w1 = wl.with_(batch=len(self.seqs))
        self.dm = oracle.Dims(w1.n_layers, w1.batch, w1.n_q_heads, w1.n_kv_heads, w1.head_dim, w1.n_visual,
                              w1.n_text, w1.window)
        k, v = full_cache(wl, "k", "cpu", seqs=self.seqs), full_cache(wl, "v", "cpu", seqs=self.seqs)
        self.kl, self.vl = to_u16(k).transpose(0, 1, 3, 2, 4), to_u16(v).transpose(0, 1, 3, 2, 4)
        self.qw = to_u16(window_queries(wl, "cpu", seqs=self.seqs))
        self.qs = [to_u16(decode_queries(wl, t, "cpu", seqs=self.seqs)) for t in range(dec_rounds)]

    def run(self, n_dec):
        """Seconds for the whole batch and n_dec rounds, scaled linearly from the sample (sequences are
        independent and decode rounds alike, so the oracle's cost is linear in both)."""
        oracle, wl, dm = self.oracle, self.wl, self.dm
        t0 = time.perf_counter()
        sc = oracle.score(dm, self.kl, self.qw, wl.scale, wl.alpha)
        st, sk = oracle.moments(sc["scores"])
        bud = oracle.allocate(st, sk, wl.n_visual, wl.ratio, 0)
        cp = oracle.compact(dm, 0, self.kl, self.vl, sc["scores"], bud)
        t_comp = time.perf_counter() - t0
        t0 = time.perf_counter()
        for q in self.qs:
            oracle.decode(dm, cp["k"], cp["v"], cp["offsets"], cp["lens"], q, wl.scale)
        t_dec = (time.perf_counter() - t0) / len(self.qs)
        f = wl.batch / len(self.seqs)
        return {"t_compress": t_comp * f, "t_decode_round": t_dec * f, "threads": oracle.num_threads(),
                "sample": f"oracle on {len(self.seqs)} of {wl.batch} sequence(s), all {wl.n_layers} layers: whole "
                          f"compression once + {len(self.qs)} decode rounds; scaled linearly to the batch and to "
                          f"{n_dec} rounds"}


def cpu_baseline(wl, n_dec):
    s = OracleSample(wl).run(n_dec)
    step_s = s["t_compress"] + n_dec * s["t_decode_round"]
    return {"value": n_dec * wl.batch / step_s, "unit": UNIT, "cores": s["threads"], "kind": "oracle",
            "sample": s["sample"], "compress_us_per_layer": s["t_compress"] * 1e6 / wl.n_layers,
            "decode_tok_s": wl.batch / s["t_decode_round"]}


class _HostArithmetic:
    """The two host-side numbers config_of() needs, without the CUDA library (the reference arm runs without it)."""

    @staticmethod
    def shape(*a):
        return a

    @staticmethod
    def aircache_kept_per_sequence(sh, ratio):
        n_layers, n_visual = sh[0], sh[5]
        return int(np.floor(ratio * float(n_visual * n_layers) + 0.5))


def run_reference(args):
    rank, _, world = dist_info()
    if rank != 0:
        return
    wl = pick_workload(args.workload, args.ratio, args.alpha)
    n_dec = args.decode_steps or wl.steps
    rotate = args.rotate or default_rotate(_HostArithmetic, wl)[0]
    sample = OracleSample(wl)
    for _ in range(min(args.warmup, 1)):
        sample.run(n_dec)
    times, last = [], None
    for _ in range(args.steps):
        last = sample.run(n_dec)
        times.append(last["t_compress"] + n_dec * last["t_decode_round"])
    step_s = sum(times) / len(times)
    value = n_dec * wl.batch / step_s
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": step_s * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_of(_HostArithmetic, wl, n_dec, rotate, not args.no_graph),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": last["threads"], "kind": "oracle",
                         "sample": last["sample"]},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


if __name__ == "__main__":
    a = parse_args()
    if a.impl == "reference":
        run_reference(a)
    else:
        run_cuda(a)
