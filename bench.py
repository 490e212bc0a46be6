#!/usr/bin/env python
"""Benchmark of the BF1 forward hot path on B200.

One step = one route plan (bf1_plan_route) followed by eight back-to-back bf1_attn_fwd
calls on eight independent sets of Q/K/V at n = 32768, 16 query / 8 KV heads, d = 128:
the eight retrofitted layers of the paper's model sharing one plan (Section 3.4, 4.3).
The eight input sets together are ~2.1 GB, far larger than L2, so no flush is needed.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Prints ONE JSON line (rank 0).  `value` is selected-pair TFLOP/s = 4 * d * pairs * Hq * layers
/ step time, summed over ranks (each rank runs its own independent copy: weak scaling, no
collective on the data path).  `--impl reference` times the CPU oracle on the host cores.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import torch  # noqa: E402

import bf1_inputs as I  # noqa: E402

WORKLOAD = "qwen_32k"
LAYERS = 8
METRIC = "bf1_fwd_prefill_selected_pair_tflops"
UNIT = "TFLOP/s"


# ---- closed-form work accounting (Proposition 1; no oracle needed) -------------------------
def degree(j: int) -> int:
    if j <= 3:
        return j + 1
    return int(math.floor(math.log2(j))) + 3 - (1 if j & (j - 1) == 0 else 0)


def row_pairs(i: int, b: int = 64) -> int:
    return b * (degree(i // b) - 1) + (i % b) + 1


def selected_pairs(n: int, b: int = 64) -> int:
    total = 0
    nb = (n + b - 1) // b
    for j in range(nb):
        rows = min(b, n - j * b)
        total += rows * b * (degree(j) - 1) + rows * (rows + 1) // 2
    return total


def flops(pairs: int, d: int, hq: int) -> float:
    return 4.0 * d * pairs * hq


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"bf16_tflops": p["bf16_tflops"], "bf16_tflops_sustained": p.get("bf16_tflops_sustained"),
                "hbm_gbs": p["hbm_gbs"], "source": "measured"}
    return {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


# ---- clock sampling through NVML (read-only) ------------------------------------------------
class ClockSampler:
    REASONS = {0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
               0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting"}

    def __init__(self, index: int):
        self.samples, self.reasons, self.stop_flag, self.thread, self.max_mhz = [], set(), False, None, None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        while not self.stop_flag:
            try:
                self.samples.append(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM))
                r = self.nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                for bit, name in self.REASONS.items():
                    if r & bit and name != "gpu_idle":
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.004)

    def start(self):
        if self.nv:
            self.thread = threading.Thread(target=self._run, daemon=True)
            self.thread.start()

    def stop(self):
        self.stop_flag = True
        if self.thread:
            self.thread.join()
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ---- reference arm / cpu baseline: the oracle on the host cores ------------------------------
def oracle_rate(w, q, k, v, target_s: float):
    """Time the CPU oracle on a strided row sample sized for ~target_s seconds.
    Returns (TFLOP/s, seconds, description, threads)."""
    from oracle import bf1_oracle as O
    n = w.seqlens[0]
    cfg = O.cfg(w.block, w.local_blocks, w.global_first, w.dyadic)
    probe = list(range(0, n, 32))
    t0 = time.perf_counter()
    O.attn_route(cfg, q, k, v, w.cu_seqlens(), rows=probe)
    t_probe = time.perf_counter() - t0
    full_est = t_probe * sum(row_pairs(i) for i in range(0, n, 16)) * 16 / max(sum(row_pairs(i) for i in probe), 1)
    stride = max(1, int(math.ceil(full_est / target_s)))
    rows = list(range(0, n, stride))
    t0 = time.perf_counter()
    O.attn_route(cfg, q, k, v, w.cu_seqlens(), rows=rows)
    dt = time.perf_counter() - t0
    fl = flops(sum(row_pairs(i) for i in rows), w.d, w.hq)
    return fl / dt / 1e12, dt, "every %d-th token row of one %s layer (%d rows x %d heads)" % (
        stride, w.name, len(rows), w.hq), O.threads()


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = I.WORKLOADS[WORKLOAD]
    q, k, v = I.draw_qkv(w)
    vals, secs, desc, thr = [], [], "", 1
    for s in range(args.warmup + args.steps):
        val, dt, desc, thr = oracle_rate(w, q, k, v, target_s=min(2.0, 150.0 / (args.warmup + args.steps)))
        if s >= args.warmup:
            vals.append(val)
            secs.append(dt)
    value = sum(vals) / len(vals)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * sum(secs) / len(secs),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "config": {"workload": "%s x %d layers, 16q/8kv d128 b64, BF1 route" % (WORKLOAD, LAYERS),
                       "sample_per_step": desc},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": thr, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ---- multi-rank bookkeeping (weak scaling: every rank runs its own copy, no data-path collective) --
def rank_layer_seed_offset(rank: int, layer: int) -> int:
    """Each rank draws its own inputs: rank r uses layers r*LAYERS .. r*LAYERS + LAYERS - 1."""
    return layer + rank * LAYERS


def max_over_ranks(ms: float, dist, device) -> float:
    """The job takes as long as its slowest rank (all-reduce MAX; identity on one rank)."""
    if dist is None:
        return ms
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(step_flops: float, ms_per_step: float, world: int) -> float:
    """Selected-pair TFLOP/s of the whole job: every rank did step_flops in ms_per_step."""
    return world * step_flops / (ms_per_step * 1e-3) / 1e12


# ---- our arm -----------------------------------------------------------------------------------
def time_region(fn, reps, stream):
    """Median CUDA-event time (ms) of fn() over reps runs."""
    out = []
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        fn()
        e1.record(stream)
        e1.synchronize()
        out.append(e0.elapsed_time(e1))
    return statistics.median(out)


GRAPH_LAUNCHES = 16


def graph_timer(fn, dev, launches=GRAPH_LAUNCHES):
    """Capture `launches` back-to-back calls of fn() in a CUDA graph on a side stream and return
    replay(reps) -> list of per-launch times in ms (CUDA events around each replay).  The GPU runs
    the launches without the host in between, so the figure is kernel time: launch gaps of a busy
    stream included, Python, ctypes and driver latency of an idle one excluded."""
    side = torch.cuda.Stream(device=dev)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        for _ in range(2):
            fn()
        side.synchronize()
        with torch.cuda.graph(graph, stream=side):
            for _ in range(launches):
                fn()

    def replay(reps):
        out = []
        with torch.cuda.stream(side):
            for _ in range(reps):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(side)
                graph.replay()
                e1.record(side)
                e1.synchronize()
                out.append(e0.elapsed_time(e1) / launches)
        return out
    return replay


def timed_with_clock(replay, local_rank, reps=30, min_ms=40.0):
    """Median per-launch time of `reps` replays, then the median SM clock sampled (read-only NVML) while
    the same graph keeps replaying for at least `min_ms`: (ms, MHz or None)."""
    ts = replay(reps)
    ms = statistics.median(ts)
    sampler = ClockSampler(local_rank)
    sampler.start()
    t0 = time.perf_counter()
    while (time.perf_counter() - t0) * 1e3 < min_ms:
        replay(4)
    clk = sampler.stop()
    return ms, clk["sm_mhz"]


def sweep(bf1, dev, local_rank=0):
    """BF1 vs the library's dense-causal mode, per layer, with the paper's protocol (Section 4.3):
    5 warm-ups, 30 repetitions, two opposite pattern orders, median of the order medians.  A repetition
    is one replay of a CUDA graph of 16 launches (kernel-only time per launch); `*_host_inclusive_ms` is
    the same protocol with one Python call between two events on an idle stream, i.e. what a caller
    that launches a single layer and waits would see.  Each point also carries the median SM clock
    while it ran and time x clock (kilo-cycles), so that a point measured while the clocks were
    still pulled down by a long dense launch can be told from a slow kernel."""
    out = []
    for name in ("qwen_2k", "qwen_4k", "qwen_8k", "qwen_16k", "qwen_32k"):
        w = I.WORKLOADS[name]
        q, k, v = (t.to(dev) for t in I.draw_qkv(w))
        cu = bf1.cu_seqlens_tensor(w.seqlens, dev)
        route = bf1.plan_route(cu, w.max_seqlen)
        o = torch.empty_like(q)
        lse = torch.empty((w.hq, w.total_tokens), dtype=torch.float32, device=dev)
        stream = torch.cuda.current_stream()
        f_s = lambda: bf1.attn_fwd(q, k, v, cu, w.max_seqlen, route, out=o, lse=lse)
        work = torch.zeros(4, dtype=torch.int32, device=dev)
        f_d = lambda: bf1.dense_causal_fwd(q, k, v, cu, w.max_seqlen, out=o, lse=lse, work=work)
        torch.cuda.synchronize()
        g_s, g_d = graph_timer(f_s, dev), graph_timer(f_d, dev)
        meds = {"bf1": [], "dense": []}
        host = {"bf1": [], "dense": []}
        mhz = {"bf1": [], "dense": []}
        for order in (("dense", "bf1"), ("bf1", "dense")):
            for which in order:
                g = g_s if which == "bf1" else g_d
                g(5)
                ms, clk = timed_with_clock(g, local_rank)
                meds[which].append(ms)
                if clk:
                    mhz[which].append(clk)
                f = f_s if which == "bf1" else f_d
                for _ in range(5):
                    f()
                host[which].append(time_region(f, 30, stream))
        ms_s, ms_d = statistics.median(meds["bf1"]), statistics.median(meds["dense"])
        n = w.seqlens[0]
        pairs = selected_pairs(n)
        m = int(math.log2(n // 64))
        closed = n * 64 * m - 64 * 64 * m + n * 65 // 2        # n log n total for n = 64 * 2^m (Prop. 1's accounting)
        point = {"n": n, "bf1_ms": round(ms_s, 5), "dense_ms": round(ms_d, 5), "speedup": round(ms_d / ms_s, 3),
                 "bf1_tflops": round(flops(pairs, w.d, w.hq) / ms_s / 1e9, 1),
                 "bf1_frac_of_bf16_peak": round(flops(pairs, w.d, w.hq) / ms_s / 1e9 / measured_peaks()["bf16_tflops"], 4),
                 "dense_tflops": round(flops(n * (n + 1) // 2, w.d, w.hq) / ms_d / 1e9, 1),
                 "bf1_host_inclusive_ms": round(statistics.median(host["bf1"]), 5),
                 "dense_host_inclusive_ms": round(statistics.median(host["dense"]), 5),
                 "selected_pairs_planner": int(route.total_pairs.item()), "selected_pairs_closed_form": closed,
                 "pair_reduction": round(n * (n + 1) / 2 / pairs, 3),
                 "timing": "CUDA graph of %d launches per repetition" % GRAPH_LAUNCHES,
                 "inputs": "L2-warm (same buffers re-run)"}
        if mhz["bf1"] and mhz["dense"]:
            c_s, c_d = statistics.median(mhz["bf1"]), statistics.median(mhz["dense"])
            point.update({"bf1_sm_mhz": c_s, "dense_sm_mhz": c_d, "bf1_kcycles": round(ms_s * c_s, 1),
                          "dense_kcycles": round(ms_d * c_d, 1), "speedup_in_cycles": round(ms_d * c_d / (ms_s * c_s), 3)})
        out.append(point)
        del q, k, v, o, lse, g_s, g_d
    # the ragged batch (3001, 8192, 12345, 16384 tokens) in one varlen launch
    w = I.WORKLOADS["ragged"]
    q, k, v = (t.to(dev) for t in I.draw_qkv(w))
    cu = bf1.cu_seqlens_tensor(w.seqlens, dev)
    route = bf1.plan_route(cu, w.max_seqlen)
    o = torch.empty_like(q)
    lse = torch.empty((w.hq, w.total_tokens), dtype=torch.float32, device=dev)
    f = lambda: bf1.attn_fwd(q, k, v, cu, w.max_seqlen, route, out=o, lse=lse)
    torch.cuda.synchronize()
    g = graph_timer(f, dev)
    g(5)
    ms = statistics.median(g(30))
    pairs = sum(selected_pairs(x) for x in w.seqlens)
    out.append({"ragged_seqlens": list(w.seqlens), "bf1_ms": round(ms, 5),
                "bf1_tflops": round(flops(pairs, w.d, w.hq) / ms / 1e9, 1),
                "selected_pairs_planner": int(route.total_pairs.item()), "selected_pairs_closed_form": pairs})
    return out


def host_route_arrays(lists, n, block=64):
    """Arrays for bf1.Route.from_host from explicit per-block lists of one sequence of n tokens."""
    counts = [len(x) for x in lists]
    deg = max(counts)
    kv_idx = [list(x) + [-1] * (deg - len(x)) for x in lists]
    pairs = []
    for j, x in enumerate(lists):
        rows = min(block, n - j * block)
        pairs.append(rows * block * (len(x) - 1) + rows * (rows + 1) // 2)
    order = sorted(range(len(lists)), key=lambda g: (-counts[g], g))
    return dict(qb_seq=[0] * len(lists), qb_block=list(range(len(lists))), kv_count=counts, kv_idx=kv_idx,
                pair_count=pairs, order=order, total_pairs=sum(pairs))


def topology_sweep(bf1, dev):
    """Does the route's topology change the kernel's cost?  (Section 5.1 reports the same sparse kernel time for BF1 and its
    sliding and static-random controls of equal pair count.)  One 32K layer through routes with about
    the same number of block pairs: BF1, a sliding window with the closest pair count, a seeded static-random
    non-local graph with exactly BF1's list lengths (uploaded from the host, not planned), BF1 without block
    0, dyadic predecessors without a local window.  Kernel time from a CUDA graph of 16 launches; reported
    per executed tile as well, so that small differences in the pair budget cancel."""
    w = I.WORKLOADS["qwen_32k"]
    n = w.seqlens[0]
    q, k, v = (t.to(dev) for t in I.draw_qkv(w))
    cu = bf1.cu_seqlens_tensor(w.seqlens, dev)
    o = torch.empty_like(q)
    lse = torch.empty((w.hq, w.total_tokens), dtype=torch.float32, device=dev)
    nb = n // 64
    target = sum(degree(j) for j in range(nb))
    best_w = min(range(1, 64), key=lambda ww: abs(sum(min(j, ww) + 1 for j in range(nb)) - target))
    routes = [("bf1", bf1.RouteCfg()), ("sliding W=%d (equal block-pair budget)" % best_w,
                                        bf1.RouteCfg(local_blocks=best_w, global_first=0, dyadic=0)),
              ("static random graph (seed 17, BF1's list lengths, host-built lists)", None),
              ("bf1 without block 0", bf1.RouteCfg(global_first=0)),
              ("dyadic only (W=0)", bf1.RouteCfg(local_blocks=0, global_first=0, dyadic=1))]
    out = []
    for name, cfg in routes:
        if cfg is None:
            route = bf1.Route.from_host(device=dev, **host_route_arrays(I.static_random_lists(nb, seed=17), n))
        else:
            route = bf1.plan_route(cu, n, cfg)
        f = lambda: bf1.attn_fwd(q, k, v, cu, n, route, out=o, lse=lse)
        torch.cuda.synchronize()
        g = graph_timer(f, dev)
        g(5)
        ms = statistics.median(g(30))
        route.check_status()
        tiles = int(route.kv_count[:nb].sum().item()) * w.hkv
        out.append({"route": name, "block_pairs": tiles // w.hkv, "ms": round(ms, 5),
                    "ns_per_tile_per_sm": round(ms * 1e6 / (tiles / 148.0), 1)})
    return out


def backward_sweep(bf1, dev):
    """Backward over the same route (Section 4.2's gradient gate), one layer, 4K .. 32K: CUDA-event median of
    10 calls (each derives the inverse route, then runs the dQ and the dK/dV kernel).  FLOPs credited =
    10 * d * pairs * Hq: the five products of the chain rule per block pair against the forward's two (the
    two kernels both recompute S and dP, seven MMA groups in all: not credited)."""
    out = []
    stream = torch.cuda.current_stream()
    for name in ("qwen_4k", "qwen_8k", "qwen_16k", "qwen_32k"):
        w = I.WORKLOADS[name]
        q, k, v = (t.to(dev) for t in I.draw_qkv(w))
        d_o = torch.randn(q.shape, generator=torch.Generator(device=dev).manual_seed(w.seed), device=dev,
                          dtype=torch.float32).to(torch.bfloat16)
        cu = bf1.cu_seqlens_tensor(w.seqlens, dev)
        route = bf1.plan_route(cu, w.max_seqlen)
        o, lse = bf1.attn_fwd(q, k, v, cu, w.max_seqlen, route)
        ws = bf1.bwd_workspace(route, w.total_tokens, w.hq, w.hkv, w.d, dev)
        f = lambda: bf1.attn_bwd(q, k, v, o, lse, d_o, cu, w.max_seqlen, route, workspace=ws)
        for _ in range(3):
            f()
        ms = time_region(f, 10, stream)
        route.check_status()
        pairs = selected_pairs(w.seqlens[0])
        tf = 10.0 * w.d * pairs * w.hq / ms / 1e9
        out.append({"n": w.seqlens[0], "bwd_ms": round(ms, 4), "bwd_tflops": round(tf, 1),
                    "frac_of_bf16_peak": round(tf / measured_peaks()["bf16_tflops"], 4)})
        del q, k, v, d_o, o, lse, ws
    return out


def decode_sweep(bf1, dev):
    """Selected-page one-token decode (Section 5.4, Table 3's grid: 32K / 64K context, batch 1 / 8 / 32).
    A pool of 8192 physical pages (2.1 GB of K and V, far larger than L2) and 32 random page tables per
    point; the 32 decode calls (each with its own plan, so each reads different, mostly cold pages) are
    captured in one CUDA graph so that host launch latency does not hide the kernel, and the graph's
    time is divided by 32.  Planning is timed the same way, on its own: one plan serves a whole
    64-token route epoch.  Bytes = selected K and V pages, read once."""
    out = []
    hq, hkv, d, reps = 16, 8, 128, 32
    peaks = measured_peaks()
    # These calls take microseconds and are bound by latency, so they follow the SM clock closely; the sweep that
    # runs before them ends with seconds of dense launches that leave the clock power-capped.  Let it recover.
    torch.cuda.synchronize()
    time.sleep(1.0)
    g = torch.Generator(device=dev)
    g.manual_seed(777)
    pool = 8192
    k_pages = torch.randn((pool, 64, hkv, d), generator=g, device=dev, dtype=torch.bfloat16)
    v_pages = torch.randn((pool, 64, hkv, d), generator=g, device=dev, dtype=torch.bfloat16)
    side = torch.cuda.Stream(device=dev)
    for n in (32768, 65536):
        for batch in (1, 8, 32):
            nb = n // 64
            q = torch.randn((batch, hq, d), generator=g, device=dev, dtype=torch.bfloat16)
            sl = torch.full((batch,), n, dtype=torch.int32, device=dev)
            tables = [torch.randint(0, pool, (batch, nb), generator=g, device=dev, dtype=torch.int32) for _ in range(reps)]
            plans = [bf1.plan_decode(sl, t) for t in tables]
            ws = bf1.decode_workspace(batch, hq, hkv, plans[0].max_degree, d, dev)
            o = torch.empty_like(q)
            lse = torch.empty((hq, batch), dtype=torch.float32, device=dev)
            torch.cuda.synchronize()
            timings = {}
            for what in ("plan", "decode"):
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.stream(side):
                    calls = (lambda i: bf1.plan_decode(sl, tables[i], plan=plans[i])) if what == "plan" else \
                            (lambda i: bf1.decode_fwd(q, k_pages, v_pages, sl, plans[i], ws, out=o, lse=lse))
                    for i in range(2):
                        calls(i)
                    side.synchronize()
                    with torch.cuda.graph(graph, stream=side):
                        for i in range(reps):
                            calls(i)
                    ts = []
                    for _ in range(12):
                        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                        e0.record(side)
                        graph.replay()
                        e1.record(side)
                        e1.synchronize()
                        ts.append(e0.elapsed_time(e1) / reps)
                timings[what] = statistics.median(ts[4:])
            assert all(int(p.status.item()) == 0 for p in plans)
            nbytes = int(plans[0].count.sum().item()) * 64 * hkv * d * 2 * 2
            ms = timings["decode"]
            out.append({"context": n, "batch": batch, "pages_per_seq": int(plans[0].count[0].item()),
                        "plan_us": round(timings["plan"] * 1e3, 2), "decode_us": round(ms * 1e3, 2),
                        "selected_kv_bytes": nbytes, "gbs": round(nbytes / ms / 1e6, 1),
                        "frac_of_hbm_peak": round(nbytes / ms / 1e6 / peaks["hbm_gbs"], 4),
                        "timing": "32 calls on 32 random page tables in one CUDA graph, pool 2.1 GB"})
    return out


def run_single_decode(args, bf1, dev):
    """A few plain decode calls at batch `--batch`, context 32768, each on its own random page table."""
    hq, hkv, d, batch, n, pool = 16, 8, 128, args.batch, 32768, 8192
    g = torch.Generator(device=dev)
    g.manual_seed(778)
    k_pages = torch.randn((pool, 64, hkv, d), generator=g, device=dev, dtype=torch.bfloat16)
    v_pages = torch.randn((pool, 64, hkv, d), generator=g, device=dev, dtype=torch.bfloat16)
    q = torch.randn((batch, hq, d), generator=g, device=dev, dtype=torch.bfloat16)
    sl = torch.full((batch,), n, dtype=torch.int32, device=dev)
    total = args.warmup + args.steps
    tables = [torch.randint(0, pool, (batch, n // 64), generator=g, device=dev, dtype=torch.int32) for _ in range(total)]
    plans = [bf1.plan_decode(sl, t) for t in tables]
    ws = bf1.decode_workspace(batch, hq, hkv, plans[0].max_degree, d, dev)
    o = torch.empty_like(q)
    lse = torch.empty((hq, batch), dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()
    ts = []
    for i in range(total):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        bf1.decode_fwd(q, k_pages, v_pages, sl, plans[i], ws, out=o, lse=lse)
        e1.record(stream)
        e1.synchronize()
        ts.append(e0.elapsed_time(e1))
    nbytes = int(plans[0].count.sum().item()) * 64 * hkv * d * 2 * 2
    ms = statistics.median(ts[args.warmup:])
    print(json.dumps({"single": "decode batch %d context 32768" % batch, "ms": ms, "steps": args.steps,
                      "selected_kv_bytes": nbytes, "gbs_incl_launch_latency": nbytes / ms / 1e6}))


def run_single(args):
    """A few plain launches of one mode on one named workload (what the ncu captures run)."""
    import paper_2608_20427_b200 as bf1
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    if args.mode == "decode":
        return run_single_decode(args, bf1, dev)
    w = I.WORKLOADS[args.single]
    q, k, v = (t.to(dev) for t in I.draw_qkv(w))
    cu = bf1.cu_seqlens_tensor(w.seqlens, dev)
    route = bf1.plan_route(cu, w.max_seqlen)
    o = torch.empty_like(q)
    lse = torch.empty((w.hq, w.total_tokens), dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()
    work = torch.zeros(4, dtype=torch.int32, device=dev)
    if args.mode == "bwd":
        d_o = torch.randn(q.shape, generator=torch.Generator(device=dev).manual_seed(w.seed), device=dev,
                          dtype=torch.float32).to(torch.bfloat16)
        bf1.attn_fwd(q, k, v, cu, w.max_seqlen, route, out=o, lse=lse)
        ws = bf1.bwd_workspace(route, w.total_tokens, w.hq, w.hkv, w.d, dev)
        f = lambda: bf1.attn_bwd(q, k, v, o, lse, d_o, cu, w.max_seqlen, route, workspace=ws)
        pairs = int(2.5 * sum(selected_pairs(n) for n in w.seqlens))   # five MMA groups against the forward's two
    elif args.mode == "dense":
        f = lambda: bf1.dense_causal_fwd(q, k, v, cu, w.max_seqlen, out=o, lse=lse, work=work)
        pairs = sum(n * (n + 1) // 2 for n in w.seqlens)
    else:
        f = lambda: bf1.attn_fwd(q, k, v, cu, w.max_seqlen, route, out=o, lse=lse)
        pairs = sum(selected_pairs(n) for n in w.seqlens)
    for _ in range(args.warmup):
        f()
    ms = time_region(f, args.steps, stream)
    route.check_status()
    print(json.dumps({"single": args.single, "mode": args.mode, "ms": ms, "steps": args.steps,
                      "tflops": flops(pairs, w.d, w.hq) / ms / 1e9}))


def run_ours(args):
    import paper_2608_20427_b200 as bf1
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    bf1.load()

    w = I.WORKLOADS[WORKLOAD]
    n, T = w.seqlens[0], w.total_tokens
    pairs = selected_pairs(n)
    layer_flops = flops(pairs, w.d, w.hq)
    step_flops = layer_flops * LAYERS

    # eight independent layers' inputs: host (pinned) and device copies
    host = []
    for layer in range(LAYERS):
        host.append(tuple(t.pin_memory() for t in I.draw_qkv(w, layer=rank_layer_seed_offset(rank, layer))))
    devb = [tuple(t.to(dev) for t in h) for h in host]
    outs = [torch.empty((T, w.hq, w.d), dtype=torch.bfloat16, device=dev) for _ in range(LAYERS)]
    lses = [torch.empty((w.hq, T), dtype=torch.float32, device=dev) for _ in range(LAYERS)]
    cu = bf1.cu_seqlens_tensor(w.seqlens, dev)
    cap, deg = bf1.route_capacity(1, T, n)
    route = bf1.Route.empty(cap, deg, dev)
    stream = torch.cuda.current_stream()

    attn_ms = []   # per step: time of the eight attention launches alone

    def step(record=False):
        bf1.plan_route(cu, n, route=route)
        if record:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
        for layer in range(LAYERS):
            q, k, v = devb[layer]
            bf1.attn_fwd(q, k, v, cu, n, route, out=outs[layer], lse=lses[layer])
        if record:
            e1.record(stream)
            attn_ms.append((e0, e1))

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        step(record=True)
    e1.record(stream)
    barrier()
    clocks = sampler.stop()
    total_ms = e0.elapsed_time(e1)
    route.check_status()
    assert int(route.total_pairs.item()) == pairs
    total_ms = max_over_ranks(total_ms, dist, dev)
    ms_per_step = total_ms / args.steps
    value = whole_job_value(step_flops, ms_per_step, world)
    kern_ms = statistics.mean(a.elapsed_time(b) for a, b in attn_ms) / LAYERS

    # ---- end to end: pinned host buffers -> device -> kernels -> host, every step
    o_host = [torch.empty((T, w.hq, w.d), dtype=torch.bfloat16).pin_memory() for _ in range(LAYERS)]
    l_host = [torch.empty((w.hq, T), dtype=torch.float32).pin_memory() for _ in range(LAYERS)]
    h2d = sum(t.numel() * t.element_size() for h in host for t in h)
    d2h = sum(t.numel() * t.element_size() for t in o_host + l_host)

    # three streams: host->device copies, kernels, device->host copies; a layer's kernel waits for its
    # inputs, its read-back waits for the kernel, and the next step's upload of a layer waits until the
    # previous kernel on those buffers is done.  The two copy directions and the kernels overlap.
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    ev_in = [torch.cuda.Event() for _ in range(LAYERS)]
    ev_k = [torch.cuda.Event() for _ in range(LAYERS)]
    ev_out = [torch.cuda.Event() for _ in range(LAYERS)]

    def e2e_step(first=False):
        bf1.plan_route(cu, n, route=route)
        for layer in range(LAYERS):
            with torch.cuda.stream(s_in):
                if not first:
                    s_in.wait_event(ev_k[layer])        # the previous step's kernel has read these buffers
                for src, dst in zip(host[layer], devb[layer]):
                    dst.copy_(src, non_blocking=True)
                ev_in[layer].record(s_in)
            stream.wait_event(ev_in[layer])
            if not first:
                stream.wait_event(ev_out[layer])        # the previous step's read-back of these outputs is done
            q, k, v = devb[layer]
            bf1.attn_fwd(q, k, v, cu, n, route, out=outs[layer], lse=lses[layer])
            ev_k[layer].record(stream)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_k[layer])
                o_host[layer].copy_(outs[layer], non_blocking=True)
                l_host[layer].copy_(lses[layer], non_blocking=True)
                ev_out[layer].record(s_out)

    def e2e_join():
        stream.wait_stream(s_in)
        stream.wait_stream(s_out)

    e2e_steps = max(2, min(args.steps, 5))
    e2e_step(first=True)
    e2e_join()
    barrier()
    e0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    e2e_join()
    e1.record(stream)
    barrier()
    assert torch.equal(o_host[LAYERS - 1], outs[LAYERS - 1].cpu())   # the read-back really happened
    e2e_ms = e0.elapsed_time(e1)
    e2e_ms = max_over_ranks(e2e_ms, dist, dev)
    e2e_value = whole_job_value(step_flops, e2e_ms / e2e_steps, world)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    achieved = layer_flops / (kern_ms * 1e-3) / 1e12
    traffic = None   # dram__bytes_read + dram__bytes_write per launch, from the committed ncu summary
    tpath = os.path.join(ROOT, "profiles", "attn_fwd_kernel_qwen_32k.md")
    if os.path.exists(tpath):
        import re
        with open(tpath) as f:
            m = re.search(r"^dram_bytes_per_launch\s*=\s*(\d+)", f.read(), re.M)
        traffic = int(m.group(1)) if m else None
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "%s x %d layers per step (one plan + %d bf1_attn_fwd), B=1 n=32768 16q/8kv d128 b64, "
                               "BF1 route (W=2, block 0, dyadic)" % (WORKLOAD, LAYERS, LAYERS),
                   "ms_per_layer": ms_per_step / LAYERS, "selected_pairs_per_layer": pairs,
                   "l2": "inputs larger than L2 (8 layers x 268 MB rotate)", "timing": "CUDA events, max over ranks"},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": e2e_ms / e2e_steps, "steps": e2e_steps},
        "gpu_launches": args.steps * (LAYERS + 1),
        "roofline": {"bound": "tensor", "kernel": "attn_fwd_kernel<128>", "achieved": achieved,
                     "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": achieved / peaks["bf16_tflops"],
                     "peak_source": "%s burst bf16 (MEASURED_PEAKS.json)" % peaks["source"],
                     "frac_of_sustained": (achieved / peaks["bf16_tflops_sustained"]) if peaks["bf16_tflops_sustained"] else None,
                     "traffic": traffic, "algorithmic_flops_per_launch": layer_flops,
                     "kernel_ms_per_launch": kern_ms},
    }
    if not args.no_sweep and world == 1:
        line["sweep"] = sweep(bf1, dev, local_rank)
        line["decode"] = decode_sweep(bf1, dev)
        line["backward"] = backward_sweep(bf1, dev)
        line["topology"] = topology_sweep(bf1, dev)
    if not args.no_cpu and world == 1:
        # the oracle, as it stands, on the host cores: whole layers of the same step (every row),
        # as many of the eight as fit in about 12 s (at least one, at most all eight)
        from oracle import bf1_oracle as O
        ocfg = O.cfg(w.block, w.local_blocks, w.global_first, w.dyadic)
        t_cpu, layers_done = 0.0, 0
        while layers_done < LAYERS and (layers_done == 0 or t_cpu * (layers_done + 1) / layers_done < 14.0):
            q, k, v = (t.contiguous() for t in host[layers_done])
            t0 = time.perf_counter()
            O.attn_route(ocfg, q, k, v, w.cu_seqlens())
            t_cpu += time.perf_counter() - t0
            layers_done += 1
        cpu_model = ""
        try:
            with open("/proc/cpuinfo") as f:
                cpu_model = next((ln.split(":", 1)[1].strip() for ln in f if ln.startswith("model name")), "")
        except OSError:
            pass
        line["cpu_baseline"] = {"value": layers_done * layer_flops / t_cpu / 1e12, "unit": UNIT, "cores": O.threads(),
                                "kind": "oracle", "seconds": t_cpu, "cpu_model": cpu_model,
                                "sample": "%d of the step's %d layers, every token row (%s, fp32 oracle)" % (
                                    layers_done, LAYERS, w.name)}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def spawn_ranks(n: int) -> int:
    """`bench.py --gpus N` started bare: run this same command line as N ranks (one process per GPU)
    under torch.distributed.run on this node and pass its exit code on."""
    import socket
    import subprocess
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.run(cmd).returncode


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--single", default=None, choices=sorted(I.WORKLOADS),
                    help="only time `--steps` launches of one workload (used for profiling)")
    ap.add_argument("--mode", default="bf1", choices=["bf1", "dense", "decode", "bwd"])
    ap.add_argument("--batch", type=int, default=32, help="sequences per decode call (with --single ... --mode decode)")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and not args.single:
        sys.exit(spawn_ranks(args.gpus))
    if args.single:
        run_single(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
