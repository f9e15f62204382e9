#!/usr/bin/env python
"""Benchmark of the scale-step re-layout: reshard GB/s and scale-step latency.

A step is one pass of the whole hot path - expert re-pack, attention re-slice,
KV head re-split / re-paging - over one synthetic model, enqueued back to back on
one stream.  `value` is 2 x bytes moved / time (every byte of the new layout is
read once and written once), with the arenas already resident in HBM.  `e2e` is
the same step on pinned HOST buffers through emoe_reshard_step_host, copies
included.  With --gpus N (under torchrun) every rank runs its own replica of the
workload: the path has no exchange step on one device per model.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2_mid]
                    [--impl reference] [--only-main]
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "reshard_gbs"
UNIT = "GB/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_PEAK_GBS = 6650.0
# DRAM bytes per launch of the dominant kernel from the ncu capture summarised under
# profiles/ (workload -> read + written bytes), or None while no capture covers it
NCU_TRAFFIC = {
    # whole step of a 2-layer cut (bulk launch 2.6139 + 2.5671 GB, the attention shard's vector
    # launch 0.0677 + 0.0236 GB; at full size both are one bulk launch): x12 for 24 layers
    "c2_mid": 12 * (2613877000 + 2567138000 + 67747000 + 23625000),
}


def measured_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_PEAK_GBS, "fallback"


# ---- clocks ---------------------------------------------------------------------------

class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self) -> dict:
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except ValueError:
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "samples": len(sm),
                "reasons": sorted(reasons)}


# ---- the device-resident arm ------------------------------------------------------------

def setup(name, torch, E, W, WD, n_layers=None):
    wl = W.make_workload(name, n_layers=n_layers)
    t0 = time.perf_counter()
    plan = E.Plan(wl.shape, wl.old, wl.new)
    plan_ms = (time.perf_counter() - t0) * 1e3
    kinds = {E.PHASE_EXPERTS: W.KIND_EXPERTS, E.PHASE_ATTN: W.KIND_ATTN, E.PHASE_KV: W.KIND_KV}
    src, dst = [], []
    for ph in range(3):
        src.append(WD.alloc_filled(plan.arena_bytes(ph, E.SIDE_OLD), wl.seed, kinds[ph]))
        dst.append(WD.alloc_const(plan.arena_bytes(ph, E.SIDE_NEW)))
    return wl, plan, src, dst, plan_ms


def one_step(plan, src, dst, stream):
    plan.reshard_step(src, dst, stream)


def time_steps(torch, plan, src, dst, steps, warmup, stream, barrier=None):
    """Total ms over `steps` whole steps (emoe_reshard_step, back to back), events recorded
    on the stream the kernels are launched on."""
    torch.cuda.synchronize()   # the arenas were filled on the default stream
    with torch.cuda.stream(stream):
        for _ in range(warmup):
            one_step(plan, src, dst, stream)
        stream.synchronize()
        if barrier:
            barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            one_step(plan, src, dst, stream)
        e1.record(stream)
        stream.synchronize()
        torch.cuda.synchronize()
    return e0.elapsed_time(e1)


def time_phases(torch, plan, src, dst, steps, stream):
    """Mean ms of each phase run on its own (the per-phase entry points), for the report."""
    with torch.cuda.stream(stream):
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(steps)]
        for i in range(steps):
            ev[i][0].record(stream)
            plan.reshard_experts(src[0], dst[0], stream)
            ev[i][1].record(stream)
            plan.reshard_attn(src[1], dst[1], stream)
            ev[i][2].record(stream)
            plan.reshard_kv(src[2], dst[2], stream)
            ev[i][3].record(stream)
        stream.synchronize()
    return [statistics.mean(e[k].elapsed_time(e[k + 1]) for e in ev) for k in range(3)]


def time_graph_steps(torch, plan, src, dst, steps, warmup, stream):
    """The same step captured once in a CUDA graph and replayed: what a launch-bound
    (tiny) configuration costs when the host is taken out of the loop.  Returns ms/step."""
    with torch.cuda.stream(stream):
        one_step(plan, src, dst, stream)
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            one_step(plan, src, dst, stream)
        for _ in range(warmup):
            graph.replay()
        stream.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            graph.replay()
        e1.record(stream)
        stream.synchronize()
    return e0.elapsed_time(e1) / steps


def config_report(E, plan, wl, total_ms, phase_ms, steps, peak, plan_ms):
    st = [plan.stats(ph) for ph in range(3)]
    moved = sum(s["bytes_moved"] for s in st)
    read = sum(s["bytes_read"] for s in st)
    ms = total_ms / steps
    gbs = 2 * moved / (ms * 1e-3) / 1e9
    names = ["experts", "attn", "kv"]
    return {
        "workload": wl.name, "reconfig": wl.notes, "bytes_moved": moved, "bytes_read": read,
        "scale_step_ms": round(ms, 4), "reshard_gbs": round(gbs, 1),
        "pct_of_nominal_8000": round(100 * gbs / NOMINAL_HBM_GBS, 2),
        "pct_of_measured_peak": round(100 * gbs / peak, 2),
        "algorithmic_min_gbs": round((moved + read) / (ms * 1e-3) / 1e9, 1),
        "planner_ms": round(plan_ms, 3),
        "phases": {n: {"ms": round(phase_ms[k], 4),
                       "gbs": round(2 * st[k]["bytes_moved"] / (phase_ms[k] * 1e-3) / 1e9, 1)
                       if phase_ms[k] > 0 else None,
                       "bytes_moved": st[k]["bytes_moved"], "segments": st[k]["n_segments"],
                       "launches": plan.num_launches(k)} for k, n in enumerate(names)},
        "launches_per_step": plan.num_launches(E.PHASE_STEP),
    }


# ---- CPU baseline: the oracle, as it stands, on the host cores ---------------------------

def cpu_baseline_sample(wl, src_layer_getter, budget_s=12.0, max_layers=64):
    """Times the single-threaded oracle on whole layers of the workload (layers are
    independent; they are taken in order, cyclically), until `budget_s` of CPU work or
    `max_layers` layer passes."""
    import oracle
    wl1 = wl.with_layers(1)
    sh = wl1.shape
    sizes_new = [oracle.expert_arena_bytes(sh, wl.new.placement),
                 oracle.attn_arena_bytes(sh, wl.new.tp),
                 oracle.kv_arena_bytes(sh, wl.new.tp, wl.new.kv_num_blocks)]
    used = sum(-(-n // sh.kv_block_tokens) for n in wl.old.seq_lens)
    kv_moved = (2 * used * sh.kv_block_tokens * sh.n_kv_heads * sh.head_dim * sh.elem_bytes)
    moved_per_layer = sum(sizes_new[0]) + sum(sizes_new[1]) + kv_moved
    spent, layers = 0.0, 0
    for i in range(max_layers):
        src = src_layer_getter(i % wl.shape.n_layers)
        dst = [[np.empty(n, np.uint8) for n in s] for s in sizes_new]
        for group in dst:
            for a in group:
                a.fill(0xCD)     # also faults the pages in before the clock starts
        t0 = time.perf_counter()
        oracle.reshard_experts(sh, wl.old.placement, wl.new.placement, src[0], dst[0])
        oracle.reshard_attn(sh, wl.old.tp, wl.new.tp, src[1], dst[1])
        oracle.reshard_kv(sh, wl.old, wl.new, src[2], dst[2])
        spent += time.perf_counter() - t0
        layers += 1
        if spent >= budget_s:
            break
    gbs = 2 * moved_per_layer * layers / spent / 1e9
    return {"value": round(gbs, 3), "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": "%d layer passes (of %d layers) of %s, all three phases, single thread; "
                      "%.2f s of CPU work" % (layers, wl.shape.n_layers, wl.name, spent),
            "ms_per_layer": round(spent / layers * 1e3, 2),
            "projected_step_ms": round(spent / layers * 1e3 * wl.shape.n_layers, 1)}


def cpu_baseline_all_cores(wl, src_layer_getter, max_threads=16):
    """The same oracle, still one thread per call, run on different layers at once (layers
    are independent): what the host manages with all its cores, so that the single-thread
    figure is not the only yardstick.  One pass: one layer per thread."""
    import concurrent.futures as cf
    import oracle
    wl1 = wl.with_layers(1)
    sh = wl1.shape
    n = max(1, min(max_threads, os.cpu_count() or 1, wl.shape.n_layers))
    try:
        import psutil
        per_layer = sum(oracle.expert_arena_bytes(sh, wl.new.placement)) * 2.6
        n = max(1, min(n, int(psutil.virtual_memory().available * 0.5 // max(per_layer, 1))))
    except Exception:
        pass
    sizes_new = [oracle.expert_arena_bytes(sh, wl.new.placement),
                 oracle.attn_arena_bytes(sh, wl.new.tp),
                 oracle.kv_arena_bytes(sh, wl.new.tp, wl.new.kv_num_blocks)]
    used = sum(-(-x // sh.kv_block_tokens) for x in wl.old.seq_lens)
    kv_moved = 2 * used * sh.kv_block_tokens * max(sh.n_kv_heads, wl.new.tp) * sh.head_dim * sh.elem_bytes
    moved_per_layer = sum(sizes_new[0]) + sum(sizes_new[1]) + kv_moved
    work = []
    for i in range(n):
        src = src_layer_getter(i)
        dst = [[np.full(k, 0xCD, np.uint8) for k in s] for s in sizes_new]
        work.append((src, dst))

    def run(item):
        src, dst = item
        oracle.reshard_experts(sh, wl.old.placement, wl.new.placement, src[0], dst[0])
        oracle.reshard_attn(sh, wl.old.tp, wl.new.tp, src[1], dst[1])
        oracle.reshard_kv(sh, wl.old, wl.new, src[2], dst[2])

    with cf.ThreadPoolExecutor(n) as ex:
        t0 = time.perf_counter()
        list(ex.map(run, work))
        spent = time.perf_counter() - t0
    return {"value": round(2 * moved_per_layer * n / spent / 1e9, 3), "unit": UNIT, "cores": n,
            "kind": "oracle", "sample": "%d layers of %s at once, one oracle thread each; %.2f s"
                                        % (n, wl.name, spent)}


def device_layer_getter(torch, src, n_layers):
    def get(l):
        out = []
        for group in src:
            g = []
            for t in group:
                per = t.numel() // n_layers
                g.append(t[l * per:(l + 1) * per].cpu().numpy())
            out.append(g)
        return out
    return get


def host_layer_getter(wl, W, WD, sizes_old_per_layer):
    kinds = [W.KIND_EXPERTS, W.KIND_ATTN, W.KIND_KV]
    def get(l):
        return [[WD.host_slice(wl.seed, kinds[ph], r, l * n, n) for r, n in enumerate(sizes)]
                for ph, sizes in enumerate(sizes_old_per_layer)]
    return get


# ---- e2e: host buffers through emoe_reshard_step_host ------------------------------------

def run_e2e(torch, plan, src, dst, steps, stream):
    """src/dst: device arenas (reused as staging).  Host buffers are pinned copies."""
    torch.cuda.synchronize()
    h_src = [[t.cpu().pin_memory() for t in g] for g in src]
    h_dst = [[torch.empty(t.numel(), dtype=torch.uint8).pin_memory() for t in g] for g in dst]
    h2d = sum(t.numel() for g in h_src for t in g)
    d2h = sum(t.numel() for g in h_dst for t in g)
    plan.reshard_step_host(h_src, h_dst, src, dst, stream)   # warm-up
    stream.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        plan.reshard_step_host(h_src, h_dst, src, dst, stream)
    e1.record(stream)
    stream.synchronize()
    ms = e0.elapsed_time(e1) / steps
    return ms, h2d, d2h


# ---- C5: reshard on a low-priority stream beside a grouped expert GEMM -------------------

def run_overlap(torch, E, plan, wl, src, dst, peak, budgets=(0, 96, 48, 24)):
    """Victim: 8 active experts x 256 tokens (top-8 routing: every active expert sees all
    tokens), gate/up/down bf16 batched GEMMs (torch.bmm, a measurement fixture, not part
    of the library) on a high-priority stream, weights taken from the old expert arena of
    rank 0, the layer cycling per step."""
    v = wl.victim
    A, T, D, F = v["active_experts"], v["tokens"], v["d_model"], v["d_ff"]
    L = wl.shape.n_layers
    arena = src[0][0].view(torch.bfloat16)
    n_slots = len(wl.old.placement[0])
    m = D * F
    slab = arena.view(L, 3, n_slots, m)
    lo, hi = torch.cuda.Stream.priority_range()[1], torch.cuda.Stream.priority_range()[0]
    lo, hi = max(lo, hi), min(lo, hi)          # numerically larger = lower priority
    s_main = torch.cuda.Stream(priority=hi)
    s_low = torch.cuda.Stream(priority=lo)
    x = (torch.randn(A, T, D, device="cuda", dtype=torch.float32) * 0.02).to(torch.bfloat16)
    n_graph_steps = 8

    def gemm_step(l):
        wg = slab[l, 0, :A].view(A, D, F)
        wu = slab[l, 1, :A].view(A, D, F)
        wd = slab[l, 2, :A].view(A, F, D)
        h = torch.bmm(x, wg) * torch.bmm(x, wu)
        return torch.bmm(h, wd)

    with torch.cuda.stream(s_main):
        for l in range(3):
            gemm_step(l)
        s_main.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=s_main):
            for i in range(n_graph_steps):
                gemm_step(i % L)
    torch.cuda.synchronize()

    def gemm_loop(n_replays):
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(n_replays + 1)]
        with torch.cuda.stream(s_main):
            evs[0].record(s_main)
            for i in range(n_replays):
                graph.replay()
                evs[i + 1].record(s_main)
        return evs

    # victim alone
    evs = gemm_loop(40)
    torch.cuda.synchronize()
    alone_us = statistics.median(evs[i].elapsed_time(evs[i + 1]) for i in range(5, 40)) \
        / n_graph_steps * 1e3
    moved = sum(plan.stats(ph)["bytes_moved"] for ph in range(3))
    out = {"victim": "torch.bmm grouped expert GEMM, %d experts x %d tokens, d_model %d, d_ff %d"
                     % (A, T, D, F), "victim_alone_us_per_step": round(alone_us, 2), "runs": []}
    for budget in budgets:
        plan.set_tuning(max_ctas=budget)
        # reshard alone on the low-priority stream
        r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        one_step(plan, src, dst, s_low); s_low.synchronize()
        r0.record(s_low); one_step(plan, src, dst, s_low); r1.record(s_low); s_low.synchronize()
        alone_ms = r0.elapsed_time(r1)
        # overlapped: enough victim replays to cover the reshard
        n_rep = int(alone_ms * 1e3 / (alone_us * n_graph_steps) * 2.5) + 20
        torch.cuda.synchronize()
        r0.record(s_low)
        one_step(plan, src, dst, s_low)
        r1.record(s_low)
        evs = gemm_loop(n_rep)
        torch.cuda.synchronize()
        both_ms = r0.elapsed_time(r1)
        # victim replays that ended while the reshard was still running
        t_end = both_ms
        inside = [evs[i].elapsed_time(evs[i + 1]) for i in range(n_rep)
                  if r0.elapsed_time(evs[i + 1]) < t_end and r0.elapsed_time(evs[i]) > 0]
        during_us = (statistics.mean(inside) / n_graph_steps * 1e3) if inside else None
        out["runs"].append({
            "max_ctas": budget or "default",
            "reshard_alone_ms": round(alone_ms, 3),
            "reshard_alone_gbs": round(2 * moved / alone_ms / 1e6, 1),
            "reshard_overlapped_ms": round(both_ms, 3),
            "reshard_overlapped_gbs": round(2 * moved / both_ms / 1e6, 1),
            "victim_us_per_step_during": round(during_us, 2) if during_us else None,
            "victim_slowdown": round(during_us / alone_us, 3) if during_us else None,
            "victim_replays_inside": len(inside)})
    plan.set_tuning()
    return out


# ---- paged expert store: the expert phase as a page re-map plus copies of arrivals -------

def run_vmm(torch, E, wl, copy_all_ms):
    """Times emoe_vmm_reshard for the workload's expert placements (old -> new) on a pool of
    uninitialised pages (byte movement does not depend on values) and sets it beside the
    dense copy-everything expert phase.  Host wall-clock: the call is synchronous."""
    torch.cuda.empty_cache()
    try:
        with E.VmmPool(wl.shape, wl.old.placement) as pool:
            torch.cuda.synchronize()
            st = pool.reshard(wl.new.placement)
    except E.EmoeError as e:
        return {"error": str(e)}
    out = {k: (round(v, 3) if isinstance(v, float) else v) for k, v in st.items()}
    out["copy_gbs"] = round((st["bytes_copied"] + st["bytes_read"]) / st["copy_ms"] / 1e6, 1) \
        if st["copy_ms"] > 0 and st["bytes_copied"] else None
    out["dense_copy_all_ms"] = round(copy_all_ms, 3)
    out["padding_overhead"] = round(st["slab_bytes"] / st["matrix_bytes"] - 1, 4)
    return out


# ---- reference arm: the oracle on the host cores -----------------------------------------

def run_reference(args):
    import workloads as W
    from workloads import device as WD
    import oracle
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = W.make_workload(args.workload)
    wl1 = wl.with_layers(1)
    sizes_old = [oracle.expert_arena_bytes(wl1.shape, wl.old.placement),
                 oracle.attn_arena_bytes(wl1.shape, wl.old.tp),
                 oracle.kv_arena_bytes(wl1.shape, wl.old.tp, wl.old.kv_num_blocks)]
    getter = host_layer_getter(wl, W, WD, sizes_old)
    cache = {}
    def cached(l):
        if l not in cache:
            cache.clear()
            cache[l] = getter(l)
        return cache[l]
    vals = []
    for i in range(args.warmup + args.steps):
        r = cpu_baseline_sample(wl, lambda l: cached(0), budget_s=0.0, max_layers=1)
        if i >= args.warmup:
            vals.append(r)
    gbs = statistics.mean(v["value"] for v in vals)
    ms = statistics.mean(v["ms_per_layer"] for v in vals)
    line = {"impl": "reference", "metric": METRIC, "value": round(gbs, 3), "unit": UNIT,
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": round(ms, 3), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "u8", "data": "synthetic",
            "config": {"workload": wl.name, "reconfig": wl.notes,
                       "sample": "each step = layer 0 of %d, all three phases" % wl.shape.n_layers},
            "cpu_baseline": {"value": round(gbs, 3), "unit": UNIT, "cores": 1, "kind": "oracle",
                             "sample": "one full layer of %s per step, single thread" % wl.name},
            "e2e": {"value": round(gbs, 3), "unit": UNIT, "h2d_bytes_per_step": 0,
                    "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ---- main --------------------------------------------------------------------------------

def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="c2_mid")
    ap.add_argument("--impl", default="emoe", choices=["emoe", "reference"])
    ap.add_argument("--only-main", action="store_true",
                    help="skip the other configs, the overlap case, e2e and the CPU baseline")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--layers", type=int, default=None,
                    help="cut the workload to this many layers (for small profiler captures "
                         "only: the result is then not the named configuration)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "emoe" else args.warmup

    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import paper_2510_02613_b200 as E
    from paper_2510_02613_b200 import replicas
    import workloads as W
    from workloads import device as WD

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the re-layout has no CPU path")
    local = local % torch.cuda.device_count()
    torch.cuda.set_device(local)
    dist = None
    # control plane only (barrier, max of the step times): NCCL, or gloo when several ranks
    # have to share one GPU (EMOE_BENCH_BACKEND=gloo, for checking the N > 1 flow on one device)
    backend = os.environ.get("EMOE_BENCH_BACKEND", "nccl")
    if world > 1:
        import torch.distributed as dist
        if backend == "nccl":
            dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        else:
            dist.init_process_group(backend)
    barrier = (lambda: dist.barrier()) if dist else None
    peak, peak_kind = measured_peak()
    stream = torch.cuda.Stream()

    tiny = W.make_workload("c1_tiny")        # loads the CUDA module, so that plan times below are the planner's
    E.Plan(tiny.shape, tiny.old, tiny.new).close()
    wl, plan, src, dst, plan_ms = setup(args.workload, torch, E, W, WD, n_layers=args.layers)
    sampler = ClockSampler(local)
    sampler.start()
    total_ms = time_steps(torch, plan, src, dst, args.steps, args.warmup, stream, barrier)
    clocks = sampler.stop()
    phase_ms = time_phases(torch, plan, src, dst, max(3, min(args.steps, 20)), stream)
    total_ms = replicas.job_time_ms(total_ms, dist, device="cuda" if backend == "nccl" else "cpu")  # max over ranks
    rep = config_report(E, plan, wl, total_ms, phase_ms, args.steps, peak, plan_ms)
    if plan.device_status() != 0:
        raise SystemExit("device status word set: a bounded wait expired")
    ms = total_ms / args.steps
    value = replicas.job_throughput_gbs(rep["bytes_moved"], world, ms)
    per_step = plan.num_launches(E.PHASE_STEP)
    launches = per_step * args.steps

    # roofline of the dominant kernel, the bulk-copy launch.  When the whole step is that one
    # launch (TP kept: every segment of every phase is a long run), its duration is the step
    # time of the timed region; otherwise the expert phase run on its own stands in.
    st_all = [plan.stats(ph) for ph in range(3)]
    if per_step == 1:
        alg_bytes = sum(x["bytes_moved"] + x["bytes_read"] for x in st_all)
        launch_ms, what = ms, "bulk_copy_kernel (whole step: experts + attention + KV in one launch)"
    else:
        alg_bytes = st_all[0]["bytes_moved"] + st_all[0]["bytes_read"]
        small = alg_bytes < (512 << 20)     # small phases are routed to the vector kernel whole
        launch_ms = phase_ms[0]
        what = ("vec_copy_kernel" if small else "bulk_copy_kernel") + " (expert re-pack, timed as its own call)"
    achieved = alg_bytes / (launch_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": what,
                "achieved": round(achieved, 1), "peak": peak, "peak_kind": "of " + peak_kind,
                "unit": UNIT, "frac": round(achieved / peak, 4),
                "algorithmic_bytes_per_launch": alg_bytes,
                "launch_ms": round(launch_ms, 4),
                "traffic": NCU_TRAFFIC.get(wl.name) if per_step == 1 and args.layers is None else None}

    line = {"metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(ms, 4),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u8",
            "data": "synthetic",
            "config": {"workload": wl.name if args.layers is None
                       else "%s cut to %d layers" % (wl.name, args.layers),
                       "reconfig": wl.notes, "parallelism": "replicas",
                       "l2": "inputs_larger_than_l2", "value_convention": "2 x bytes moved / time",
                       "scale_step_ms": rep["scale_step_ms"],
                       "pct_of_nominal_8000": rep["pct_of_nominal_8000"],
                       "pct_of_measured_peak": rep["pct_of_measured_peak"]},
            "clocks": clocks, "gpu_launches": launches, "roofline": roofline,
            "phases": rep["phases"], "planner_ms": rep["planner_ms"]}

    if rank == 0 and not args.only_main:
        # e2e on host buffers (the whole workload; needs it twice in pinned host memory)
        try:
            import psutil
            need = sum(t.numel() for g in src + dst for t in g)
            if psutil.virtual_memory().available < need * 1.15:
                raise MemoryError("host has %.0f GB available, the step needs %.0f GB pinned"
                                  % (psutil.virtual_memory().available / 1e9, need / 1e9))
            with E.Plan(wl.shape, wl.old, wl.new, host_step=True) as e2e_plan:   # pipelined form
                e_ms, h2d, d2h = run_e2e(torch, e2e_plan, src, dst, args.e2e_steps, stream)
            line["e2e"] = {"value": round(2 * rep["bytes_moved"] / (e_ms * 1e-3) / 1e9, 2),
                           "unit": UNIT, "ms_per_step": round(e_ms, 2), "steps": args.e2e_steps,
                           "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}
        except Exception as e:  # report, never hide
            line["e2e"] = {"value": None, "unit": UNIT, "error": repr(e)[:200]}
        # CPU baseline: the oracle on sampled layers of the same arenas
        getter = device_layer_getter(torch, src, wl.shape.n_layers)
        line["cpu_baseline"] = cpu_baseline_sample(wl, getter)
        try:
            line["cpu_baseline_all_cores"] = cpu_baseline_all_cores(wl, getter)
        except Exception as e:  # report, never hide
            line["cpu_baseline_all_cores"] = {"value": None, "error": repr(e)[:200]}
    elif world > 1:
        line["e2e"] = {"value": None, "unit": UNIT, "note": "measured at --gpus 1 only"}

    del src, dst
    plan.close()
    torch.cuda.empty_cache()
    if rank == 0 and not args.only_main:
        rep["vmm_expert_step"] = run_vmm(torch, E, wl, rep["phases"]["experts"]["ms"])

    if not args.only_main and world == 1:
        others = {}
        for name in W.WORKLOAD_NAMES:
            if name == args.workload:
                others[name] = rep
                continue
            wl2, plan2, src2, dst2, pms = setup(name, torch, E, W, WD)
            k = max(5, args.steps // 2) if name != "c1_tiny" else 200
            tot = time_steps(torch, plan2, src2, dst2, k, 3, stream)
            ph = time_phases(torch, plan2, src2, dst2, max(3, min(k, 20)), stream)
            r = config_report(E, plan2, wl2, tot, ph, k, peak, pms)
            if name == "c1_tiny":    # launch-bound: also as a CUDA-graph replay
                g_ms = time_graph_steps(torch, plan2, src2, dst2, k, 3, stream)
                r["cuda_graph"] = {"scale_step_ms": round(g_ms, 4),
                                   "reshard_gbs": round(2 * r["bytes_moved"] / g_ms / 1e6, 1)}
            if name == "c5_overlap":
                r["overlap"] = run_overlap(torch, E, plan2, wl2, src2, dst2, peak)
            others[name] = r
            del src2, dst2
            plan2.close()
            torch.cuda.empty_cache()
            if name != "c5_overlap":
                r["vmm_expert_step"] = run_vmm(torch, E, wl2, r["phases"]["experts"]["ms"])
        line["configs"] = others

    if dist:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(line))


if __name__ == "__main__":
    main()
