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
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "traffic.json")
KERNEL_SOURCES = [os.path.join(ROOT, "paper_2510_02613_b200", "csrc", f)
                  for f in ("kernels.cu", "kernels.h", "capi.cpp", "planner.cpp", "planner.h")]


def kernel_sources_sha() -> str:
    import hashlib
    h = hashlib.sha256()
    for f in KERNEL_SOURCES:
        with open(f, "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def load_traffic():
    """DRAM bytes per kernel from the ncu captures recorded in profiles/traffic.json (small
    cuts of the workloads; see --record-traffic).  Returns {} when the kernel sources have
    changed since the counters were taken: stale counters are not reported."""
    try:
        with open(TRAFFIC_FILE) as f:
            t = json.load(f)
    except Exception:
        return {}
    if t.get("kernel_sources_sha256") != kernel_sources_sha():
        return {}
    return t.get("captures", {})


def traffic_split(traffic, wl_name, kernel, full_layers):
    """(read, written) DRAM bytes of one launch of `kernel` at full size (kernel None: of all
    kernels of one step), or None: the capture's bytes scaled by layers (every layer has
    identical units, so traffic grows in proportion)."""
    cap = traffic.get({"c5_overlap": "c3_fine"}.get(wl_name, wl_name))   # the overlap case runs the c3 reshard
    if not cap:
        return None
    ks = cap.get("kernels", {})
    if kernel is not None and kernel not in ks:
        ks = cap.get("phase_kernels", {})       # a kernel that only the per-phase entry points launch
    pick = list(ks.values()) if kernel is None else [ks[kernel]] if kernel in ks else []
    if not pick:
        return None
    scale = full_layers / cap["layers"]
    rd = sum(k["dram_bytes_read"] / max(k["launches"], 1) for k in pick)
    wr = sum(k["dram_bytes_write"] / max(k["launches"], 1) for k in pick)
    return int(rd * scale), int(wr * scale)


def traffic_per_launch(traffic, wl_name, kernel, full_layers):
    """Read + written DRAM bytes of one launch (see traffic_split), or None."""
    t = traffic_split(traffic, wl_name, kernel, full_layers)
    return None if t is None else t[0] + t[1]


def record_traffic(args):
    """Parses an `ncu --page raw --csv` dump of a capture of `bench.py --only-main --workload W
    --layers N` and stores the kernels' DRAM byte counters in profiles/traffic.json."""
    import csv
    rows = list(csv.reader(open(args.record_traffic, newline="")))
    head = next(i for i, r in enumerate(rows) if "Kernel Name" in r)
    cols = {n: i for i, n in enumerate(rows[head])}
    units = rows[head + 1]
    scale = {"byte": 1, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9, "Tbyte": 1e12}
    kernels = {}
    for r in rows[head + 2:]:
        if len(r) <= cols["Kernel Name"]:
            continue
        name = r[cols["Kernel Name"]].split("(")[0].split("<")[0].split("::")[-1].strip()
        k = kernels.setdefault(name, {"launches": 0, "dram_bytes_read": 0.0, "dram_bytes_write": 0.0,
                                      "duration_us": 0.0})
        k["launches"] += 1
        for key, col in (("dram_bytes_read", "dram__bytes_read.sum"), ("dram_bytes_write", "dram__bytes_write.sum")):
            k[key] += float(r[cols[col]].replace(",", "")) * scale[units[cols[col]]]
        if "gpu__time_duration.sum" in cols:
            c = cols["gpu__time_duration.sum"]
            k["duration_us"] += float(r[c].replace(",", "")) * {"ns": 1e-3, "us": 1, "ms": 1e3, "s": 1e6}.get(units[c], 1)
    try:
        with open(TRAFFIC_FILE) as f:
            t = json.load(f)
    except Exception:
        t = {}
    sha = kernel_sources_sha()
    if t.get("kernel_sources_sha256") != sha:
        t = {"kernel_sources_sha256": sha, "captures": {}}
    t["note"] = ("DRAM counters (dram__bytes_read.sum / dram__bytes_write.sum, summed over the captured "
                 "launches) of small cuts of the workloads; bench.py scales them by layers and drops them "
                 "when the kernel sources no longer hash to kernel_sources_sha256")
    new = {n: {k: (int(v) if k != "duration_us" else round(v, 1)) for k, v in d.items()}
           for n, d in kernels.items()}
    old = t["captures"].get(args.workload)
    if args.traffic_merge and old and old.get("layers") == args.layers:
        # kernels of the per-phase entry points, captured apart from the whole-step kernels
        old.setdefault("phase_kernels", {}).update(new)
        old["phase_command"] = args.traffic_command or ""
    else:
        t["captures"][args.workload] = {"layers": args.layers, "command": args.traffic_command or "",
                                        "kernels": new}
    with open(TRAFFIC_FILE, "w") as f:
        json.dump(t, f, indent=1, sort_keys=True)
        f.write("\n")
    print(json.dumps(t["captures"][args.workload]))


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


def time_steps(torch, plan, src, dst, steps, warmup, stream, barrier=None, per_step=True):
    """(total ms over `steps` whole steps, per-step ms list).  The steps run back to back
    (emoe_reshard_step) between two events on the stream the kernels are launched on; with
    per_step an event is also recorded between consecutive steps, so that the spread over
    the region can be reported (median / min / max) beside the mean the total gives."""
    torch.cuda.synchronize()   # the arenas were filled on the default stream
    with torch.cuda.stream(stream):
        for _ in range(warmup):
            one_step(plan, src, dst, stream)
        stream.synchronize()
        if barrier:
            barrier()
        torch.cuda.synchronize()
        n_ev = steps + 1 if per_step else 2
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(n_ev)]
        ev[0].record(stream)
        for i in range(steps):
            one_step(plan, src, dst, stream)
            if per_step or i == steps - 1:
                ev[i + 1 if per_step else 1].record(stream)
        stream.synchronize()
        torch.cuda.synchronize()
    each = [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)] if per_step else []
    return ev[0].elapsed_time(ev[-1]), each


def step_spread(each):
    if not each:
        return None
    return {"median_ms": round(statistics.median(each), 4), "min_ms": round(min(each), 4),
            "max_ms": round(max(each), 4), "n": len(each)}


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


KERNEL_OF = {"ring_units": "bulk_copy_kernel", "vector_units": "vec_copy_kernel", "kv_tiles": "kv_rows_kernel"}


def kernels_of(work):
    """Names of the kernels a launch set consists of, from emoe_plan_launch_work."""
    return [KERNEL_OF[k] for k in ("ring_units", "vector_units", "kv_tiles") if work[k]]


def roofline_block(kernel, alg_bytes, ms, peak, peak_kind, traffic):
    achieved = alg_bytes / (ms * 1e-3) / 1e9
    return {"bound": "hbm", "kernel": kernel, "achieved": round(achieved, 1), "peak": peak,
            "peak_kind": "of " + peak_kind, "unit": UNIT, "frac": round(achieved / peak, 4),
            "frac_of_nominal_8000": round(achieved / NOMINAL_HBM_GBS, 4),
            "algorithmic_bytes_per_launch": alg_bytes, "launch_ms": round(ms, 4), "traffic": traffic}


def config_rooflines(E, plan, wl, step_ms, phase_ms, peak, peak_kind, traffic, full_layers, cut):
    """One roofline block for the whole step and one per kernel.  Algorithmic bytes of a launch =
    bytes_read + bytes_moved of what it covers (a source that feeds k destinations is read
    once).  A kernel's duration: the step's, when the step is that one launch; otherwise the
    phase that consists of that kernel alone, run through its own entry point (in a step the
    launch sets overlap, so their durations cannot be told apart there)."""
    st = [plan.stats(ph) for ph in range(3)]
    alg = [x["bytes_moved"] + x["bytes_read"] for x in st]
    work = plan.launch_work(E.PHASE_STEP)
    names = kernels_of(work)
    fused = plan.num_launches(E.PHASE_STEP) < len(names)     # vector work and KV tiles share a kernel
    tr = (lambda k: None) if cut else (lambda k: traffic_per_launch(traffic, wl.name, k, full_layers))
    out = {"step": roofline_block(" + ".join(names) + (" (vector and KV work in one kernel)" if fused else ""),
                                  sum(alg), step_ms, peak, peak_kind, tr(None)),
           "kernels": []}
    # read and written bytes apart: a source that feeds several destinations must show up once
    out["step"]["algorithmic_bytes_read"] = sum(x["bytes_read"] for x in st)
    out["step"]["algorithmic_bytes_written"] = sum(x["bytes_moved"] for x in st)
    split = None if cut else traffic_split(traffic, wl.name, None, full_layers)
    out["step"]["traffic_read"], out["step"]["traffic_written"] = split if split else (None, None)
    if len(names) == 1:
        out["kernels"].append(dict(out["step"], kernel=names[0], timed_as="the whole step (one launch)"))
        return out
    for ph, pname in enumerate(("experts", "attn", "kv")):
        w = plan.launch_work(ph)
        k = kernels_of(w)
        if len(k) != 1 or phase_ms[ph] <= 0:
            continue
        # the ring kernel's capture is the whole step's launch: it stands for a phase only if
        # that phase is all the ring work of the step
        same = k[0] != "bulk_copy_kernel" or work["ring_units"] == w["ring_units"]
        b = roofline_block(k[0], alg[ph], phase_ms[ph], peak, peak_kind, tr(k[0]) if same else None)
        b["timed_as"] = "the %s phase through its own entry point" % pname
        out["kernels"].append(b)
    return out


def config_report(E, plan, wl, total_ms, each, phase_ms, steps, peak, peak_kind, plan_ms, traffic,
                  cut=False):
    st = [plan.stats(ph) for ph in range(3)]
    moved = sum(s["bytes_moved"] for s in st)
    read = sum(s["bytes_read"] for s in st)
    ms = total_ms / steps
    gbs = 2 * moved / (ms * 1e-3) / 1e9
    names = ["experts", "attn", "kv"]
    return {
        "workload": wl.name, "reconfig": wl.notes, "bytes_moved": moved, "bytes_read": read,
        "scale_step_ms": round(ms, 4), "step_spread": step_spread(each), "reshard_gbs": round(gbs, 1),
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
        "roofline": config_rooflines(E, plan, wl, ms, phase_ms, peak, peak_kind, traffic,
                                     wl.shape.n_layers, cut),
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
    return ms, h2d, d2h, host_link_rates(torch, h_src, h_dst, src, dst)


def host_link_rates(torch, h_src, h_dst, src, dst):
    """The yardstick for the end-to-end number: plain pinned copies of the largest old arena
    host->device and the largest new arena device->host, on two streams at once (no kernel in
    between), GB/s per direction while both run."""
    hs, ds = max(((h, d) for hg, dg in zip(h_src, src) for h, d in zip(hg, dg)), key=lambda x: x[0].numel())
    hd, dd = max(((h, d) for hg, dg in zip(h_dst, dst) for h, d in zip(hg, dg)), key=lambda x: x[0].numel())
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    reps = 3
    torch.cuda.synchronize()
    for timed in (False, True):
        with torch.cuda.stream(s_in):
            ev[0].record()
            for _ in range(reps if timed else 1):
                ds.copy_(hs, non_blocking=True)
            ev[1].record()
        with torch.cuda.stream(s_out):
            ev[2].record()
            for _ in range(reps if timed else 1):
                hd.copy_(dd, non_blocking=True)
            ev[3].record()
        torch.cuda.synchronize()
    return {"h2d_gbs": round(reps * hs.numel() / (ev[0].elapsed_time(ev[1]) * 1e-3) / 1e9, 2),
            "d2h_gbs": round(reps * hd.numel() / (ev[2].elapsed_time(ev[3]) * 1e-3) / 1e9, 2),
            "bytes_each_way": [hs.numel(), hd.numel()], "how": "pinned copies both ways at once, no kernel"}


# ---- C5: reshard on a low-priority stream beside a grouped expert GEMM -------------------

OVERLAP_POINTS = (
    dict(), dict(max_ctas=96), dict(max_ctas=48), dict(max_ctas=24), dict(max_ctas=16), dict(max_ctas=8),
    dict(max_ctas=4), dict(bw_limit_gbs=5500), dict(bw_limit_gbs=4500), dict(bw_limit_gbs=3500),
    dict(bw_limit_gbs=2500), dict(bw_limit_gbs=1500), dict(bw_limit_gbs=3500, bulk_hints=2),
    dict(max_ctas=37, bw_limit_gbs=3000), dict(max_ctas=24, bulk_stages=2), dict(max_ctas=16, bw_limit_gbs=1000),
    dict(max_ctas=1000000, bulk_tile_bytes=16384, bulk_stages=12),   # one short-lived CTA per unit
    dict(path=3),                                                    # driver copies on the copy engines: no SM taken
)


def run_overlap(torch, E, plan, wl, src, dst, peak, victim, points=OVERLAP_POINTS, verify=True):
    """Victim: 8 active experts x 256 tokens (top-8 routing: every active expert sees all
    tokens), gate/up/down bf16 batched GEMMs (torch.bmm, a measurement fixture, not part
    of the library) on a high-priority stream, CUDA-graph replayed; the reshard runs on a
    least-priority stream.  Weights are taken from the old expert arena of rank 0 when the
    shapes agree (the layer cycling per step), else from a buffer of their own.  Every
    point of `points` is one launch tuning: the trade-off curve victim slowdown against
    reshard bandwidth."""
    v = victim
    A, T, D, F = v["active_experts"], v["tokens"], v["d_model"], v["d_ff"]
    L = wl.shape.n_layers
    if D == wl.shape.d_model and F == wl.shape.d_ff and len(wl.old.placement[0]) >= A:
        slab = src[0][0].view(torch.bfloat16).view(L, 3, len(wl.old.placement[0]), D * F)
        n_l = L
    else:
        n_l = 4        # 4 x 138 MB of weights: larger than L2
        slab = (torch.randn(n_l, 3, A, D * F, device="cuda", dtype=torch.float32) * 0.02).to(torch.bfloat16)
    least, greatest = torch.cuda.Stream.priority_range()
    s_main = torch.cuda.Stream(priority=greatest)
    s_low = torch.cuda.Stream(priority=least)
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
            gemm_step(l % n_l)
        s_main.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=s_main):
            for i in range(n_graph_steps):
                gemm_step(i % n_l)
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
    st = [plan.stats(ph) for ph in range(3)]
    moved = sum(x_["bytes_moved"] for x_ in st)
    alg = sum(x_["bytes_moved"] + x_["bytes_read"] for x_ in st)
    weight_bytes = 3 * A * D * F * 2
    victim_gbs = weight_bytes / alone_us / 1e3
    out = {"victim": "torch.bmm grouped expert GEMM, %d experts x %d tokens, d_model %d, d_ff %d"
                     % (A, T, D, F), "victim_alone_us_per_step": round(alone_us, 2),
           "victim_weight_bytes_per_step": weight_bytes, "victim_alone_gbs": round(victim_gbs, 1),
           "runs": []}
    hbm_total = None
    for tuning in points:
        plan.set_tuning(**tuning)
        # reshard alone on the low-priority stream
        r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        one_step(plan, src, dst, s_low); s_low.synchronize()
        r0.record(s_low); one_step(plan, src, dst, s_low); r1.record(s_low); s_low.synchronize()
        alone_ms = r0.elapsed_time(r1)
        if hbm_total is None:
            hbm_total = alg / alone_ms / 1e6       # what the unconstrained reshard gets out of HBM
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
        inside = [evs[i].elapsed_time(evs[i + 1]) for i in range(n_rep)
                  if r0.elapsed_time(evs[i + 1]) < both_ms and r0.elapsed_time(evs[i]) > 0]
        during_us = (statistics.mean(inside) / n_graph_steps * 1e3) if inside else None
        alg_gbs = alg / both_ms / 1e6
        # if the two only competed for HBM bytes, the victim would keep what the reshard leaves
        left = max(hbm_total - alg_gbs, 1.0)
        out["runs"].append({
            "tuning": tuning or "default",
            "reshard_alone_ms": round(alone_ms, 3),
            "reshard_alone_gbs": round(2 * moved / alone_ms / 1e6, 1),
            "reshard_overlapped_ms": round(both_ms, 3),
            "reshard_overlapped_gbs": round(2 * moved / both_ms / 1e6, 1),
            "reshard_overlapped_hbm_gbs": round(alg_gbs, 1),
            "victim_us_per_step_during": round(during_us, 2) if during_us else None,
            "victim_slowdown": round(during_us / alone_us, 3) if during_us else None,
            "slowdown_if_only_hbm_bytes_were_shared": round(max(1.0, victim_gbs / left), 3),
            "victim_replays_inside": len(inside)})
    out["hbm_gbs_of_unconstrained_reshard"] = round(hbm_total, 1)
    ok = [r for r in out["runs"] if r["victim_slowdown"] and r["victim_slowdown"] <= 1.5]
    best = max(ok, key=lambda r: r["reshard_overlapped_gbs"]) if ok else None
    out["best_with_victim_within_1p5x"] = ({"tuning": best["tuning"], "victim_slowdown": best["victim_slowdown"],
                                            "reshard_overlapped_gbs": best["reshard_overlapped_gbs"]}
                                           if best else None)
    plan.set_tuning()
    if verify:
        # harness check, outside every timed part: layer 0 of what the LAST overlapped run wrote,
        # against the CPU oracle run on that layer alone (layers are independent)
        out["overlapped_output_matches_oracle_layer0"] = verify_layer(torch, E, plan, wl, src, dst, 0)
    return out


def verify_layer(torch, E, plan, wl, src, dst, layer):
    import oracle
    wl1 = wl.with_layers(1)
    L = wl.shape.n_layers
    ok = True
    for ph in range(3):
        h_src = [t[layer * (t.numel() // L):(layer + 1) * (t.numel() // L)].cpu().numpy() for t in src[ph]]
        got = [t[layer * (t.numel() // L):(layer + 1) * (t.numel() // L)].cpu().numpy() for t in dst[ph]]
        want = [g.copy() for g in got]       # bytes the step does not write must stay as they are
        if ph == 0:
            oracle.reshard_experts(wl1.shape, wl.old.placement, wl.new.placement, h_src, want)
        elif ph == 1:
            oracle.reshard_attn(wl1.shape, wl.old.tp, wl.new.tp, h_src, want)
        else:
            oracle.reshard_kv(wl1.shape, wl.old, wl.new, h_src, want)
        ok = ok and all(np.array_equal(g, w) for g, w in zip(got, want))
    return bool(ok)


# ---- KV phase into a compacting (identity-order) new table --------------------------------

def run_kv_compacting(torch, E, W, WD, name, random_ms, reps=30):
    """The KV phase of the workload once more, with the new block table COMPACTING the pool
    (emoe_kv_compact_table: mapped blocks get the destination ids 0, 1, 2, ...) instead of a
    random permutation - as a scale-down that packs the surviving pool would choose: once with
    the ids handed out in table order, once in the order of the blocks' old physical ids, so
    that the migration writes the new pool in address order as it reads the old one."""
    import dataclasses
    wl = W.make_workload(name)
    B = wl.shape.kv_block_tokens
    out = {"random_new_table_ms": round(random_ms, 4)}
    stream = torch.cuda.Stream()
    for label, old_table in (("table_order", None), ("old_address_order", wl.old.block_table)):
        table = E.kv_compact_table(B, wl.old.seq_lens, wl.new.kv_num_blocks, old_table=old_table)
        w2 = dataclasses.replace(wl, new=dataclasses.replace(wl.new, block_table=table))
        with E.Plan(w2.shape, w2.old, w2.new) as plan:
            src = WD.alloc_filled(plan.arena_bytes(E.PHASE_KV, E.SIDE_OLD), w2.seed, W.KIND_KV)
            dst = WD.alloc_const(plan.arena_bytes(E.PHASE_KV, E.SIDE_NEW))
            torch.cuda.synchronize()
            for _ in range(3):
                plan.reshard_kv(src, dst, stream)
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1)]
            ev[0].record(stream)
            for i in range(reps):
                plan.reshard_kv(src, dst, stream)
                ev[i + 1].record(stream)
            stream.synchronize()
            ms = statistics.median(ev[i].elapsed_time(ev[i + 1]) for i in range(reps))
            st = plan.stats(E.PHASE_KV)
            out[label] = {"ms": round(ms, 4), "gbs": round(2 * st["bytes_moved"] / ms / 1e6, 1),
                          "device_status_ok": plan.device_status() == 0}
        del src, dst
        torch.cuda.empty_cache()
    return out


# ---- in-place expert step: only arrivals move ---------------------------------------------

def run_inplace(torch, E, wl, copy_all_ms, peak, reps=30):
    """The expert phase as the paper runs it - what a device already holds stays where it is,
    only arrivals are copied - on dense arenas with spare slots (emoe_plan_create_inplace),
    beside the copy-everything expert phase of the same reconfiguration.  Two wanted
    placements: the workload's own, and (when every expert is held once) the balanced
    placement that keeps the most experts in place.  Arena contents are left uninitialised:
    byte movement does not depend on values."""
    m_bytes = wl.shape.d_model * wl.shape.d_ff * wl.shape.elem_bytes * wl.shape.n_layers * 3
    out = {"dense_copy_all_ms": round(copy_all_ms, 4),
           # device memory an expert step needs while it runs: copy-all holds the old AND the new arenas
           "dense_copy_all_peak_bytes": m_bytes * (sum(len(p) for p in wl.old.placement)
                                                   + sum(len(p) for p in wl.new.placement)),
           "variants": []}
    held_once = all(sum(e in p for p in wl.old.placement) == 1 for e in range(wl.shape.n_experts))
    wants = [("workload placement", [list(p) for p in wl.new.placement])]
    if held_once:
        wants.append(("placement that keeps the most experts in place",
                      E.place_min_transfer(wl.shape.n_experts, wl.old.placement, wl.new.ep)[0]))
    stream = torch.cuda.Stream()
    m = wl.shape.d_model * wl.shape.d_ff * wl.shape.elem_bytes
    for label, want in wants:
        old = []
        for r, p in enumerate(wl.old.placement):
            arrivals = len([e for e in want[r] if e not in p]) if r < len(want) else 0
            old.append(list(p) + [-1] * arrivals)
        cap_new = [len(t) for t in old][:len(want)] + [len(want[r]) for r in range(len(old), len(want))]
        try:
            with E.InplacePlan(wl.shape, old, want, cap_new) as plan:
                arenas = [torch.empty(wl.shape.n_layers * 3 * c * m, dtype=torch.uint8, device="cuda")
                          for c in plan.caps]
                torch.cuda.synchronize()
                st = plan.stats(E.PHASE_EXPERTS)
                for _ in range(3):
                    plan.reshard(arenas, stream)
                ev = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1)]
                ev[0].record(stream)
                for i in range(reps):
                    plan.reshard(arenas, stream)
                    ev[i + 1].record(stream)
                stream.synchronize()
                each = [ev[i].elapsed_time(ev[i + 1]) for i in range(reps)]
                ms = statistics.median(each)
                ok = plan.device_status() == 0
                del arenas
        except E.EmoeError as e:
            out["variants"].append({"wanted": label, "error": str(e)})
            continue
        torch.cuda.empty_cache()
        alg = st["bytes_moved"] + st["bytes_read"]
        out["variants"].append({
            "wanted": label, "experts_kept_in_place": sum(len(set(want[r]) & set(wl.old.placement[r]))
                                                          for r in range(min(len(want), wl.old.ep))),
            "expert_slots_wanted": sum(len(w) for w in want),
            "bytes_moved": st["bytes_moved"], "peak_bytes": m_bytes * sum(plan.caps),
            "ms": round(ms, 4), "min_ms": round(min(each), 4),
            "reshard_gbs": round(2 * st["bytes_moved"] / ms / 1e6, 1),
            "hbm_gbs": round(alg / ms / 1e6, 1), "frac_of_measured_peak": round(alg / ms / 1e6 / peak, 4),
            "speedup_over_copy_all": round(copy_all_ms / ms, 2), "device_status_ok": ok})
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


def run_vmm_slots(torch, E, wl, copy_all_ms):
    """The paged store with slot tables (ranges kept across steps, only changed slots mapped,
    copied or unmapped, arrivals served from pages created beforehand) on the workload's
    expert placements, on uninitialised pages.  Host wall-clock of the synchronous call."""
    torch.cuda.empty_cache()
    want = [list(p) for p in wl.new.placement]
    old, arrivals = [], 0
    for r, p in enumerate(wl.old.placement):
        k = len([e for e in want[r] if e not in p]) if r < len(want) else 0
        old.append(list(p) + [-1] * k)
    cap_new = [len(t) for t in old][:len(want)] + [len(want[r]) for r in range(len(old), len(want))]
    arrivals = sum(len([e for e in w if r >= len(wl.old.placement) or e not in wl.old.placement[r]])
                   for r, w in enumerate(want))
    try:
        with E.VmmSlots(wl.shape, old, spare_slots=arrivals) as pool:
            torch.cuda.synchronize()
            st = pool.reshard(want, cap_new)
            back = pool.reshard([list(p) for p in wl.old.placement], [len(t) for t in old])  # and down again
    except E.EmoeError as e:
        return {"error": str(e)}
    out = {k: (round(v, 3) if isinstance(v, float) else v) for k, v in st.items()}
    out["step_back_total_ms"] = round(back["total_ms"], 3)
    out["step_back_alloc_ms"] = round(back["alloc_ms"], 3)
    out["dense_copy_all_ms"] = round(copy_all_ms, 3)
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


# ---- exchange mode: one rank per GPU, the step as a pull over the interconnect -----------

def run_exchange(args):
    """bench.py --gpus N --mode exchange (under torchrun): rank = GPU.  Every process owns the
    old and the new arenas of its rank index, builds the same plan, restricts it to its own
    destination rank and PULLS what it needs from its peers' old arenas through CUDA IPC
    mappings - the library's own kernels reading peer memory (plain loads and bulk copies that
    every CTA issues for itself); torch.distributed carries handles, barriers and the max of the step times only.
    value = 2 x bytes all ranks wrote / slowest rank's time."""
    import torch
    import torch.distributed as dist
    import paper_2510_02613_b200 as E
    from paper_2510_02613_b200 import exchange, replicas
    import workloads as W
    from workloads import device as WD

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world < 2:
        raise SystemExit("--mode exchange needs at least two ranks (torchrun --nproc-per-node N)")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the re-layout has no CPU path")
    local = local % torch.cuda.device_count()
    torch.cuda.set_device(local)
    backend = os.environ.get("EMOE_BENCH_BACKEND", "nccl")
    if backend == "nccl":
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    else:
        dist.init_process_group(backend)
    peak, peak_kind = measured_peak()
    wl = W.make_exchange_workload(world, n_layers=args.layers)
    kinds = (W.KIND_EXPERTS, W.KIND_ATTN, W.KIND_KV)
    stream = torch.cuda.Stream()
    with E.Plan(wl.shape, wl.old, wl.new) as plan:
        old, new = [], []
        for ph in range(3):
            so, sn = plan.arena_bytes(ph, E.SIDE_OLD), plan.arena_bytes(ph, E.SIDE_NEW)
            mine = None
            if rank < len(so):      # this process owns rank index `rank` of either side
                mine = torch.empty(so[rank], dtype=torch.uint8, device="cuda")
                W.rng.torch_fill_bytes(mine, W.arena_key(wl.seed, kinds[ph], rank))
            old.append(mine)
            new.append(WD.alloc_const([sn[rank]])[0] if rank < len(sn) else None)
        torch.cuda.synchronize()
        dist.barrier()
        ex = exchange.Exchange(dist, plan, rank, old, new, whole_step=True)
        try:
            pulled = ex.bytes_pulled()
            for _ in range(args.warmup):
                ex.step(stream)
            stream.synchronize()
            dist.barrier()
            torch.cuda.synchronize()
            sampler = ClockSampler(local)
            sampler.start()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(args.steps):
                ex.step(stream)
            e1.record(stream)
            stream.synchronize()
            torch.cuda.synchronize()
            clocks = sampler.stop()
            dist.barrier()
            local_ms = e0.elapsed_time(e1)
            dev = "cuda" if backend == "nccl" else "cpu"
            total_ms = replicas.job_time_ms(local_ms, dist, device=dev)
            status = plan.device_status()
            n_launch = plan.num_launches(E.PHASE_STEP)
            per_rank = [None] * world
            dist.all_gather_object(per_rank, dict(rank=rank, ms_per_step=round(local_ms / args.steps, 4),
                                                  bytes_written=pulled["written"],
                                                  bytes_from_peers=pulled["from_peers"],
                                                  pull_gbs=round(pulled["from_peers"] / (local_ms / args.steps) / 1e6, 1),
                                                  launches_per_step=n_launch, device_status=status))
        finally:
            ex.close()
    if rank == 0:
        moved = sum(r["bytes_written"] for r in per_rank)
        ms = total_ms / args.steps
        line = {"metric": METRIC, "value": round(2 * moved / ms / 1e6, 1), "unit": UNIT, "n_gpus": world,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(ms, 4),
                "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": "u8",
                "data": "synthetic", "mode": "exchange",
                "config": {"workload": wl.name if args.layers is None
                           else "%s cut to %d layers" % (wl.name, args.layers),
                           "reconfig": wl.notes, "parallelism": "one rank per GPU, pull over peer mappings",
                           "l2": "inputs_larger_than_l2", "value_convention": "2 x bytes written by all ranks / slowest rank's time",
                           "control_plane": backend},
                "clocks": clocks, "per_rank": per_rank,
                "bytes_from_peers_total": sum(r["bytes_from_peers"] for r in per_rank),
                "e2e": {"value": None, "unit": UNIT, "note": "measured in the default mode at --gpus 1 only"},
                "gpu_launches": sum(r["launches_per_step"] for r in per_rank) * args.steps}
        print(json.dumps(line))
    dist.barrier()
    dist.destroy_process_group()


# ---- main --------------------------------------------------------------------------------

def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="c2_mid")
    ap.add_argument("--impl", default="emoe", choices=["emoe", "reference"])
    ap.add_argument("--mode", default="replicas", choices=["replicas", "exchange"],
                    help="replicas (default): every GPU runs the whole workload on its own; exchange: one "
                         "rank per GPU, the step pulled over the interconnect (needs --gpus >= 2)")
    ap.add_argument("--only-main", action="store_true",
                    help="skip the other configs, the overlap case, e2e and the CPU baseline")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--layers", type=int, default=None,
                    help="cut the workload to this many layers (for small profiler captures "
                         "only: the result is then not the named configuration)")
    ap.add_argument("--steps-only", action="store_true",
                    help="with --only-main: run nothing but the warm-up and the timed steps (for profiler captures)")
    ap.add_argument("--record-traffic", default=None, metavar="NCU_RAW_CSV",
                    help="do not run: parse `ncu -i X.ncu-rep --page raw --csv` of a capture of "
                         "`bench.py --only-main --steps-only --workload W --layers N` into profiles/traffic.json")
    ap.add_argument("--traffic-command", default=None, help="the capture's command line, stored with --record-traffic")
    ap.add_argument("--traffic-merge", action="store_true",
                    help="with --record-traffic: add the capture's kernels to the workload's entry as the kernels "
                         "of the per-phase entry points instead of replacing the entry")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "emoe" else args.warmup
    if args.record_traffic:
        record_traffic(args)
        return

    if args.impl == "reference":
        run_reference(args)
        return
    if args.mode == "exchange":
        run_exchange(args)
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
    traffic = load_traffic()
    sampler = ClockSampler(local)
    sampler.start()
    total_ms, each = time_steps(torch, plan, src, dst, args.steps, args.warmup, stream, barrier)
    clocks = sampler.stop()
    if args.steps_only:
        phase_ms = [0.0, 0.0, 0.0]
    else:
        phase_ms = time_phases(torch, plan, src, dst, max(3, min(args.steps, 20)), stream)
    total_ms = replicas.job_time_ms(total_ms, dist, device="cuda" if backend == "nccl" else "cpu")  # max over ranks
    rep = config_report(E, plan, wl, total_ms, each, phase_ms, args.steps, peak, peak_kind, plan_ms, traffic,
                        cut=args.layers is not None)
    if plan.device_status() != 0:
        raise SystemExit("device status word set: a bounded wait expired")
    ms = total_ms / args.steps
    value = replicas.job_throughput_gbs(rep["bytes_moved"], world, ms)
    per_step = plan.num_launches(E.PHASE_STEP)
    launches = per_step * args.steps

    # roofline of the dominant kernel, the ring-copy launch: the whole step when the step is
    # that one launch (TP kept: every segment of every phase is a long run), otherwise the
    # kernel block timed through the expert phase's own entry point
    blocks = rep["roofline"]["kernels"]
    roofline = next((b for b in blocks if b["kernel"] == "bulk_copy_kernel"), None) or rep["roofline"]["step"]

    line = {"metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(ms, 4),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u8",
            "data": "synthetic",
            "config": {"workload": wl.name if args.layers is None
                       else "%s cut to %d layers" % (wl.name, args.layers),
                       "reconfig": wl.notes, "parallelism": "replicas",
                       "l2": "inputs_larger_than_l2", "value_convention": "2 x bytes moved / time",
                       "scale_step_ms": rep["scale_step_ms"], "step_spread": rep["step_spread"],
                       "pct_of_nominal_8000": rep["pct_of_nominal_8000"],
                       "pct_of_measured_peak": rep["pct_of_measured_peak"]},
            "clocks": clocks, "gpu_launches": launches, "roofline": roofline,
            "roofline_step": rep["roofline"]["step"],
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
                e_ms, h2d, d2h, link = run_e2e(torch, e2e_plan, src, dst, args.e2e_steps, stream)
            # the step cannot beat the slower direction of the host link carrying its bytes
            link_ms = max(h2d / link["h2d_gbs"], d2h / link["d2h_gbs"]) / 1e6
            line["e2e"] = {"value": round(2 * rep["bytes_moved"] / (e_ms * 1e-3) / 1e9, 2),
                           "unit": UNIT, "ms_per_step": round(e_ms, 2), "steps": args.e2e_steps,
                           "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                           "host_link": link, "host_link_bound_ms": round(link_ms, 2),
                           "frac_of_host_link": round(link_ms / e_ms, 3)}
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
        for key, fn in (("kv_compacting_new_table", lambda: run_kv_compacting(torch, E, W, WD, wl.name, rep["phases"]["kv"]["ms"])),
                        ("inplace_expert_step", lambda: run_inplace(torch, E, wl, rep["phases"]["experts"]["ms"], peak)),
                        ("vmm_expert_step", lambda: run_vmm(torch, E, wl, rep["phases"]["experts"]["ms"])),
                        ("vmm_slots_expert_step", lambda: run_vmm_slots(torch, E, wl, rep["phases"]["experts"]["ms"]))):
            try:
                rep[key] = fn()
            except Exception as e:      # report, never hide
                rep[key] = {"error": repr(e)[:300]}
                torch.cuda.empty_cache()

    def measure_config(name):
        wl2, plan2, src2, dst2, pms = setup(name, torch, E, W, WD)
        try:
            # at least 100 steps and about a second of timed region each; the tiny config is
            # timed without per-step events (an event costs a tenth of its step)
            k = {"c1_tiny": 2000}.get(name, max(100, args.steps // 2))
            tot, each2 = time_steps(torch, plan2, src2, dst2, k, 3, stream, per_step=name != "c1_tiny")
            ph = time_phases(torch, plan2, src2, dst2, 20, stream)
            r = config_report(E, plan2, wl2, tot, each2, ph, k, peak, peak_kind, pms, traffic)
            if plan2.device_status() != 0:
                r["error"] = "device status word set: a bounded wait expired"
            if name == "c1_tiny":    # launch-bound: also as a CUDA-graph replay
                g_ms = time_graph_steps(torch, plan2, src2, dst2, k, 3, stream)
                r["cuda_graph"] = {"scale_step_ms": round(g_ms, 4),
                                   "reshard_gbs": round(2 * r["bytes_moved"] / g_ms / 1e6, 1)}
            if name == "c5_overlap":
                r["overlap"] = run_overlap(torch, E, plan2, wl2, src2, dst2, peak, wl2.victim)
            if name == "c4_large":   # the same victim beside the TP-changing reshard
                r["overlap"] = run_overlap(torch, E, plan2, wl2, src2, dst2, peak,
                                           W.make_workload("c5_overlap").victim,
                                           points=(dict(), dict(bw_limit_gbs=4500), dict(bw_limit_gbs=2500)))
        finally:
            del src2, dst2
            plan2.close()
            torch.cuda.empty_cache()
        if name in ("c2_mid", "c3_fine", "c4_large"):
            for key, fn in (("kv_compacting_new_table", lambda: run_kv_compacting(torch, E, W, WD, name, r["phases"]["kv"]["ms"])),
                            ("inplace_expert_step", lambda: run_inplace(torch, E, wl2, r["phases"]["experts"]["ms"], peak)),
                            ("vmm_expert_step", lambda: run_vmm(torch, E, wl2, r["phases"]["experts"]["ms"])),
                            ("vmm_slots_expert_step", lambda: run_vmm_slots(torch, E, wl2, r["phases"]["experts"]["ms"]))):
                try:
                    r[key] = fn()
                except Exception as e:
                    r[key] = {"error": repr(e)[:300]}
                    torch.cuda.empty_cache()
        return r

    if not args.only_main and world == 1:
        others = {}
        for name in W.WORKLOAD_NAMES + W.EXTRA_WORKLOAD_NAMES:
            if name == args.workload:
                others[name] = rep
                continue
            # a config that cannot be measured (out of memory on a smaller device, ...) is
            # reported as such in its place; it does not take the line down with it
            try:
                others[name] = measure_config(name)
            except Exception as e:
                others[name] = {"workload": name, "error": repr(e)[:300]}
                torch.cuda.empty_cache()
        line["configs"] = others

    if dist:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(line))


if __name__ == "__main__":
    main()
