#!/usr/bin/env python
"""Throughput of the schedule-exact reduction on B200: `python bench.py --gpus N --steps K --warmup W`.

A step is one pass of the reduction path over one batch of synthetic inputs: for every schedule and
operation the workload names, one tree-mode reduction of the p resident messages (fp32) into a root
buffer.  The schedules themselves (cost model, event generation, combine programs) are plans built once
and reused; their build time is reported beside the throughput.  Metric: reduction GB/s, counting p*m
input bytes plus m output bytes per reduction.

The default workload is the large-message one (p = 32 processes, 1 GiB per process, 1 MiB segments,
uni- and bi-greedy schedules, sum and max): the largest of the named workloads that one GPU holds, and
the only one with messages above 64 MB.  The small workload with 4 MiB messages (one batch launch per
step, two streams) is measured in the same run and reported under `config2_batch`.

One JSON line is printed by rank 0.  With N > 1 every rank runs an independent replica on its own
GPU (the path needs no exchange between GPUs); times are taken on the device and the slowest rank
counts.  `--impl reference` times the plain CPU checker instead, on rank 0 only.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

TICK = 1e-15
# schedules per workload: (label, algo name, bidirectional ports)
WORKLOAD_SCHEDULES = {
    "config1": [("uni_greedy", "uni_greedy", False)],
    "config2": [("uni_greedy", "uni_greedy", False), ("binomial", "binomial", False),
                ("pipeline", "pipeline", False), ("binary", "binary", False)],
    "config3": [("bi_greedy", "bi_greedy", True), ("butterfly", "butterfly", True), ("binomial", "binomial", True),
                ("pipeline", "pipeline", True), ("binary", "binary", True)],
    "config4": [("uni_greedy", "uni_greedy", False), ("bi_greedy", "bi_greedy", True)],
}
WORKLOAD_OPS = {"config1": ["sum"], "config2": ["sum"], "config3": ["sum"], "config4": ["sum", "max"]}
KERNEL_SOURCE = os.path.join(ROOT, "paper_1310_4645_b200", "csrc", "rd_kernels.cu")
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "rd_tree_stream_kernel_dram_traffic.txt")


def profiled_traffic(p, n, launch):
    """DRAM bytes per launch of the streaming kernel as a profiler counted them, from the capture file kept
    beside the profile summaries: one `capture key=value ...` line per captured launch shape.  A capture made
    with the same number of processes and launch form on shorter messages is scaled by the message length
    (the kernel reads every input word once and writes every output word once, whatever the length).
    None when no capture applies or the kernel source is no longer the one that was profiled."""
    try:
        with open(KERNEL_SOURCE, "rb") as f:
            sha = hashlib.sha256(f.read()).hexdigest()
        best = None
        with open(TRAFFIC_FILE) as f:
            for ln in f:
                if not ln.startswith("capture "):
                    continue
                kv = dict(t.split("=", 1) for t in ln.split()[1:])
                if kv.get("kernel_sha256") != sha or int(kv["p"]) != p or kv.get("launch") != launch:
                    continue
                if n % int(kv["n_elems"]):
                    continue
                scale = n // int(kv["n_elems"])
                if best is None or scale < best[0]:
                    best = (scale, float(kv["dram_bytes_per_launch"]) * scale,
                            "ncu dram__bytes_read.sum + dram__bytes_write.sum of one launch with %s elements per process, times %d"
                            % (kv["n_elems"], scale) if scale > 1 else "ncu dram__bytes_read.sum + dram__bytes_write.sum of this launch shape")
        return (best[1], best[2]) if best else (None, None)
    except Exception:
        return None, None


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs, copy read+write)"
    except Exception:
        return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs (read only)."""

    def __init__(self, index):
        super().__init__(daemon=True)
        self.index, self.samples, self.reasons, self.max_mhz = index, [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
            "hw_power_brake": getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80),
        }
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.02)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2] if s else None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(s)}


def max_over_ranks(value, device=None):
    """The largest `value` over all ranks of the default process group (the slowest rank sets the time)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replica_throughput(bytes_per_rank, ms, world):
    """Whole-job GB/s of `world` independent replicas that each moved bytes_per_rank in at most ms."""
    return world * bytes_per_rank / (ms * 1e-3) / 1e9


def visible_gpu_index(local_rank):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


# ------------------------------------------------------------------------------------------------
# The CPU checker's legs (the reference arm and cpu_baseline): nothing of the GPU path is used here.
# ------------------------------------------------------------------------------------------------
def oracle_events(algo_name, bidir, p, msg_bytes, seg_bytes, model):
    """(events, segment offsets in elements) of the CPU checker's own schedule simulators."""
    import numpy as np
    from oracle import rd_oracle as O
    A, B, G = (int(round(v / TICK)) for v in model)
    if algo_name == "butterfly":
        ev, off, _ = O.butterfly(p, msg_bytes // 4, 4, A, B, G)
        return ev, off
    sizes = O.equal_sizes(msg_bytes, min(seg_bytes, msg_bytes))
    if algo_name == "uni_greedy":
        ev, _ = O.uni_greedy(p, sizes, A, B, G)
    elif algo_name == "bi_greedy":
        ev, _ = O.bi_greedy(p, sizes, A, B, G)
    elif algo_name == "binomial":
        ev, _ = O.binomial(p, sizes, A, B, G)
    elif algo_name == "pipeline":
        ev, _ = O.pipeline(p, sizes, A, B, G, bidir)
    else:
        ev, _ = O.binary(p, sizes, A, B, G, bidir)
    off = np.concatenate([[0], np.cumsum(np.asarray(sizes, dtype=np.int64) // 4)])
    return ev, off


def oracle_schedule_ms(w, wname):
    """Time the CPU checker's simulators take to generate the workload's schedules at FULL size."""
    t0 = time.perf_counter()
    for _, algo_name, bidir in WORKLOAD_SCHEDULES[wname]:
        oracle_events(algo_name, bidir, w["p"], 4 * w["n"], w["seg_bytes"], (w["alpha"], w["beta"], w["gamma"]))
    return (time.perf_counter() - t0) * 1e3


def cpu_plans(w, wname, n):
    return [oracle_events(algo_name, bidir, w["p"], 4 * n, w["seg_bytes"], (w["alpha"], w["beta"], w["gamma"]))
            for _, algo_name, bidir in WORKLOAD_SCHEDULES[wname]]


def cpu_pass(plans, ops, x_host, budget_s, max_passes, openmp):
    """Times the CPU checker's reductions (every schedule x operation) on x_host; repeats until the budget
    is used.  Returns (GB/s, passes, seconds)."""
    from oracle import rd_oracle as O
    p, n = x_host.shape
    bytes_per_pass = len(plans) * len(ops) * (p + 1) * n * 4
    t_total, passes = 0.0, 0
    while passes < max_passes and (passes == 0 or t_total < budget_s):
        t0 = time.perf_counter()
        for ev, off in plans:
            for op in ops:
                O.reduce(ev, x_host, off, op, openmp=openmp)
        t_total += time.perf_counter() - t0
        passes += 1
    return bytes_per_pass * passes / t_total / 1e9, passes, t_total


def host_slab(w, max_bytes):
    """Host copy of the workload, or of its first whole segments when it exceeds max_bytes."""
    from paper_1310_4645_b200.inputs import make_inputs
    p, n = w["p"], w["n"]
    seg = w["seg_bytes"] // 4
    if p * n * 4 > max_bytes:
        n = max(seg, (max_bytes // (4 * p)) // seg * seg)
    return make_inputs(p, n, w["dist"], w["seed"], device="cpu"), n


def cpu_baseline(w, wname, budget_s):
    """The CPU checker on a slab of whole segments of the workload: its plain build on one core, and its
    OpenMP build (same source, threads share the elements of every segment) on all cores the box gives us."""
    from oracle import rd_oracle as O
    x, n_s = host_slab(w, 512 << 20)
    xh = x.numpy()
    plans = cpu_plans(w, wname, n_s)
    ops = WORKLOAD_OPS[wname]
    v1, passes1, dt1 = cpu_pass(plans, ops, xh, budget_s / 2, 200, openmp=False)
    cores = O.threads(openmp=True)
    cpu_pass(plans, ops, xh, 0.0, 1, openmp=True)                        # the thread team's first start
    vn, passesn, dtn = cpu_pass(plans, ops, xh, budget_s / 2, 400, openmp=True)
    what = "every schedule x op of the workload on the first %d of %d elements per process (whole segments)" % (n_s, w["n"])
    return {"value": vn, "unit": "GB/s", "cores": cores, "kind": "oracle",
            "sample": "%d passes over %s, %.1f s, OpenMP build of the checker (threads split the elements)" % (passesn, what, dtn),
            "one_core": {"value": v1, "unit": "GB/s", "cores": 1,
                         "sample": "%d passes over the same sample, %.1f s, plain build" % (passes1, dt1)},
            "affinity_cores": len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else None,
            "oracle_schedule_ms": oracle_schedule_ms(w, wname)}


def run_reference(args, wname, w):
    """The CPU checker as it stands, timed on the host cores: one step = one pass over a bounded slab."""
    from oracle import rd_oracle as O
    x, n = host_slab(w, 512 << 20)
    xh = x.numpy()
    plans = cpu_plans(w, wname, n)
    ops = WORKLOAD_OPS[wname]
    for _ in range(args.warmup):
        cpu_pass(plans, ops, xh, 0.0, 1, openmp=True)
    t0 = time.perf_counter()
    gb = 0.0
    for _ in range(args.steps):
        v, _, dt = cpu_pass(plans, ops, xh, 0.0, 1, openmp=True)
        gb += v * dt
    dt = time.perf_counter() - t0
    value = gb / dt
    v1, _, _ = cpu_pass(plans, ops, xh, 0.0, 1, openmp=False)
    sample = ("each step: every schedule x op of the workload on the first %d of %d elements per process (whole segments), "
              "OpenMP build of the checker" % (n, w["n"]))
    line = {"impl": "reference", "metric": "reduction_throughput", "value": value, "unit": "GB/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "i32" if w["dist"].startswith("int") else "f32", "data": "synthetic",
            "config": {"workload": wname, "p": w["p"], "n_elems": w["n"], "segment_bytes": w["seg_bytes"],
                       "schedules": [s[0] for s in WORKLOAD_SCHEDULES[wname]], "ops": WORKLOAD_OPS[wname]},
            "cpu_baseline": {"value": value, "unit": "GB/s", "cores": O.threads(openmp=True), "kind": "oracle", "sample": sample,
                             "one_core": {"value": v1, "unit": "GB/s", "cores": 1, "sample": "one pass, plain build"}},
            "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------
# The GPU path
# ------------------------------------------------------------------------------------------------
class TreeBench:
    """Resident inputs, plans and the timed loops of one workload on one GPU."""

    def __init__(self, rd, torch, wname, w, dev, issue, streams):
        from paper_1310_4645_b200.inputs import make_inputs
        self.rd, self.torch, self.wname, self.w, self.dev = rd, torch, wname, w, dev
        p, n = w["p"], w["n"]
        self.p, self.n = p, n
        self.bytes_per_reduce = (p + 1) * n * 4
        self.model = (w["alpha"], w["beta"], w["gamma"])
        self.schedules = WORKLOAD_SCHEDULES[wname]
        self.op_names = WORKLOAD_OPS[wname]
        n_plans = len(self.schedules)
        # Batch issue: every job of a step reads its own messages (jobs of one launch that read the same bytes
        # would meet in L2), and steps that may overlap on two streams read different sets of them.
        if issue == "batch" and p * n * 4 * n_plans * 2 > (48 << 30):
            issue = "calls"                  # too much memory for a set of messages per job and stream
        self.issue = issue
        # Call issue: the kernel never reads the arena the previous launch read, and two arenas together exceed
        # L2; a workload whose single arena is many times L2 needs no rotation.
        if issue == "batch":
            self.batch_sets = 2
            n_arenas = n_plans * self.batch_sets
        else:
            self.batch_sets = 0
            n_arenas = 3 if p * n * 4 <= (1 << 30) else 1
        if streams is None:                  # launches of one arena that is far larger than L2 go back to back
            streams = 2 if n_arenas > 1 else 1
        self.n_streams = streams
        self.arenas = [make_inputs(p, n, w["dist"], w["seed"] + 1000 * a, device=str(dev)) for a in range(n_arenas)]
        self.n_arenas = n_arenas
        self.out = torch.empty(n, dtype=self.arenas[0].dtype, device=dev)
        self.tables = [rd.PointerTable(a) for a in self.arenas]
        t0 = time.perf_counter()
        self.plans = []
        for label, algo_name, bidir in self.schedules:
            h = rd.rd_schedule_create(rd.ALGOS[algo_name], rd.RD_PORT_BI if bidir else rd.RD_PORT_UNI, p, 4 * n,
                                      w["seg_bytes"], *self.model)
            self.plans.append((label, h))
        self.create_ms = (time.perf_counter() - t0) * 1e3
        for _, h in self.plans:
            rd.rd_schedule_upload(h)
        self.ops = [rd.RD_SUM if o == "sum" else rd.RD_MAX for o in self.op_names]
        self.reduces_per_step = len(self.plans) * len(self.ops)
        self.launches_per_step = len(self.ops) if issue == "batch" else self.reduces_per_step
        self.counter = 0
        self.outs = [torch.empty(n, dtype=self.arenas[0].dtype, device=dev) for _ in range(self.reduces_per_step)]
        self.main_stream = torch.cuda.current_stream(dev)
        self.side = [torch.cuda.Stream(device=dev) for _ in range(streams)] if streams > 1 else [self.main_stream]
        self.batches = None
        if issue == "batch":
            self.batches = [[rd.Batch([(h, self.tables[s_ * n_plans + j], self.outs[k * n_plans + j])
                                       for j, (_, h) in enumerate(self.plans)])
                             for k in range(len(self.ops))] for s_ in range(self.batch_sets)]

    def close(self):
        for _, h in self.plans:
            self.rd.rd_destroy(h)
        self.plans = []
        self.arenas = self.tables = self.outs = self.batches = self.out = None
        self.torch.cuda.empty_cache()

    # A step reduces messages under every schedule (and operation) of the workload: independent reductions,
    # each with its own output.
    #   batch issue: one rd_reduce_batch call per operation, i.e. ONE launch of the streaming kernel whose
    #     tiles are those of all the schedules' reductions (each job on its own messages);
    #   call issue: one rd_reduce call per schedule and operation; launch i of the run reads arena i mod n_arenas.
    # The calls alternate over the given CUDA streams: with two streams one launch's thread blocks take the SM
    # slots the other frees while its last blocks are still running.
    def step(self, streams):
        rd = self.rd
        if self.batches is not None:
            for k, op in enumerate(self.ops):
                c = self.counter
                rd.rd_reduce_batch(self.batches[c % self.batch_sets][k], op, stream=streams[c % len(streams)])
                self.counter += 1
            return
        i = 0
        for _, h in self.plans:
            for op in self.ops:
                rd.rd_reduce(h, self.tables[self.counter % self.n_arenas], self.outs[i], op, stream=streams[i % len(streams)])
                self.counter += 1
                i += 1

    def timed(self, streams, steps):
        """Device time of `steps` steps: the events sit on the main stream, the other streams start after
        the first event and the second one waits for them."""
        torch = self.torch
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(self.main_stream)
        for st in streams:
            if st is not self.main_stream:
                st.wait_event(e0)
        self.step_marks = [e0]
        for _ in range(steps):
            self.step(streams)
            if len(streams) == 1:
                # one stream: an event after every step gives the spread over the steps (median, best)
                mark = torch.cuda.Event(enable_timing=True)
                mark.record(self.main_stream)
                self.step_marks.append(mark)
        for st in streams:
            if st is not self.main_stream:
                done = torch.cuda.Event()
                done.record(st)
                self.main_stream.wait_event(done)
        e1.record(self.main_stream)
        return e0, e1

    def step_spread(self):
        """Median and best step time (ms) of the last one-stream timed region, or None."""
        marks = getattr(self, "step_marks", [])
        if len(marks) < 2:
            return None
        t = sorted(a.elapsed_time(b) for a, b in zip(marks[:-1], marks[1:]))
        return {"median": t[len(t) // 2], "best": t[0], "worst": t[-1]}

    def per_schedule(self, reps):
        rd, torch = self.rd, self.torch
        res = {}
        for label, h in self.plans:
            for opname, op in zip(self.op_names, self.ops):
                for _ in range(3):
                    rd.rd_reduce(h, self.tables[self.counter % self.n_arenas], self.out, op); self.counter += 1
                torch.cuda.synchronize()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                for _ in range(reps):
                    rd.rd_reduce(h, self.tables[self.counter % self.n_arenas], self.out, op); self.counter += 1
                b.record()
                torch.cuda.synchronize()
                res["%s/%s" % (label, opname)] = round(self.bytes_per_reduce * reps / (a.elapsed_time(b) * 1e-3) / 1e9, 1)
        return res

    def faithful(self, reps=9):
        """Schedule-faithful execution: measured makespan of every schedule beside the linear model's prediction.
        The schedules take turns (one run of each per round), so that a drift of the clocks touches all alike;
        the median of `reps` rounds counts.  Two rankings are compared: as measured, and with schedules whose
        medians lie within 3 % of each other counted as tied (their order is then within the run-to-run noise)."""
        rd = self.rd
        spans = {label: [] for label, _ in self.plans}
        for rep in range(reps + 2):
            for label, h in self.plans:
                st = rd.rd_reduce(h, self.tables[rep % self.n_arenas], self.out, self.ops[0], exec_mode=rd.RD_EXEC_FAITHFUL, want_stats=True)
                if rep >= 2:
                    spans[label].append(st.makespan_ns)
        rows = {}
        for label, h in self.plans:
            v = sorted(spans[label])
            shape = rd.rd_schedule_faithful_shape(h)
            rows[label] = {"measured_us": v[len(v) // 2] / 1e3, "best_us": v[0] / 1e3,
                           "predicted_us": rd.rd_schedule_info(h)["predicted_seconds"] * 1e6,
                           "blocks_per_process": shape["blocks_per_process"], "slots_per_process": shape["slots_per_process"]}
        by_model = sorted(rows, key=lambda k: rows[k]["predicted_us"])
        by_gpu = sorted(rows, key=lambda k: rows[k]["measured_us"])
        # the model's order holds up to ties: no pair it orders a < b was measured the other way round by more than 3 %
        within = all(rows[a]["measured_us"] <= 1.03 * rows[b]["measured_us"]
                     for i, a in enumerate(by_model) for b in by_model[i + 1:])
        return {"schedules": rows, "rank_by_model": by_model, "rank_measured": by_gpu,
                "ranks_agree": by_model == by_gpu, "ranks_agree_up_to_3pct_ties": within,
                "fastest_agrees": by_model[0] == by_gpu[0],
                "models_fastest_within_3pct_of_measured_fastest": rows[by_model[0]]["measured_us"] <= 1.03 * rows[by_gpu[0]]["measured_us"]}

    def launch_shape(self):
        rd = self.rd
        shape0 = rd.rd_schedule_tree_shape(self.plans[0][1])
        if self.issue == "batch":                   # the batch launch: all jobs' tiles, the deepest stack among them
            tiles = sum(rd.rd_schedule_tree_shape(h)["n_tiles"] for _, h in self.plans)
            return {"blocks_per_sm": "chosen for the batch's tiles and deepest stack",
                    "ring_stages": "chosen for the batch's tiles and deepest stack", "tiles": tiles}, "rd_tree_stream_kernel"
        kernel = "rd_tree_direct_kernel" if shape0["variant"] == rd.RD_TREE_DIRECT else "rd_tree_stream_kernel"
        return {"blocks_per_sm": shape0["blocks_per_sm"], "ring_stages": shape0["ring_stages"], "tiles": shape0["n_tiles"]}, kernel

    def describe(self, world):
        p, n, w = self.p, self.n, self.w
        n_plans = len(self.plans)
        if self.issue == "batch":
            issue = ("a step is one rd_reduce_batch call per operation: one launch for the step's %d independent reductions, "
                     "each on its own messages; steps alternate over %d CUDA stream(s) and %d sets of messages"
                     % (n_plans, self.n_streams, self.batch_sets))
            l2 = ("a launch reads %.0f MiB that no launch running beside it reads (%d arenas of %.0f MiB)"
                  % (n_plans * p * n * 4 / 2**20, self.n_arenas, p * n * 4 / 2**20))
        else:
            issue = ("the step's %d independent reductions are separate rd_reduce calls (one kernel launch each) on %d CUDA stream(s)"
                     % (self.reduces_per_step, self.n_streams))
            l2 = ("inputs rotate over %d arenas of %.0f MiB each (> L2 between reuses)" % (self.n_arenas, p * n * 4 / 2**20)
                  if self.n_arenas > 1 else "inputs (%.1f GiB per reduction) exceed L2 (126 MB) many times over" % (p * n * 4 / 2**30))
        return {"workload": self.wname, "p": p, "n_elems": n, "segment_bytes": w["seg_bytes"],
                "schedules": [s[0] for s in self.schedules], "ops": self.op_names,
                "bytes_counted": "p*m + m per reduction", "issue": issue, "l2": l2,
                "parallelism": "replicas only" if world > 1 else "single GPU"}


def measure(tb, steps, warmup, barrier, dev, world, sample_clocks, local_rank):
    """Warm-up, the timed region (value) and the same launches back to back on one stream (the kernel's own time)."""
    for _ in range(warmup):
        tb.step(tb.side)
    barrier()
    sampler = None
    if sample_clocks:
        sampler = ClockSampler(visible_gpu_index(local_rank))
        sampler.start()
    e0, e1 = tb.timed(tb.side, steps)
    barrier()
    clocks = sampler.stop() if sampler else None
    ms = max_over_ranks(e0.elapsed_time(e1), dev)
    spread = tb.step_spread()
    value = replica_throughput(steps * tb.reduces_per_step * tb.bytes_per_reduce, ms, world)
    if tb.n_streams > 1:
        k_steps = max(3, steps // 2)
        for _ in range(3):
            tb.step([tb.main_stream])
        barrier()
        k0, k1 = tb.timed([tb.main_stream], k_steps)
        barrier()
        kernel_ms = max_over_ranks(k0.elapsed_time(k1), dev) / (k_steps * tb.launches_per_step)
        timed_over = "%d launches back to back on one stream after the timed region, %.2f us each" % (k_steps * tb.launches_per_step, kernel_ms * 1e3)
    else:
        kernel_ms = ms / (steps * tb.launches_per_step)
        timed_over = "the %d launches of the timed region (one stream, CUDA events around it), %.2f us each" % (steps * tb.launches_per_step, kernel_ms * 1e3)
    return value, ms, kernel_ms, timed_over, clocks, spread


def roofline_block(tb, kernel_ms, timed_over):
    peak, peak_src = measured_peak()
    bytes_per_launch = tb.bytes_per_reduce * tb.reduces_per_step // tb.launches_per_step
    achieved = bytes_per_launch / (kernel_ms * 1e-3) / 1e9
    shape, kernel = tb.launch_shape()
    n_jobs = len(tb.plans) if tb.issue == "batch" else 1
    traffic, traffic_src = profiled_traffic(tb.p, tb.n, "batch%d" % n_jobs if tb.issue == "batch" else "single")
    return {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
            "traffic": traffic, "traffic_unit": "bytes per launch", "traffic_source": traffic_src,
            "algorithmic_bytes": bytes_per_launch, "peak_source": peak_src, "kernel": kernel, "launch_shape": shape,
            "timed_over": timed_over, "frac_of_nominal_8000": achieved / 8000.0}


def end_to_end(rd, torch, tb, dev, world, barrier, steps):
    """Host buffers in, host result out, through rd_reduce_host: the H2D copy of all p messages and the D2H
    copy of the result are inside the timed region.  A workload above 4 GiB is run on a slab of whole
    segments (its first `n` elements per process, a schedule of the same kind built for that length)."""
    w, p = tb.w, tb.p
    seg = w["seg_bytes"] // 4
    n = tb.n
    if p * n * 4 > (4 << 30):
        n = max(seg, ((2 << 30) // (4 * p)) // seg * seg)
    host_bytes = p * n * 4
    hx = tb.arenas[0][:, :n].cpu().pin_memory()
    hout = torch.empty(n, dtype=hx.dtype).pin_memory()
    staging = torch.empty((p + 1) * n, dtype=hx.dtype, device=dev)
    if n == tb.n:
        plans, own = tb.plans, False
    else:
        plans = [(label, rd.rd_schedule_create(rd.ALGOS[algo_name], rd.RD_PORT_BI if bidir else rd.RD_PORT_UNI, p, 4 * n,
                                               w["seg_bytes"], *tb.model)) for label, algo_name, bidir in tb.schedules]
        own = True
    try:
        e_steps = max(3, min(steps, int(2.0 / (tb.reduces_per_step * host_bytes / 40e9)) or 1))
        for _, h in plans:
            rd.rd_reduce_host(h, hx, hout, staging, tb.ops[0])
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(e_steps):
            for _, h in plans:
                for op in tb.ops:
                    rd.rd_reduce_host(h, hx, hout, staging, op)
        b.record()
        barrier()
        e_ms = max_over_ranks(a.elapsed_time(b), dev)
    finally:
        if own:
            for _, h in plans:
                rd.rd_destroy(h)
    return {"value": replica_throughput(e_steps * tb.reduces_per_step * (p + 1) * n * 4, e_ms, world), "unit": "GB/s",
            "h2d_bytes_per_step": tb.reduces_per_step * host_bytes, "d2h_bytes_per_step": tb.reduces_per_step * n * 4,
            "steps": e_steps, "ms_per_step": e_ms / e_steps,
            "sample": "rd_reduce_host (pinned host buffers) on %s" % ("the whole workload" if n == tb.n else
                      "the first %d of %d elements per process (%d whole segments), every schedule x op" % (n, tb.n, n // seg))}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="config4", choices=sorted(WORKLOAD_SCHEDULES))
    ap.add_argument("--n-elems", type=int, default=None,
                    help="elements per process instead of the workload's (a multiple of its segment): a smaller case of the "
                         "same launches, for profiler captures; the line then names the workload with its changed length")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-small", action="store_true", help="skip the extra small-message (config2, batch launch) measurement")
    ap.add_argument("--no-faithful", action="store_true", help="skip the schedule-faithful makespan measurement")
    ap.add_argument("--issue", default="batch", choices=["batch", "calls"],
                    help="batch: a step is one rd_reduce_batch call per operation (one launch for all schedules; used when a set of "
                         "messages per job and stream fits in 48 GiB); calls: one rd_reduce call per schedule and operation")
    ap.add_argument("--streams", type=int, default=None, choices=[1, 2],
                    help="CUDA streams the independent reductions of the timed region alternate over "
                         "(default: 2 when the inputs rotate over several arenas, 1 when one arena far above L2 is read)")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    from paper_1310_4645_b200.inputs import WORKLOADS
    wname = args.workload
    w = WORKLOADS[wname]
    if args.n_elems is not None:
        if args.n_elems <= 0 or (4 * args.n_elems) % w["seg_bytes"]:
            ap.error("--n-elems must be a positive multiple of the workload's segment (%d elements)" % (w["seg_bytes"] // 4))
        w = dict(w, n=args.n_elems)

    if args.impl == "reference":
        if rank != 0:
            return 0
        args.steps = args.steps if args.steps is not None else 5
        args.warmup = args.warmup if args.warmup is not None else 1
        run_reference(args, wname, w)
        return 0

    import torch
    import paper_1310_4645_b200 as rd

    p, n = w["p"], w["n"]
    bytes_per_step = len(WORKLOAD_SCHEDULES[wname]) * len(WORKLOAD_OPS[wname]) * (p + 1) * n * 4
    if args.steps is None:                   # about a second of timed work, at least 20 steps
        args.steps = max(20, int(1.0 / (bytes_per_step / 5e12)))
    if args.warmup is None:
        args.warmup = max(3, args.steps // 20)
    args.warmup = max(args.warmup, 3)

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist_on = world > 1
    if dist_on:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if dist_on:
            dist.barrier()
        torch.cuda.synchronize()

    tb = TreeBench(rd, torch, wname, w, dev, args.issue, args.streams)
    value, ms, kernel_ms, timed_over, clocks, spread = measure(tb, args.steps, args.warmup, barrier, dev, world, True, local_rank)
    per_schedule = tb.per_schedule(max(5, min(10, args.steps // 2)))
    e2e = None if args.no_e2e else end_to_end(rd, torch, tb, dev, world, barrier, args.steps)
    faithful = None
    if not args.no_faithful and world == 1 and p > 1:
        faithful = tb.faithful()
    config = tb.describe(world)
    roof = roofline_block(tb, kernel_ms, timed_over) if rank == 0 else None
    gpu_launches = args.steps * tb.launches_per_step
    reductions_per_step, create_ms = tb.reduces_per_step, tb.create_ms
    tb.close()

    # the small-message workload (4 MiB per process, four schedules): one batch launch per step, two streams
    small = None
    if not args.no_small and world == 1 and wname != "config2":
        w2 = WORKLOADS["config2"]
        tb2 = TreeBench(rd, torch, "config2", w2, dev, "batch", 2)
        steps2 = 200
        v2, ms2, k2, over2, _, _ = measure(tb2, steps2, 10, barrier, dev, world, False, local_rank)
        small = {"config": tb2.describe(world), "value": v2, "unit": "GB/s", "steps": steps2, "ms_per_step": ms2 / steps2,
                 "roofline": roofline_block(tb2, k2, over2), "per_schedule_gbs": tb2.per_schedule(20),
                 "schedule_create_ms": tb2.create_ms,
                 "faithful": None if args.no_faithful else tb2.faithful()}
        tb2.close()

    if rank == 0:
        cpu = None
        if not args.no_cpu_baseline and world == 1:
            cpu = cpu_baseline(w, wname, 20.0)
        peak = roof["peak"]
        line = {
            "metric": "reduction_throughput", "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "ms_per_step_spread": spread, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "i32" if w["dist"].startswith("int") else "f32", "data": "synthetic",
            "config": config, "roofline": roof, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": gpu_launches, "clocks": clocks,
            "reductions_per_step": reductions_per_step, "per_schedule_gbs": per_schedule, "schedule_create_ms": create_ms,
            "oracle_schedule_ms": cpu["oracle_schedule_ms"] if cpu else None,
            "faithful": faithful, "config2_batch": small,
            "percent_of_peak": {"measured_copy": 100 * value / peak, "nominal_8TBs": 100 * value / 8000.0},
        }
        print(json.dumps(line), flush=True)
    if dist_on:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
