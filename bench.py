#!/usr/bin/env python
"""Throughput of the schedule-exact reduction on B200: `python bench.py --gpus N --steps K --warmup W`.

A step is one pass of the reduction path over one batch of synthetic inputs: for every schedule the
workload names, one tree-mode rd_reduce of the p resident messages (fp32) into the root buffer.
The schedules themselves (cost model, event generation, combine programs) are plans built once and
reused; their build time is reported beside the throughput.  Metric: reduction GB/s, counting
p*m input bytes plus m output bytes per reduction.

One JSON line is printed by rank 0.  With N > 1 every rank runs an independent replica on its own
GPU (the path needs no exchange between GPUs); times are taken on the device and the slowest rank
counts.  `--impl reference` times the plain CPU checker instead, on rank 0 only.
"""
from __future__ import annotations

import argparse
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


# DRAM bytes per launch of the streaming kernel from ncu captures (profiles/rd_tree_stream_kernel_config2.md):
# dram__bytes_read.sum + dram__bytes_write.sum, mean of three launches, for the batch launch (four reductions)
# and for a single reduction's launch.  Reported only while the kernel source is the one that was profiled.
NCU_TRAFFIC = {"workload": "config2",
               "bytes_per_launch": {"calls": 274.7e6, "batch": 1092.1e6},
               "kernel_sha256": "cc2287fe4fcf0d6eb3ff8444d5d1dc9a5e8ee665a02ed9fae7100b7b86535525"}


def profiled_traffic(wname, issue):
    import hashlib
    try:
        with open(os.path.join(ROOT, "paper_1310_4645_b200", "csrc", "rd_kernels.cu"), "rb") as f:
            same = hashlib.sha256(f.read()).hexdigest() == NCU_TRAFFIC["kernel_sha256"]
    except OSError:
        same = False
    return NCU_TRAFFIC["bytes_per_launch"][issue] if same and wname == NCU_TRAFFIC["workload"] else None


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


def oracle_events(rdmod, algo_name, bidir, p, msg_bytes, seg_bytes, model):
    """Events, offsets for the CPU checker (used by the reference arm and the cpu_baseline leg only)."""
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


def cpu_pass(w, wname, x_host, budget_s, max_passes):
    """Times the CPU checker's reduction on the workload (or a slab of whole segments of it when one pass
    would exceed the budget).  Returns (GB/s, description, cores)."""
    import numpy as np
    from oracle import rd_oracle as O
    p, n = x_host.shape
    model = (w["alpha"], w["beta"], w["gamma"])
    plans = []
    for label, algo_name, bidir in WORKLOAD_SCHEDULES[wname]:
        ev, off = oracle_events(None, algo_name, bidir, p, 4 * n, w["seg_bytes"], model)
        plans.append((ev, off))
    bytes_per_pass = len(plans) * len(WORKLOAD_OPS[wname]) * (p + 1) * n * 4
    t_total, passes = 0.0, 0
    while passes < max_passes and (passes == 0 or t_total < budget_s):
        t0 = time.perf_counter()
        for ev, off in plans:
            for op in WORKLOAD_OPS[wname]:
                O.reduce(ev, x_host, off, op)
        t_total += time.perf_counter() - t0
        passes += 1
    return bytes_per_pass * passes / t_total / 1e9, passes, t_total


def host_slab(w, wname, max_bytes):
    """Host copy of the workload, or of its first whole segments when it exceeds max_bytes."""
    from paper_1310_4645_b200.inputs import make_inputs
    p, n = w["p"], w["n"]
    seg = w["seg_bytes"] // 4
    if p * n * 4 > max_bytes:
        n = max(seg, (max_bytes // (4 * p)) // seg * seg)
    return make_inputs(p, n, w["dist"], w["seed"], device="cpu"), n


def run_reference(args, wname, w):
    """The CPU checker as it stands, timed on the host cores: one step = one pass over a bounded slab."""
    import torch
    x, n = host_slab(w, wname, 1 << 30)
    xh = x.numpy()
    slab = dict(w, n=n)
    for _ in range(args.warmup):
        cpu_pass(slab, wname, xh, 0.0, 1)
    t0 = time.perf_counter()
    gb = 0.0
    for _ in range(args.steps):
        v, passes, dt = cpu_pass(slab, wname, xh, 0.0, 1)
        gb += v * dt
    dt = time.perf_counter() - t0
    value = gb / dt
    sample = "each step: every schedule x op of the workload on the first %d of %d elements per process" % (n, w["n"])
    line = {"impl": "reference", "metric": "reduction_throughput", "value": value, "unit": "GB/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "i32" if w["dist"].startswith("int") else "f32", "data": "synthetic",
            "config": {"workload": wname, "p": w["p"], "n_elems": w["n"], "segment_bytes": w["seg_bytes"],
                       "schedules": [s[0] for s in WORKLOAD_SCHEDULES[wname]], "ops": WORKLOAD_OPS[wname]},
            "cpu_baseline": {"value": value, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="config2", choices=sorted(WORKLOAD_SCHEDULES))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-large", action="store_true", help="skip the extra large-message (config4) measurement")
    ap.add_argument("--no-faithful", action="store_true", help="skip the schedule-faithful makespan measurement")
    ap.add_argument("--issue", default="batch", choices=["batch", "calls"],
                    help="batch: a step is one rd_reduce_batch call per operation (one launch for all schedules); "
                         "calls: one rd_reduce call per schedule and operation")
    ap.add_argument("--streams", type=int, default=2, choices=[1, 2],
                    help="CUDA streams the independent reductions of the timed region alternate over (default 2)")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    from paper_1310_4645_b200.inputs import make_inputs, WORKLOADS
    wname = args.workload
    w = WORKLOADS[wname]

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
    bytes_per_reduce = (p + 1) * n * 4
    # default step count: about a second of timed work
    if args.steps is None:
        args.steps = max(20, int(1.0 / (len(WORKLOAD_SCHEDULES[wname]) * len(WORKLOAD_OPS[wname]) * bytes_per_reduce / 5e12)))
    if args.warmup is None:
        args.warmup = max(3, args.steps // 20)
    if args.warmup < 3:
        args.warmup = 3

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist_on = world > 1
    if dist_on:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    model = (w["alpha"], w["beta"], w["gamma"])
    n_plans = len(WORKLOAD_SCHEDULES[wname])
    # Batch issue: every job of a step reads its own messages (jobs of one launch that read the same bytes
    # would meet in L2), and steps that may overlap on two streams read different sets of them.
    batch_sets = max(2, args.streams)
    if args.issue == "batch" and p * n * 4 * n_plans * batch_sets > (48 << 30):
        args.issue = "calls"                # too much memory for a set of messages per job and stream
    # Call issue: the kernel never reads the arena the previous launch read, and two arenas together exceed L2.
    if args.issue == "batch":
        n_arenas = n_plans * batch_sets
    else:
        n_arenas = 3 if p * n * 4 <= (1 << 30) else 1
    arenas = [make_inputs(p, n, w["dist"], w["seed"] + 1000 * a, device=str(dev)) for a in range(n_arenas)]
    out = torch.empty(n, dtype=arenas[0].dtype, device=dev)
    tables = [rd.PointerTable(a) for a in arenas]

    t0 = time.perf_counter()
    plans = []
    for label, algo_name, bidir in WORKLOAD_SCHEDULES[wname]:
        h = rd.rd_schedule_create(rd.ALGOS[algo_name], rd.RD_PORT_BI if bidir else rd.RD_PORT_UNI, p, 4 * n,
                                  w["seg_bytes"], *model)
        plans.append((label, h))
    create_ms = (time.perf_counter() - t0) * 1e3
    for _, h in plans:
        rd.rd_schedule_upload(h)
    ops = [rd.RD_SUM if o == "sum" else rd.RD_MAX for o in WORKLOAD_OPS[wname]]
    reduces_per_step = len(plans) * len(ops)
    launches_per_step = len(ops) if args.issue == "batch" else reduces_per_step

    counter = [0]
    # A step reduces messages under every schedule (and operation) of the workload: independent reductions,
    # each with its own output.
    #   batch issue: one rd_reduce_batch call per operation, i.e. ONE launch of the streaming kernel whose
    #     tiles are those of all the schedules' reductions (each job on its own messages);
    #   call issue: one rd_reduce call per schedule and operation; launch i of the run reads arena i mod n_arenas.
    # Either way the calls alternate over args.streams CUDA streams: with two streams one launch's thread
    # blocks take the SM slots the other frees while its last blocks are still running.
    outs = [torch.empty(n, dtype=arenas[0].dtype, device=dev) for _ in range(reduces_per_step)]
    main_stream = torch.cuda.current_stream(dev)
    side = [torch.cuda.Stream(device=dev) for _ in range(args.streams)] if args.streams > 1 else [main_stream]
    batches = None
    if args.issue == "batch":
        batches = [[rd.Batch([(h, tables[s_ * n_plans + j], outs[k * n_plans + j]) for j, (_, h) in enumerate(plans)])
                    for k in range(len(ops))] for s_ in range(batch_sets)]

    def step(streams):
        if batches is not None:
            for k, op in enumerate(ops):
                c = counter[0]
                rd.rd_reduce_batch(batches[c % batch_sets][k], op, stream=streams[c % len(streams)])
                counter[0] += 1
            return
        i = 0
        for _, h in plans:
            for op in ops:
                rd.rd_reduce(h, tables[counter[0] % n_arenas], outs[i], op, stream=streams[i % len(streams)])
                counter[0] += 1
                i += 1

    def barrier():
        if dist_on:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(streams, steps):
        """Device time of `steps` steps: the events sit on the main stream, the other streams start after
        the first event and the second one waits for them."""
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(main_stream)
        for st in streams:
            if st is not main_stream:
                st.wait_event(e0)
        for _ in range(steps):
            step(streams)
        for st in streams:
            if st is not main_stream:
                done = torch.cuda.Event()
                done.record(st)
                main_stream.wait_event(done)
        e1.record(main_stream)
        return e0, e1

    for _ in range(args.warmup):
        step(side)
    barrier()
    sampler = ClockSampler(visible_gpu_index(local_rank))
    sampler.start()
    e0, e1 = timed(side, args.steps)
    barrier()
    clocks = sampler.stop()
    ms = max_over_ranks(e0.elapsed_time(e1), dev)
    value = replica_throughput(args.steps * reduces_per_step * bytes_per_reduce, ms, world)

    # the kernel by itself: the same launches back to back on ONE stream (what the roofline entry reports)
    if args.streams > 1:
        k_steps = max(3, args.steps // 2)
        for _ in range(3):
            step([main_stream])
        barrier()
        k0, k1 = timed([main_stream], k_steps)
        barrier()
        kernel_ms_per_launch = max_over_ranks(k0.elapsed_time(k1), dev) / (k_steps * launches_per_step)
    else:
        k_steps = args.steps
        kernel_ms_per_launch = ms / (args.steps * launches_per_step)

    # per-schedule throughput (same launches, timed one schedule at a time)
    per_schedule = {}
    for label, h in plans:
        for opname, op in zip(WORKLOAD_OPS[wname], ops):
            reps = max(5, args.steps // 2)
            for _ in range(3):
                rd.rd_reduce(h, tables[counter[0] % n_arenas], out, op); counter[0] += 1
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(reps):
                rd.rd_reduce(h, tables[counter[0] % n_arenas], out, op); counter[0] += 1
            b.record()
            torch.cuda.synchronize()
            per_schedule["%s/%s" % (label, opname)] = round(bytes_per_reduce * reps / (a.elapsed_time(b) * 1e-3) / 1e9, 1)

    # end to end: host buffers in, host result out, through rd_reduce_host
    e2e = None
    if not args.no_e2e:
        e2e_n_plans = plans
        host_bytes = p * n * 4
        if host_bytes <= (8 << 30):
            hx = arenas[0].cpu().pin_memory()
            hout = torch.empty(n, dtype=arenas[0].dtype).pin_memory()
            staging = torch.empty((p + 1) * n, dtype=arenas[0].dtype, device=dev)
            e_steps = max(3, min(args.steps, int(2.0 / (reduces_per_step * host_bytes / 40e9)) or 1))
            for _, h in e2e_n_plans:
                rd.rd_reduce_host(h, hx, hout, staging, ops[0])
            barrier()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(e_steps):
                for _, h in e2e_n_plans:
                    for op in ops:
                        rd.rd_reduce_host(h, hx, hout, staging, op)
            b.record()
            barrier()
            e_ms = max_over_ranks(a.elapsed_time(b), dev)
            e2e = {"value": replica_throughput(e_steps * reduces_per_step * bytes_per_reduce, e_ms, world), "unit": "GB/s",
                   "h2d_bytes_per_step": reduces_per_step * host_bytes, "d2h_bytes_per_step": reduces_per_step * n * 4,
                   "steps": e_steps}
            del hx, hout, staging

    # schedule-faithful execution: measured makespan of every schedule beside the linear model's prediction
    faithful = None
    if not args.no_faithful and world == 1 and p > 1:
        rows = {}
        for label, h in plans:
            spans = []
            for rep in range(7):
                st = rd.rd_reduce(h, tables[rep % n_arenas], out, ops[0], exec_mode=rd.RD_EXEC_FAITHFUL, want_stats=True)
                if rep >= 2:
                    spans.append(st.makespan_ns)
            spans.sort()
            shape = rd.rd_schedule_faithful_shape(h)
            rows[label] = {"measured_us": spans[len(spans) // 2] / 1e3, "best_us": spans[0] / 1e3,
                           "predicted_us": rd.rd_schedule_info(h)["predicted_seconds"] * 1e6,
                           "blocks_per_process": shape["blocks_per_process"], "slots_per_process": shape["slots_per_process"]}
        by_model = sorted(rows, key=lambda k: rows[k]["predicted_us"])
        by_gpu = sorted(rows, key=lambda k: rows[k]["measured_us"])
        faithful = {"schedules": rows, "rank_by_model": by_model, "rank_measured": by_gpu,
                    "ranks_agree": by_model == by_gpu, "fastest_agrees": by_model[0] == by_gpu[0]}

    # the large-message workload (1 GiB per process), measured beside the main one when it fits
    large = None
    if not args.no_large and world == 1 and wname != "config4":
        del arenas, tables
        torch.cuda.empty_cache()
        free_b, _ = torch.cuda.mem_get_info(dev)
        w4 = WORKLOADS["config4"]
        need = (w4["p"] + 1) * w4["n"] * 4
        if free_b > need + (4 << 30):
            x4 = make_inputs(w4["p"], w4["n"], w4["dist"], w4["seed"], device=str(dev))
            t4 = rd.PointerTable(x4)
            out4 = torch.empty(w4["n"], dtype=torch.float32, device=dev)
            m4 = (w4["alpha"], w4["beta"], w4["gamma"])
            res, tot_ms, tot_b = {}, 0.0, 0
            for label, algo_name, bidir in WORKLOAD_SCHEDULES["config4"]:
                h4 = rd.rd_schedule_create(rd.ALGOS[algo_name], rd.RD_PORT_BI if bidir else rd.RD_PORT_UNI, w4["p"],
                                           4 * w4["n"], w4["seg_bytes"], *m4)
                for opname in WORKLOAD_OPS["config4"]:
                    op = rd.RD_SUM if opname == "sum" else rd.RD_MAX
                    for _ in range(3):
                        rd.rd_reduce(h4, t4, out4, op)
                    torch.cuda.synchronize()
                    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    a.record()
                    for _ in range(10):
                        rd.rd_reduce(h4, t4, out4, op)
                    b.record()
                    torch.cuda.synchronize()
                    res["%s/%s" % (label, opname)] = round(need * 10 / (a.elapsed_time(b) * 1e-3) / 1e9, 1)
                    tot_ms += a.elapsed_time(b); tot_b += need * 10
                rd.rd_destroy(h4)
            large = {"workload": "config4", "p": w4["p"], "n_elems": w4["n"], "segment_bytes": w4["seg_bytes"],
                     "value": tot_b / (tot_ms * 1e-3) / 1e9, "unit": "GB/s", "per_schedule_gbs": res,
                     "l2": "inputs (32 GiB) exceed L2"}
            del x4, out4, t4

    if rank == 0:
        peak, peak_src = measured_peak()
        if large:
            large["frac_of_measured_peak"] = large["value"] / peak
            large["frac_of_nominal_8000"] = large["value"] / 8000.0
        bytes_per_launch = bytes_per_reduce * reduces_per_step // launches_per_step
        achieved = bytes_per_launch / (kernel_ms_per_launch * 1e-3) / 1e9
        cpu = None
        if not args.no_cpu_baseline and world == 1:
            x, n_s = host_slab(w, wname, 1 << 30)
            v, passes, dt = cpu_pass(dict(w, n=n_s), wname, x.numpy(), 10.0, 200)
            cpu = {"value": v, "unit": "GB/s", "cores": 1, "kind": "oracle",
                   "sample": "%d passes over every schedule x op on %d of %d elements per process (%.1f s)"
                             % (passes, n_s, n, dt)}
        shape0 = rd.rd_schedule_tree_shape(plans[0][1])
        if args.issue == "batch":                   # the batch launch: all jobs' tiles, the deepest stack among them
            tiles = sum(rd.rd_schedule_tree_shape(h)["n_tiles"] for _, h in plans)
            shape0 = dict(variant=rd.RD_TREE_STREAM, n_tiles=tiles, blocks_per_sm="chosen for the batch's tiles and deepest stack",
                          ring_stages="chosen for the batch's tiles and deepest stack")
        line = {
            "metric": "reduction_throughput", "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "i32" if w["dist"].startswith("int") else "f32", "data": "synthetic",
            "config": {"workload": wname, "p": p, "n_elems": n, "segment_bytes": w["seg_bytes"],
                       "schedules": [s[0] for s in WORKLOAD_SCHEDULES[wname]], "ops": WORKLOAD_OPS[wname],
                       "bytes_counted": "p*m + m per reduction",
                       "issue": ("a step is one rd_reduce_batch call per operation: one launch for the step's %d independent "
                                 "reductions, each on its own messages; steps alternate over %d CUDA stream(s) and %d sets of messages"
                                 % (n_plans, args.streams, batch_sets)) if args.issue == "batch" else
                                "the step's independent reductions are separate rd_reduce calls that alternate over %d CUDA stream(s)" % args.streams,
                       "l2": "a launch reads %.0f MiB that no launch running beside it reads (%d arenas of %.0f MiB)"
                             % (n_plans * p * n * 4 / 2**20, n_arenas, p * n * 4 / 2**20) if args.issue == "batch" else
                             "inputs rotate over %d arenas of %.0f MiB each (> L2 between reuses)" % (n_arenas, p * n * 4 / 2**20)
                             if n_arenas > 1 else "inputs (%.1f GiB) exceed L2" % (p * n * 4 / 2**30),
                       "parallelism": "replicas only" if world > 1 else "single GPU"},
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": profiled_traffic(wname, args.issue), "traffic_unit": "bytes per launch", "algorithmic_bytes": bytes_per_launch,
                         "peak_source": peak_src,
                         "kernel": "rd_tree_direct_kernel" if shape0["variant"] == rd.RD_TREE_DIRECT else "rd_tree_stream_kernel",
                         "launch_shape": {"blocks_per_sm": shape0["blocks_per_sm"], "ring_stages": shape0["ring_stages"],
                                          "tiles": shape0["n_tiles"]},
                         "timed_over": "%d launches back to back on one stream, %.2f us each" % (k_steps * launches_per_step, kernel_ms_per_launch * 1e3),
                         "frac_of_nominal_8000": achieved / 8000.0},
            "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": args.steps * launches_per_step, "clocks": clocks,
            "reductions_per_step": reduces_per_step,
            "per_schedule_gbs": per_schedule, "schedule_create_ms": create_ms, "large_message": large, "faithful": faithful,
            "percent_of_peak": {"measured_copy": 100 * value / peak, "nominal_8TBs": 100 * value / 8000.0},
        }
        print(json.dumps(line), flush=True)
    for _, h in plans:
        rd.rd_destroy(h)
    if dist_on:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
