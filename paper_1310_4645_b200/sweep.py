"""Sweep of the tree-mode reduction over process counts, message sizes, element types, operations and
schedules, every schedule at its own optimal segment size (the paper tunes each algorithm's segment
size before comparing, Sections V-B and VII).

    python -m paper_1310_4645_b200.sweep --out sweep.jsonl [--max-total-gib 64] [--reps 5]

For every case one JSON line: shape, segment size chosen, the schedule's predicted completion time
under the linear model, measured microseconds and GB/s ((p+1)*m bytes per reduction), and whether the
result passed its check (integers, max and min: exact against torch's order-free result; fp32 sum:
|r - r64| <= 1e-5 * sum|x| against an fp64 sum, fp64 sum: the same with 1e-14, bf16 sum: the fp32 bound plus
one rounding, 2^-8 |r64|; on the whole message or on sampled slices of it).
These checks are order free and run on every one of the thousands of cases; the bit-for-bit comparison with the CPU
checker at these same tuned segment sizes is made by the test suite on a thinned grid of the cells.
Inputs: uniform random numbers from seed 4 (integers in [-2^20, 2^20], floating point in [-1, 1)), one
arena per element type (--dtypes), every case a view of its first p*n elements.
"""
from __future__ import annotations

import argparse
import json
import sys
import time

import torch

from . import binding as rd

ALPHA, BETA, GAMMA = 2e-6, 1e-10, 5e-11
TORCH_DTYPES = {"int32": torch.int32, "fp32": torch.float32, "int64": torch.int64, "fp64": torch.float64,
                "bf16": torch.bfloat16, "fp16": torch.float16}
ELEM_BYTES = {"int32": 4, "fp32": 4, "int64": 8, "fp64": 8, "bf16": 2, "fp16": 2}
SCHEDULES = [("uni_greedy", rd.RD_UNI_GREEDY, rd.RD_PORT_UNI), ("bi_greedy", rd.RD_BI_GREEDY, rd.RD_PORT_BI),
             ("binomial", rd.RD_BINOMIAL, rd.RD_PORT_UNI), ("pipeline", rd.RD_PIPELINE, rd.RD_PORT_UNI),
             ("binary", rd.RD_BINARY, rd.RD_PORT_UNI), ("butterfly", rd.RD_BUTTERFLY, rd.RD_PORT_BI)]


def fill_arena(n_elems, dtype, dev):
    gen = torch.Generator(device=dev)
    gen.manual_seed(4)
    arena = torch.empty(n_elems, dtype=dtype, device=dev)
    step = 1 << 28
    for lo in range(0, n_elems, step):
        part = arena[lo:lo + step]
        if dtype in (torch.int32, torch.int64):
            part.random_(-(1 << 20), (1 << 20) + 1, generator=gen)
        else:
            part.uniform_(-1.0, 1.0, generator=gen)
    return arena


def check(x, out, op, max_check_elems=1 << 22):
    """Order-free check on the whole message when small, else on the first, middle and last slices."""
    p, n = x.shape
    per = max(1, max_check_elems // p)
    spans = [(0, n)] if n <= 3 * per else [(0, per), ((n - per) // 2, (n - per) // 2 + per), (n - per, n)]
    for lo, hi in spans:
        xs, o = x[:, lo:hi], out[lo:hi]
        if op in ("max", "min"):
            if not torch.equal(o, xs.amax(dim=0) if op == "max" else xs.amin(dim=0)):
                return False
        elif x.dtype == torch.int64:
            if not torch.equal(o, xs.sum(dim=0)):
                return False
        elif x.dtype == torch.int32:
            want = xs.to(torch.int64).sum(dim=0)
            want = ((want + (1 << 31)) % (1 << 32) - (1 << 31)).to(torch.int32)
            if not torch.equal(o, want):
                return False
        else:
            ref = xs.to(torch.float64).sum(dim=0)
            mag = xs.to(torch.float64).abs().sum(dim=0)
            tol = (1e-14 if x.dtype == torch.float64 else 1e-5) * mag
            if x.dtype == torch.bfloat16:           # combined in fp32, then one rounding to 8 significant bits
                tol = tol + 2.0 ** -8 * ref.abs()
            if x.dtype == torch.float16:            # ... to 11 significant bits (inputs in [-1, 1): no overflow)
                tol = tol + 2.0 ** -11 * ref.abs() + 2.0 ** -24
            if not bool(((o.to(torch.float64) - ref).abs() <= tol).all()):
                return False
    return True


def copy_reference(args, dev, sink):
    """What a kernel that only copies reaches at the launch sizes of the sweep's largest messages: one JSON line per
    p with the median and best GB/s (bytes read plus bytes written) of 5 loops of 20 back-to-back copies that rotate
    over three destinations."""
    m = 1 << args.max_log2_bytes
    for p in args.p:
        nbytes = (p + 1) * m // 2 // 4 * 4
        if 4 * nbytes > int(args.max_total_gib * (1 << 30)):
            continue
        src = torch.empty(nbytes // 4, dtype=torch.float32, device=dev).normal_()
        dst = [torch.empty_like(src) for _ in range(3)]
        for i in range(5):
            dst[i % 3].copy_(src)
        torch.cuda.synchronize()
        rates = []
        for _ in range(5):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for i in range(20):
                dst[i % 3].copy_(src)
            b.record()
            torch.cuda.synchronize()
            rates.append(2 * nbytes * 20 / (a.elapsed_time(b) * 1e-3) / 1e9)
        rates.sort()
        sink.write(json.dumps({"copy_reference": True, "p": p, "msg_bytes": m, "traffic_bytes": 2 * nbytes,
                               "gbs_median": rates[2], "gbs_best": rates[-1]}) + "\n")
        sink.flush()
        del src, dst
        torch.cuda.empty_cache()


def allreduce_timing(args, dev, sink):
    """rd_allreduce for every p at the largest message size: one JSON line per p with the time of both kernels together,
    GB/s counting (p + 1) m bytes for the reduce plus m read and (p - 1) m written by the broadcast, and a check that
    every process's copy equals the root's and the root's passes the order-free check."""
    m = 1 << args.max_log2_bytes
    n = m // 4
    for p in args.p:
        if 2 * p * m > int(args.max_total_gib * (1 << 30)):
            continue
        x = fill_arena(p * n, torch.float32, dev).view(p, n)
        outs = torch.empty_like(x)
        seg = rd.rd_optimal_segment(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, p, m, ALPHA, BETA, GAMMA)
        h = rd.rd_schedule_create(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, p, m, seg, ALPHA, BETA, GAMMA)
        try:
            tin, tout = rd.PointerTable(x), rd.PointerTable(outs)
            rd.rd_allreduce(h, tin, tout, rd.RD_SUM)
            ok = check(x, outs[0], "sum") and all(torch.equal(outs[i], outs[0]) for i in range(1, p))
            us = float("inf")
            for _ in range(3):                                   # the best of three runs of 4 * reps calls each
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                for _ in range(4 * args.reps):
                    rd.rd_allreduce(h, tin, tout, rd.RD_SUM)
                b.record()
                torch.cuda.synchronize()
                us = min(us, a.elapsed_time(b) * 1e3 / (4 * args.reps))
            moved = (p + 1) * m + (p * m if p > 1 else 0)
            sink.write(json.dumps({"allreduce": True, "p": p, "msg_bytes": m, "seg_bytes": seg, "measured_us": us,
                                   "bytes_moved": moved, "gbs": moved / us / 1e3, "ok": ok}) + "\n")
            sink.flush()
        finally:
            rd.rd_destroy(h)
        del x, outs
        torch.cuda.empty_cache()


def main(argv=None):
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--out", default="-")
    ap.add_argument("--max-total-gib", type=float, default=64.0, help="skip cases whose p*m exceeds this")
    ap.add_argument("--reps", type=int, default=5)
    ap.add_argument("--p", type=int, nargs="*", default=[2 ** k for k in range(1, 11)])
    ap.add_argument("--min-log2-bytes", type=int, default=3)
    ap.add_argument("--max-log2-bytes", type=int, default=26)
    ap.add_argument("--faithful", action="store_true",
                    help="also run every schedule in schedule-faithful mode (fp32 sum) and record its makespan")
    ap.add_argument("--dtypes", nargs="*", default=["int32", "fp32"], choices=list(TORCH_DTYPES))
    ap.add_argument("--ops", nargs="*", default=["sum", "max"], choices=["sum", "max", "min"])
    ap.add_argument("--schedules", nargs="*", default=[s[0] for s in SCHEDULES], choices=[s[0] for s in SCHEDULES])
    ap.add_argument("--copy-reference", action="store_true",
                    help="instead of the sweep: time a plain device-to-device copy (torch copy_) whose traffic, read plus written, "
                         "is that of a reduction of p messages of the largest size, (p + 1) * m bytes, for every p")
    ap.add_argument("--allreduce", action="store_true",
                    help="instead of the sweep: time rd_allreduce (the reduce, then the broadcast of the root's result to every "
                         "process) for every p at the largest message size, uni-greedy at its tuned segment size, fp32 sum")
    ap.add_argument("--variant", default="auto", choices=["auto", "stream", "paired", "direct"],
                    help="tree-mode kernel: the library's choice, the streaming kernel with one / two operand tiles per ring stage, or "
                         "the direct kernel (at most 8 processes; the library falls back to the streaming kernel where it does not apply)")
    args = ap.parse_args(argv)
    dev = torch.device("cuda", torch.cuda.current_device())
    sink = sys.stdout if args.out == "-" else open(args.out, "w")
    if args.copy_reference or args.allreduce:
        (copy_reference if args.copy_reference else allreduce_timing)(args, dev, sink)
        if sink is not sys.stdout:
            sink.close()
        return 0
    sizes = [1 << k for k in range(args.min_log2_bytes, args.max_log2_bytes + 1)]
    limit = int(args.max_total_gib * (1 << 30))
    biggest = max(p * m for p in args.p for m in sizes if p * m <= limit)
    want = list(args.dtypes) + (["fp32"] if args.faithful and "fp32" not in args.dtypes else [])
    arenas = {dt: fill_arena(biggest // ELEM_BYTES[dt], TORCH_DTYPES[dt], dev) for dt in want}
    out_buf = {dt: torch.empty(max(sizes) // ELEM_BYTES[dt], dtype=TORCH_DTYPES[dt], device=dev) for dt in want}
    opcodes = {"sum": rd.RD_SUM, "max": rd.RD_MAX, "min": rd.RD_MIN}
    n_cases = n_bad = 0
    t_start = time.time()
    for p in args.p:
        for m in sizes:
            if p * m > limit:
                continue
            n = m // 4
            for name, algo, port in SCHEDULES:
                if name not in args.schedules:
                    continue
                t0 = time.perf_counter()
                seg = rd.rd_optimal_segment(algo, port, p, m, ALPHA, BETA, GAMMA)
                if any(ELEM_BYTES[dt] == 8 for dt in args.dtypes):
                    seg = min(m, (seg + 7) // 8 * 8)       # whole elements of every type
                h = rd.rd_schedule_create(algo, port, p, m, seg, ALPHA, BETA, GAMMA)
                create_ms = (time.perf_counter() - t0) * 1e3
                info = rd.rd_schedule_info(h)
                rd.rd_schedule_upload(h)
                if args.variant != "auto":
                    rd.rd_schedule_set_tree_variant(h, {"stream": rd.RD_TREE_STREAM, "paired": rd.RD_TREE_STREAM_PAIRED,
                                                        "direct": rd.RD_TREE_DIRECT}[args.variant])
                try:
                    if args.faithful and p > 1:
                        x = arenas["fp32"][: p * n].view(p, n)
                        out = out_buf["fp32"][:n]
                        tab = rd.PointerTable(x)
                        rec = {"faithful": True, "p": p, "msg_bytes": m, "schedule": name, "seg_bytes": seg, "q": info["q"],
                               "predicted_us": info["predicted_seconds"] * 1e6}
                        try:
                            spans = []
                            for rep in range(4):
                                st = rd.rd_reduce(h, tab, out, rd.RD_SUM, exec_mode=rd.RD_EXEC_FAITHFUL, want_stats=True)
                                if rep:
                                    spans.append(st.makespan_ns)
                            spans.sort()
                            rec.update(makespan_us=spans[len(spans) // 2] / 1e3, ok=check(x, out, "sum"))
                            n_bad += 0 if rec["ok"] else 1
                        except rd.RdError as e:            # scratch does not fit beside the arenas, or too many processes
                            if e.status not in (rd.RD_ERR_NOMEM, rd.RD_ERR_UNSUPPORTED):
                                raise
                            rec.update(skipped=rd.rd_strerror(e.status))
                        sink.write(json.dumps(rec) + "\n")
                        n_cases += 1
                    for dt in args.dtypes:
                        ne = m // ELEM_BYTES[dt]
                        x = arenas[dt][: p * ne].view(p, ne)
                        out = out_buf[dt][:ne]
                        tab = rd.PointerTable(x)
                        if ELEM_BYTES[dt] == 8 and name == "butterfly" and ne % (1 << (p.bit_length() - 1)):
                            continue                       # halving would cut through an element
                        for op, opc in ((o, opcodes[o]) for o in args.ops):
                            rd.rd_reduce(h, tab, out, opc)
                            ok = check(x, out, op)
                            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                            a.record()
                            for _ in range(args.reps):
                                rd.rd_reduce(h, tab, out, opc)
                            b.record()
                            torch.cuda.synchronize()
                            us = a.elapsed_time(b) * 1e3 / args.reps
                            rec = {"p": p, "msg_bytes": m, "dtype": dt, "op": op, "schedule": name, "seg_bytes": seg,
                                   "q": info["q"], "predicted_us": info["predicted_seconds"] * 1e6, "measured_us": us,
                                   "gbs": (p + 1) * m / us / 1e3, "ok": ok, "create_ms": create_ms,
                                   "cache": "L2 resident (inputs re-read every repetition)" if p * m < (96 << 20) else "HBM"}
                            sink.write(json.dumps(rec) + "\n")
                            n_cases += 1
                            n_bad += 0 if ok else 1
                finally:
                    rd.rd_destroy(h)
        sink.flush()
    summary = {"summary": True, "cases": n_cases, "failed_checks": n_bad, "seconds": time.time() - t_start}
    sink.write(json.dumps(summary) + "\n")
    if sink is not sys.stdout:
        sink.close()
        print(json.dumps(summary))
    return 1 if n_bad else 0


if __name__ == "__main__":
    sys.exit(main())
