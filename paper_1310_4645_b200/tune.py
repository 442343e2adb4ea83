"""Every schedule tuned by measurement, then compared (the procedure of Section VII).

The paper compares the algorithms "each optimally tuned": for a message of m bytes it runs every segment
size 2^i, keeps the best time per algorithm (each time the minimum of 10 runs), and plots the tuned times
against the message size.  This tool does the same on one GPU with the schedule-faithful kernel, in which
thread-block groups play the processes:

  1. fit (alpha', beta') to the kernel as `calibrate` does (the greedy schedules depend on the model's
     ratio of start-up to per-byte cost, so they are generated under the fitted one);
  2. for every message size and schedule, run the power-of-two segment sizes (from --min-seg-bytes, and
     never more than --max-segments segments) plus the unsegmented message, min over --reps runs each;
  3. print, per message size, each schedule's best segment size and time, the segment size the model
     would have chosen with its measured time, and the ranking of the tuned schedules.

    python -m paper_1310_4645_b200.tune [--p 64] [--min-log2-bytes 12] [--max-log2-bytes 24] [--out tune.jsonl]

Binomial and butterfly are run as the paper defines them (Sections III and IV: whole messages, respectively
halves), without a segment search.
"""
from __future__ import annotations

import argparse
import json
import sys

import numpy as np
import torch

from . import binding as rd
from .calibrate import pair_durations

SEGMENTED = [("uni_greedy", rd.RD_UNI_GREEDY, rd.RD_PORT_UNI), ("bi_greedy", rd.RD_BI_GREEDY, rd.RD_PORT_BI),
             ("pipeline", rd.RD_PIPELINE, rd.RD_PORT_BI), ("binary", rd.RD_BINARY, rd.RD_PORT_BI)]
WHOLE = [("binomial", rd.RD_BINOMIAL, rd.RD_PORT_UNI), ("butterfly", rd.RD_BUTTERFLY, rd.RD_PORT_BI)]


def best_of(algo, port, p, m, seg, model, x, out, reps):
    """Minimum makespan over reps runs (seconds) after two warm-up runs, and the number of segments."""
    h = rd.rd_schedule_create(algo, port, p, m, seg, *model)
    try:
        q = rd.rd_schedule_info(h)["q"]
        best = float("inf")
        for rep in range(reps + 2):
            st = rd.rd_reduce(h, x, out, rd.RD_SUM, exec_mode=rd.RD_EXEC_FAITHFUL, want_stats=True)
            if rep >= 2:
                best = min(best, st.makespan_ns * 1e-9)
        return best, q
    finally:
        rd.rd_destroy(h)


def fit_model(p, m, x, out):
    sizes = [s for s in (4 << 10, 16 << 10, 64 << 10, 256 << 10, 1 << 20) if s <= m]
    dur = np.asarray([pair_durations(p, m, s, x, out) for s in sizes])
    A = np.stack([np.ones(len(sizes)), np.asarray(sizes, dtype=np.float64)], axis=1)
    (alpha, beta), *_ = np.linalg.lstsq(A / dur[:, None], np.ones(len(sizes)), rcond=None)
    return max(float(alpha), 1e-9), max(float(beta), 1e-15), 0.0


def main(argv=None):
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--p", type=int, default=64)
    ap.add_argument("--min-log2-bytes", type=int, default=12)
    ap.add_argument("--max-log2-bytes", type=int, default=24)
    ap.add_argument("--min-seg-bytes", type=int, default=1024)
    ap.add_argument("--max-segments", type=int, default=1024)
    ap.add_argument("--reps", type=int, default=10)
    ap.add_argument("--seed", type=int, default=1)
    ap.add_argument("--out", default="-")
    args = ap.parse_args(argv)
    p = args.p
    biggest = 1 << args.max_log2_bytes
    gen = torch.Generator(device="cuda").manual_seed(args.seed)
    arena = torch.empty((p, biggest // 4), dtype=torch.float32, device="cuda").normal_(generator=gen)
    out_full = torch.empty(biggest // 4, dtype=torch.float32, device="cuda")
    fit_m = min(biggest, 4 << 20)
    model = fit_model(p, fit_m, arena[:, : fit_m // 4].contiguous(), out_full[: fit_m // 4])
    sink = sys.stdout if args.out == "-" else open(args.out, "w")
    sink.write(json.dumps({"fitted": {"alpha_s": model[0], "beta_s_per_byte": model[1], "gamma_s_per_byte": 0.0}, "p": p}) + "\n")
    agree = total = bad = 0
    for k in range(args.min_log2_bytes, args.max_log2_bytes + 1):
        m = 1 << k
        x = arena[:, : m // 4].contiguous()
        out = out_full[: m // 4]
        want = x.sum(dim=0, dtype=torch.float64)
        mag = x.abs().sum(dim=0, dtype=torch.float64)
        row = {"msg_bytes": m, "schedules": {}}
        for name, algo, port in SEGMENTED:
            tried = {}
            seg = m
            while seg >= max(args.min_seg_bytes, 4) and m // seg <= args.max_segments:
                tried[seg] = best_of(algo, port, p, m, seg, model, x, out, args.reps)[0]
                seg //= 2
            best_seg = min(tried, key=tried.get)
            model_seg = rd.rd_optimal_segment(algo, port, p, m, *model)
            model_time, _ = best_of(algo, port, p, m, model_seg, model, x, out, args.reps)
            ok = bool(((out.to(torch.float64) - want).abs() <= 1e-5 * mag).all())
            row["schedules"][name] = {"best_seg_bytes": best_seg, "best_us": tried[best_seg] * 1e6,
                                      "model_seg_bytes": model_seg, "model_seg_us": model_time * 1e6,
                                      "tried_us": {str(s): t * 1e6 for s, t in tried.items()}, "ok": ok}
        for name, algo, port in WHOLE:
            t, _ = best_of(algo, port, p, m, 0 if algo == rd.RD_BUTTERFLY else m, model, x, out, args.reps)
            ok = bool(((out.to(torch.float64) - want).abs() <= 1e-5 * mag).all())
            row["schedules"][name] = {"best_seg_bytes": None, "best_us": t * 1e6, "ok": ok}
        order = sorted(row["schedules"], key=lambda n: row["schedules"][n]["best_us"])
        row["rank_tuned"] = order
        row["greedy_is_fastest"] = order[0] in ("uni_greedy", "bi_greedy")
        total += 1
        agree += 1 if row["greedy_is_fastest"] else 0
        bad += sum(0 if v["ok"] else 1 for v in row["schedules"].values())
        sink.write(json.dumps(row) + "\n")
        sink.flush()
    summary = {"summary": True, "message_sizes": total, "greedy_fastest_in": agree, "failed_checks": bad}
    sink.write(json.dumps(summary) + "\n")
    if sink is not sys.stdout:
        sink.close()
        print(json.dumps(summary))
    return 1 if bad else 0


if __name__ == "__main__":
    sys.exit(main())
