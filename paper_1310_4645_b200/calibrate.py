"""Fit the linear model's parameters to this GPU and re-rank the schedules with them.

The paper compares schedules under a linear cost model (alpha + beta*s per message, gamma*s per
combine, Section II) and notes that the machine's parameters decide which algorithm wins and have to
be tuned (Sections III and VII).  This tool measures them for the schedule-faithful kernel, in which
thread-block groups play the processes:

  1. run the (one-port) pipeline schedule for several segment sizes and read the per-pair time stamps
     (rd_schedule_trace): duration of a pair = data available -> combined segment written;
  2. least-squares fit  duration = alpha' + b' * segment_bytes.  With one port the sender is held until
     the receiver has combined, so the whole per-byte cost is charged to the communication:
     beta' = b', gamma' = 0 (the "one-port fit", which the tuning tool uses);
  3. separate the combine from the hand-off with a second, two-port run of the same pipeline.  In the
     model a process in the middle of a pipeline handles one segment per period, and the period is
     2 t_comm + t_comp with one port (it cannot send and receive at once, Table I) but t_comm + t_comp
     with two (Table III).  The periods P1(s), P2(s) are read off the root's time stamps (median distance
     between consecutive segments) and fitted as lines in s; then t_comm = P1 - P2 and t_comp = 2 P2 - P1,
     i.e. alpha' = a1 - a2, beta' = b1 - b2, gamma' = 2 b2 - b1 (what is left of the constant term,
     2 a2 - a1, has no place in the model and is printed as `unmodelled_constant_s`).  Values that come
     out negative are set to zero;
  4. build every schedule again under (alpha', beta', gamma') of step 2 and of step 3, each with its
     optimal segment size, run it, and print predicted and measured makespans and the two rankings.

    python -m paper_1310_4645_b200.calibrate [--p 64] [--msg-bytes 4194304]
"""
from __future__ import annotations

import argparse
import json
import sys

import numpy as np
import torch

from . import binding as rd

ONE_PORT = [("uni_greedy", rd.RD_UNI_GREEDY), ("binomial", rd.RD_BINOMIAL), ("pipeline", rd.RD_PIPELINE),
            ("binary", rd.RD_BINARY)]


def pair_durations(p, msg_bytes, seg_bytes, x, out, reps=3):
    """Median over pairs and repetitions of (combine written - data available), in seconds."""
    h = rd.rd_schedule_create(rd.RD_PIPELINE, rd.RD_PORT_UNI, p, msg_bytes, seg_bytes, 2e-6, 1e-10, 5e-11)
    try:
        med = []
        for _ in range(reps):
            rd.rd_reduce(h, x, out, rd.RD_SUM, exec_mode=rd.RD_EXEC_FAITHFUL, want_stats=True)
            t = rd.rd_schedule_trace(h).astype(np.float64)
            ev = rd.rd_schedule_events(h)
            full = ev["seg"] < (msg_bytes // seg_bytes)            # leave a shorter last segment out
            med.append(np.median((t[full, 2] - t[full, 1]) * 1e-9))
        return float(np.median(med))
    finally:
        rd.rd_destroy(h)


def pipeline_period(p, msg_bytes, seg_bytes, port, x, out, reps=3):
    """Median distance in time between the root's consecutive segments in a pipeline run, in seconds."""
    h = rd.rd_schedule_create(rd.RD_PIPELINE, port, p, msg_bytes, seg_bytes, 2e-6, 1e-10, 5e-11)
    try:
        med = []
        for _ in range(reps):
            rd.rd_reduce(h, x, out, rd.RD_SUM, exec_mode=rd.RD_EXEC_FAITHFUL, want_stats=True)
            t = rd.rd_schedule_trace(h).astype(np.float64)
            ev = rd.rd_schedule_events(h)
            at_root = np.flatnonzero((ev["dst"] == 0) & (ev["seg"] < (msg_bytes // seg_bytes)))
            done = np.sort(t[at_root, 2])
            if len(done) >= 3:
                med.append(np.median(np.diff(done)) * 1e-9)
        return float(np.median(med)) if med else float("nan")
    finally:
        rd.rd_destroy(h)


def fit_line(sizes, values):
    """Relative least squares of values = a + b * sizes (small segments, which fix a, count as much as large ones)."""
    sizes, values = np.asarray(sizes, dtype=np.float64), np.asarray(values, dtype=np.float64)
    A = np.stack([np.ones(len(sizes)), sizes], axis=1)
    wgt = 1.0 / values
    (a, b), *_ = np.linalg.lstsq(A * wgt[:, None], values * wgt, rcond=None)
    return float(a), float(b)


def two_port_fit(p, m, sizes, x, out):
    """Step 3 of the module's description.  Returns (alpha', beta', gamma', unmodelled constant, periods)."""
    use = [s for s in sizes if m // s >= 8]                    # a steady state needs some segments
    p1 = [pipeline_period(p, m, s, rd.RD_PORT_UNI, x, out) for s in use]
    p2 = [pipeline_period(p, m, s, rd.RD_PORT_BI, x, out) for s in use]
    if len(use) < 2 or not np.all(np.isfinite(p1 + p2)):
        return None
    a1, b1 = fit_line(use, p1)
    a2, b2 = fit_line(use, p2)
    return (max(a1 - a2, 1e-9), max(b1 - b2, 0.0), max(2 * b2 - b1, 0.0), 2 * a2 - a1,
            {str(s): {"one_port_us": u * 1e6, "two_port_us": v * 1e6} for s, u, v in zip(use, p1, p2)})


def rerank(p, m, model, x, out):
    rows = {}
    for name, algo in ONE_PORT:
        seg = rd.rd_optimal_segment(algo, rd.RD_PORT_UNI, p, m, *model)
        measured, predicted, q = measure(algo, rd.RD_PORT_UNI, p, m, seg, model, x, out)
        rows[name] = {"seg_bytes": seg, "q": q, "predicted_us": predicted * 1e6, "measured_us": measured * 1e6}
    by_model = sorted(rows, key=lambda k: rows[k]["predicted_us"])
    by_gpu = sorted(rows, key=lambda k: rows[k]["measured_us"])
    return {"schedules": rows, "rank_by_model": by_model, "rank_measured": by_gpu,
            "ranks_agree": by_model == by_gpu, "fastest_agrees": by_model[0] == by_gpu[0]}


def measure(algo, port, p, msg_bytes, seg_bytes, model, x, out, reps=5):
    h = rd.rd_schedule_create(algo, port, p, msg_bytes, seg_bytes, *model)
    try:
        spans = []
        for rep in range(reps + 2):
            st = rd.rd_reduce(h, x, out, rd.RD_SUM, exec_mode=rd.RD_EXEC_FAITHFUL, want_stats=True)
            if rep >= 2:
                spans.append(st.makespan_ns * 1e-9)
        info = rd.rd_schedule_info(h)
        return float(np.median(spans)), info["predicted_seconds"], info["q"]
    finally:
        rd.rd_destroy(h)


def main(argv=None):
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--p", type=int, default=64)
    ap.add_argument("--msg-bytes", type=int, default=4 << 20)
    ap.add_argument("--seed", type=int, default=1)
    args = ap.parse_args(argv)
    p, m = args.p, args.msg_bytes
    gen = torch.Generator(device="cuda").manual_seed(args.seed)
    x = torch.empty((p, m // 4), dtype=torch.float32, device="cuda").normal_(generator=gen)
    out = torch.empty(m // 4, dtype=torch.float32, device="cuda")

    sizes = [s for s in (4 << 10, 16 << 10, 64 << 10, 256 << 10, 1 << 20) if s <= m]
    dur = [pair_durations(p, m, s, x, out) for s in sizes]
    A = np.stack([np.ones(len(sizes)), np.asarray(sizes, dtype=np.float64)], axis=1)
    # relative least squares, so that the small segments (which fix alpha') count as much as the large ones
    wgt = 1.0 / np.asarray(dur)
    (alpha, beta), *_ = np.linalg.lstsq(A * wgt[:, None], np.asarray(dur) * wgt, rcond=None)
    alpha, beta = max(float(alpha), 1e-9), max(float(beta), 1e-15)
    fitted = (alpha, beta, 0.0)

    report = {
        "p": p, "msg_bytes": m,
        "pair_time_by_segment_us": {str(s): d * 1e6 for s, d in zip(sizes, dur)},
        "fitted": {"alpha_s": alpha, "beta_s_per_byte": beta, "gamma_s_per_byte": 0.0,
                   "per_process_GBps": 1e-9 / beta},
    }
    report.update(rerank(p, m, fitted, x, out))
    two = two_port_fit(p, m, sizes, x, out)
    if two is not None:
        a2, b2, g2, rest, periods = two
        if b2 + g2 > 0:
            report["two_port_fit"] = {"alpha_s": a2, "beta_s_per_byte": b2, "gamma_s_per_byte": g2, "unmodelled_constant_s": rest,
                                      "pipeline_period_by_segment": periods}
            report["two_port_fit"].update(rerank(p, m, (a2, max(b2, 1e-15), g2), x, out))
    print(json.dumps(report, indent=1))
    return 0


if __name__ == "__main__":
    sys.exit(main())
