"""The library's scheduler (heap / event driven, C++) against the oracle's simulators (plain C):
identical send/receive pairs, start times, segment boundaries and completion time."""
import numpy as np
import pytest

import paper_1310_4645_b200 as rd
from oracle import rd_oracle as O
from helpers import oracle_schedule, ticks

M1 = (2e-6, 1e-10, 5e-11)       # the model of workloads 1-3
M4 = (5e-6, 2.5e-11, 1e-11)     # the model of the large-message workload
PORTS = {rd.RD_UNI_GREEDY: [rd.RD_PORT_UNI], rd.RD_BI_GREEDY: [rd.RD_PORT_BI],
         rd.RD_BINOMIAL: [rd.RD_PORT_UNI, rd.RD_PORT_BI], rd.RD_PIPELINE: [rd.RD_PORT_UNI, rd.RD_PORT_BI],
         rd.RD_BINARY: [rd.RD_PORT_UNI, rd.RD_PORT_BI], rd.RD_BUTTERFLY: [rd.RD_PORT_BI]}


def compare(algo, port, p, msg, seg, model, sizes=None):
    if sizes is None:
        h = rd.rd_schedule_create(algo, port, p, msg, seg, *model)
    else:
        h = rd.rd_schedule_create_segments(algo, port, p, sizes, *model)
    try:
        info = rd.rd_schedule_info(h)
        ev = rd.rd_schedule_events(h)
        off = rd.rd_schedule_segments(h)
    finally:
        rd.rd_destroy(h)
    oev, ooff, ocomp = oracle_schedule(algo, port, p, msg, seg, *model, sizes=sizes)
    assert info["predicted_ticks"] == ocomp
    assert abs(info["predicted_seconds"] - ocomp * 1e-15) <= 1e-12 * max(1.0, ocomp * 1e-15)
    assert (off.astype(np.int64) == np.asarray(ooff, dtype=np.int64)).all()
    assert len(ev) == len(oev)
    for f in ("t_start", "seg", "src", "dst", "kind"):
        assert (ev[f] == oev[f]).all(), f
    return info


@pytest.mark.parametrize("algo", list(PORTS))
def test_grid_of_small_cases(algo):
    for port in PORTS[algo]:
        for p in (1, 2, 3, 4, 5, 7, 8, 13, 16, 31, 32, 33, 64):
            for msg, seg in ((64, 64), (64, 16), (4096, 512), (1000, 96), (36, 4), (4, 4)):
                compare(algo, port, p, msg, seg, M1)
            compare(algo, port, p, 2048, 256, (0.0, 1e-10, 0.0))          # ties everywhere
            compare(algo, port, p, 2048, 256, (1e-6, 0.0, 0.0))


def test_named_workloads():
    """The schedules the benchmark and the parity tests use."""
    assert compare(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, 8, 16384, 2048, M1)["predicted_ticks"] == 39222400000
    for algo in (rd.RD_UNI_GREEDY, rd.RD_BINOMIAL, rd.RD_PIPELINE, rd.RD_BINARY):
        compare(algo, rd.RD_PORT_UNI, 64, 4 << 20, 16 << 10, M1)
    for algo in (rd.RD_BI_GREEDY, rd.RD_BUTTERFLY, rd.RD_BINOMIAL, rd.RD_PIPELINE, rd.RD_BINARY):
        compare(algo, rd.RD_PORT_BI, 256, 16 << 20, 64 << 10, M1)
    compare(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, 32, 1 << 30, 1 << 20, M4)
    info = compare(rd.RD_BI_GREEDY, rd.RD_PORT_BI, 32, 1 << 30, 1 << 20, M4)
    A, B, G = ticks(*M4)
    assert info["predicted_ticks"] == (5 + 1024 - 1) * (A + (B + G) * (1 << 20))   # Table III, bi-greedy row


def test_large_process_counts():
    for algo, port in ((rd.RD_UNI_GREEDY, rd.RD_PORT_UNI), (rd.RD_BI_GREEDY, rd.RD_PORT_BI),
                       (rd.RD_BINARY, rd.RD_PORT_UNI), (rd.RD_BUTTERFLY, rd.RD_PORT_BI)):
        compare(algo, port, 1024, 1 << 16, 1 << 13, M1)
    compare(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, 1000, 40000, 4000, M1)
    compare(rd.RD_BI_GREEDY, rd.RD_PORT_BI, 777, 40000, 4000, M1)


def test_unequal_segmentation():
    """Section VIII: Algorithm 1 for arbitrary segment sizes (paper units scaled to 4-byte elements)."""
    model = (3e-15, 0.25e-15 * 4, 0.25e-15 * 4)     # alpha = 3, beta = gamma = 1 per 4-byte unit, tick 1e-15
    for sizes in ([20, 12, 8], [4, 4, 4, 28], [12, 8, 12, 8], [40]):
        for p in (6, 16, 48):
            compare(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, p, sum(sizes), 0, model, sizes=sizes)
            compare(rd.RD_BI_GREEDY, rd.RD_PORT_BI, p, sum(sizes), 0, model, sizes=sizes)
            compare(rd.RD_PIPELINE, rd.RD_PORT_UNI, p, sum(sizes), 0, model, sizes=sizes)


def test_random_models_and_segmentations():
    """Seeded random cases: process counts around powers of two, equal, ragged and arbitrary segment sizes, models
    with zero terms (many ties).  The library's generators skip work the simulators do (bi-greedy stops visiting
    segments of a length that found no pair at an instant, the fixed trees are emitted or bucketed by round instead
    of sorted), so every shortcut has to reproduce the simulators' pairs exactly."""
    rng = np.random.default_rng(20131017)
    kinds = [(a, port) for a in PORTS if a != rd.RD_BUTTERFLY for port in PORTS[a]] + [(rd.RD_BI_GREEDY, rd.RD_PORT_BI)] * 3
    for _ in range(250):
        algo, port = kinds[int(rng.integers(len(kinds)))]
        p = int(rng.choice([1, 2, 3, 4, 5, 7, 8, 13, 16, 31, 32, 33, 64, 100, 257]))
        q = int(rng.choice([1, 2, 3, 5, 8, 17, 40, 129]))
        how = rng.random()
        if how < 0.4:
            sizes = [4 * int(rng.integers(1, 51))] * q
        elif how < 0.7:
            sizes = [4 * int(rng.integers(1, 51))] * (q - 1) + [4 * int(rng.integers(1, 51))]
        else:
            sizes = [4 * int(s) for s in rng.integers(1, 51, size=q)]
        A, B, G = int(rng.choice([0, 1, 3, 10, 1000, 12345])), int(rng.choice([0, 1, 2, 7, 100])), int(rng.choice([0, 0, 1, 3, 50]))
        if A == 0 and B == 0:
            B = 1
        compare(algo, port, p, sum(sizes), 0, (A * 1e-15, B * 1e-15, G * 1e-15), sizes=sizes)


def test_library_schedules_pass_the_oracle_validator():
    for algo in PORTS:
        for port in PORTS[algo]:
            p, msg, seg = 16, 4096, 512
            h = rd.rd_schedule_create(algo, port, p, msg, seg, *M1)
            ev = rd.rd_schedule_events(h)
            off = rd.rd_schedule_segments(h).astype(np.int64)
            comp = rd.rd_schedule_info(h)["predicted_ticks"]
            rd.rd_destroy(h)
            oev = np.zeros(len(ev), dtype=O.EVENT_DTYPE)
            for f in ("t_start", "seg", "src", "dst", "kind"):
                oev[f] = ev[f]
            sizes = np.diff(off) * 4
            rc, last = O.validate(oev, p, sizes, *ticks(*M1), port == rd.RD_PORT_BI,
                                  tree_rules=algo != rd.RD_BUTTERFLY, in_order=algo == rd.RD_UNI_GREEDY)
            assert rc == 0 and last == comp
            assert O.contributions(oev, p, len(sizes)) == 0
