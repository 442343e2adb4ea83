"""rd_optimal_segment (Tables I and III s_opt rows, Section VII tuning protocol) against the oracle's
simulated completion times."""
import math

import numpy as np
import pytest

import paper_1310_4645_b200 as rd
from oracle import rd_oracle as O
from helpers import oracle_schedule, ticks

M1 = (2e-6, 1e-10, 5e-11)


def oracle_time(algo, port, p, m, s, model):
    return oracle_schedule(algo, port, p, m, s, *model)[2]


@pytest.mark.parametrize("algo,port", [(rd.RD_PIPELINE, rd.RD_PORT_UNI), (rd.RD_PIPELINE, rd.RD_PORT_BI),
                                        (rd.RD_BINARY, rd.RD_PORT_UNI), (rd.RD_BINARY, rd.RD_PORT_BI),
                                        (rd.RD_BI_GREEDY, rd.RD_PORT_BI)])
@pytest.mark.parametrize("p", [4, 8, 64])
@pytest.mark.parametrize("m", [1 << 10, 1 << 14, 1 << 16])
def test_closed_form_choice_is_as_good_as_any_equal_segmentation(algo, port, p, m):
    """The chosen segment's simulated time is within 1 % of the best over a dense grid of segment sizes
    (the closed forms are exact when s divides m, upper bounds otherwise)."""
    s = rd.rd_optimal_segment(algo, port, p, m, *M1)
    assert s % 4 == 0 and 4 <= s <= m
    chosen = oracle_time(algo, port, p, m, s, M1)
    grid = sorted({max(4, min(m, int(round(m / q / 4)) * 4)) for q in
                   list(range(1, 65)) + [int(1.25 ** k) for k in range(18, 29)] if q <= m // 4})
    best = min(oracle_time(algo, port, p, m, g, M1) for g in grid)
    assert chosen <= best * 1.01, (s, chosen, best)


def test_closed_forms_at_exact_parameters():
    """Table I pipeline: p = 5, alpha = 4, beta + gamma = 1, m = 16 units -> s_opt = 8 (here 1 unit = 4 bytes)."""
    model = (4e-15, 0.25e-15, 0.0, 0.25e-15)       # tick = 0.25 fs: alpha = 16 ticks, beta = 1 tick per byte (4 per unit)
    assert rd.rd_optimal_segment(rd.RD_PIPELINE, rd.RD_PORT_UNI, 5, 64, *model) == 32
    # Table III bi-greedy: s_opt = sqrt(m alpha / ((ceil(log2 p) - 1)(beta + gamma))); p = 32, m = 64 units, alpha = 4 -> 8 units
    assert rd.rd_optimal_segment(rd.RD_BI_GREEDY, rd.RD_PORT_BI, 32, 256, *model) == 32
    # no latency: the smallest segment; no bandwidth or compute cost: one segment
    assert rd.rd_optimal_segment(rd.RD_PIPELINE, rd.RD_PORT_BI, 64, 4096, 0.0, 1e-10, 0.0) == 4
    assert rd.rd_optimal_segment(rd.RD_PIPELINE, rd.RD_PORT_BI, 64, 4096, 1e-6, 0.0, 0.0) == 4096
    # small p: the formulas' denominators vanish -> one segment
    assert rd.rd_optimal_segment(rd.RD_PIPELINE, rd.RD_PORT_UNI, 3, 4096, *M1) == 4096
    assert rd.rd_optimal_segment(rd.RD_BI_GREEDY, rd.RD_PORT_BI, 2, 4096, *M1) == 4096
    # binomial and butterfly take the whole message
    assert rd.rd_optimal_segment(rd.RD_BINOMIAL, rd.RD_PORT_UNI, 64, 4096, *M1) == 4096
    assert rd.rd_optimal_segment(rd.RD_BUTTERFLY, rd.RD_PORT_BI, 64, 4096, *M1) == 4096


@pytest.mark.parametrize("p", [4, 16, 64])
@pytest.mark.parametrize("m", [64, 1 << 12, 1 << 15])
def test_unigreedy_search_over_powers_of_two(p, m):
    """Section VII: segment sizes 2^i are tried and the best time kept (ties: the larger segment)."""
    s = rd.rd_optimal_segment(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, p, m, *M1)
    times = {}
    for i in range(2, int(math.log2(m)) + 1):
        if m // (1 << i) <= 1 << 11:
            times[1 << i] = oracle_time(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, p, m, 1 << i, M1)
    best = min(times.values())
    assert times[s] == best and s == max(k for k, v in times.items() if v == best)


def test_small_messages_make_unigreedy_the_binomial_tree():
    """Section V-B: for small messages the best uni-greedy has one segment and costs what binomial costs."""
    A, B, G = ticks(*M1)
    for p in (4, 64, 1024):
        m = 64
        assert rd.rd_optimal_segment(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, p, m, *M1) == m
        h = rd.rd_schedule_create(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, p, m, 0, *M1)       # 0 = the optimum
        info = rd.rd_schedule_info(h)
        rd.rd_destroy(h)
        assert info["q"] == 1 and info["predicted_ticks"] == math.ceil(math.log2(p)) * (A + (B + G) * m)


def test_seg_bytes_zero_uses_the_optimum():
    for algo, port in ((rd.RD_PIPELINE, rd.RD_PORT_UNI), (rd.RD_BI_GREEDY, rd.RD_PORT_BI), (rd.RD_BINARY, rd.RD_PORT_BI)):
        m = 1 << 18
        s = rd.rd_optimal_segment(algo, port, 64, m, *M1)
        h = rd.rd_schedule_create(algo, port, 64, m, 0, *M1)
        assert rd.rd_schedule_info(h)["q"] == -(-m // s)
        rd.rd_destroy(h)


def test_unequal_segmentation_search_on_table4():
    """Section VIII: the local search (one unit moved at a time, starting from the best equi-segmentation)
    never ends worse than the best equi-segmentation, and on the table's experiments it reaches the true
    optimum in most cases, as the paper observes for one or two unit moves."""
    from test_oracle_schedules import TABLE4, COMPS
    rows = [r for r in TABLE4 if r[0] <= 128]
    reached = improved = 0
    for p, a, g, ratio, equi, opts in rows:
        # one paper unit = 4 bytes; beta = gamma_paper... per byte 1 tick, so every time is 4x the paper's
        sizes, t = rd.rd_search_segmentation(p, 40, 4, 4 * a * 1e-15, 1e-15, g * 1e-15)
        times = O.unequal_times(p, a, g)
        best = int(times.min())
        best_equi = min(int(times[COMPS.index(tuple(O.equal_sizes(10, s)))]) for s in range(1, 11))
        assert sum(sizes) == 40 and all(s % 4 == 0 and s > 0 for s in sizes)
        found = int(times[COMPS.index(tuple(s // 4 for s in sizes))])
        assert t == 4 * found                   # the library's own prediction for what it returns
        assert best <= found <= best_equi
        improved += found < best_equi           # these are the experiments an unequal segmentation wins
        reached += found == best
    assert improved >= 0.9 * len(rows) and reached >= 0.8 * len(rows), (improved, reached, len(rows))
