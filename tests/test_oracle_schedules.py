"""Pins of the oracle's schedule simulators (no GPU, no library code).

Every expected value below comes from the paper (tables, worked examples,
theorem) or from mathematics that does not go through the oracle.
"""
import math
import os
from concurrent.futures import ThreadPoolExecutor
from fractions import Fraction
from functools import lru_cache

import numpy as np
import pytest

from oracle import rd_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def clog2(v):
    return max(0, (int(v) - 1).bit_length())


def check_valid(ev, p, sizes, A, B, G, bidir, tree_rules=True, in_order=False):
    rc, last = O.validate(ev, p, sizes, A, B, G, bidir, tree_rules, in_order)
    assert rc == 0, "validity rule %d broken" % rc
    assert O.contributions(ev, p, len(sizes)) == 0
    return last


# --------------------------------------------------------------------------- Table I
GRID = [(p, q, s, A, B, G)
        for p in (2, 3, 4, 5, 7, 8, 15, 16, 17, 31, 33, 64)
        for q in (1, 2, 5)
        for s in (1, 8)
        for (A, B, G) in ((10, 1, 0), (3, 2, 1), (0, 1, 1))]


@pytest.mark.parametrize("p,q,s,A,B,G", GRID)
def test_table1_unidirectional_times(p, q, s, A, B, G):
    """Table I 'Time' rows: the end of the last activity of the simulated event list."""
    sizes = [s] * q
    unit = A + B * s + G * s
    ev, comp = O.pipeline(p, sizes, A, B, G, bidir=False)
    last = check_valid(ev, p, sizes, A, B, G, bidir=False)
    assert last == comp == (p - 1) * unit + 2 * (q - 1) * unit
    ev, comp = O.binary(p, sizes, A, B, G, bidir=False)
    last = check_valid(ev, p, sizes, A, B, G, bidir=False)
    N = clog2(p + 1)
    if p >= 3:      # the table's formulae are stated for p > 3; with p = 2 the root has no right child
        assert last == comp == 2 * (N - 1) * unit + 4 * (q - 1) * unit
    else:
        assert last == comp == unit + 4 * (q - 1) * unit
    # binomial is unsegmented in the paper: m = s, one segment
    ev, comp = O.binomial(p, [s], A, B, G)
    last = check_valid(ev, p, [s], A, B, G, bidir=False)
    assert last == comp == clog2(p) * (A + B * s + G * s)


def test_table1_optimal_segment_rows():
    """s_opt and T_opt of Table I at parameters where s_opt divides m: Time(s_opt) = T_opt and no
    other divisor of m does better."""
    # pipeline: p=5, alpha=4, beta+gamma=1, m=16 -> s_opt = sqrt(2*16*4/(2*1)) = 8, T_opt = (sqrt 8 + sqrt 32)^2 = 72
    p, A, B, G, m = 5, 4, 1, 0, 16
    times = {}
    for s in (1, 2, 4, 8, 16):
        ev, comp = O.pipeline(p, [s] * (m // s), A, B, G, bidir=False)
        _, times[s] = O.validate(ev, p, [s] * (m // s), A, B, G, False)
    s_opt = math.sqrt(2 * m * A / ((p - 3) * (B + G)))
    t_opt = (math.sqrt((p - 3) * A) + math.sqrt(2 * m * (B + G))) ** 2
    assert s_opt == 8 and abs(t_opt - 72) < 1e-9
    assert times[8] == 72 and min(times.values()) == 72
    # binary: p=31 (N=5), alpha=4, beta+gamma=1, m=16 -> s_opt = 8, T_opt = 2 (sqrt 8 + sqrt 32)^2 = 144
    p = 31
    times = {}
    for s in (1, 2, 4, 8, 16):
        ev, comp = O.binary(p, [s] * (m // s), A, B, G, bidir=False)
        _, times[s] = O.validate(ev, p, [s] * (m // s), A, B, G, False)
    assert times[8] == 144 and min(times.values()) == 144


# --------------------------------------------------------------------------- Table III
@pytest.mark.parametrize("p,q,s,A,B,G", GRID)
def test_table3_bidirectional_times(p, q, s, A, B, G):
    sizes = [s] * q
    unit = A + B * s + G * s
    ev, comp = O.pipeline(p, sizes, A, B, G, bidir=True)
    last = check_valid(ev, p, sizes, A, B, G, bidir=True)
    assert last == comp == (p + q - 2) * unit
    # binary: the printed Time row is two rounds longer than its own s_opt / T_opt rows imply; the
    # consistent form is 2(N + q - 2) rounds
    ev, comp = O.binary(p, sizes, A, B, G, bidir=True)
    last = check_valid(ev, p, sizes, A, B, G, bidir=True)
    N = clog2(p + 1)
    if p >= 3:
        assert last == comp == 2 * (N + q - 2) * unit
    else:
        assert last == comp == unit + 2 * (q - 1) * unit
    # bi-greedy: the time of a reverse optimal broadcast
    ev, comp = O.bi_greedy(p, sizes, A, B, G)
    last = check_valid(ev, p, sizes, A, B, G, bidir=True)
    assert last == comp == (clog2(p) + q - 1) * unit


def test_table3_binary_topt_consistency():
    """Bidirectional binary: T_opt = 2(sqrt((N-2)alpha) + sqrt(m(beta+gamma)))^2 is reached at s_opt."""
    p, A, B, G, m = 63, 4, 1, 0, 16      # N = 6: s_opt = sqrt(16*4/4) = 4, T_opt = 2 (4 + 4)^2 = 128
    best = None
    for s in (1, 2, 4, 8, 16):
        ev, _ = O.binary(p, [s] * (m // s), A, B, G, bidir=True)
        _, last = O.validate(ev, p, [s] * (m // s), A, B, G, True)
        best = last if best is None else min(best, last)
        if s == 4:
            assert last == 128
    assert best == 128


@pytest.mark.parametrize("p", [1, 2, 4, 8, 16, 64, 256])
@pytest.mark.parametrize("A,B,G", [(10, 1, 0), (3, 2, 1), (50000, 6, 1)])
def test_table3_butterfly_time(p, A, B, G):
    """Butterfly Time row, p a power of two dividing the message length."""
    n = 4 * 256
    ev, off, comp = O.butterfly(p, n, 1, A, B, G)
    L = clog2(p)
    exact = Fraction(2 * L * A) + Fraction(2 * (p - 1) * B * n, p) + Fraction((p - 1) * G * n, p)
    assert exact.denominator == 1 and comp == exact
    sizes = np.diff(off)
    assert (sizes == n // p).all()
    rc, last = O.validate(ev, p, sizes, A, B, G, True, tree_rules=False)
    assert rc == 0 and last == comp
    assert O.contributions(ev, p, p) == 0


def test_butterfly_ragged_and_short_messages():
    for p, n in ((8, 13), (16, 5), (4, 0), (8, 1001)):
        ev, off, comp = O.butterfly(p, n, 4, 7, 1, 1)
        assert off[0] == 0 and off[-1] == n and (np.diff(off) >= 0).all()
        # halves of odd ranges differ by one element, so a process's own (longer) send can still run when
        # its (shorter) receive is done; rounds are lock-step and as long as their longest message, and the
        # port and data-safety rules are checked on the communication pattern alone (gamma = 0)
        rc, last = O.validate(ev, p, np.diff(off) * 4, 7, 1, 0, True, tree_rules=False)
        assert rc == 0 and last <= comp
        assert O.contributions(ev, p, p) == 0
        L = clog2(p)
        assert comp * p >= 2 * L * 7 * p + 2 * (p - 1) * 1 * 4 * n + (p - 1) * 1 * 4 * n


@pytest.mark.parametrize("p", [3, 5, 6, 7, 12, 24, 100])
def test_butterfly_folds_extra_processes_in_first(p):
    """Not a power of two (an extension: the paper only cites an improved algorithm): the processes beyond
    the largest power of two P send their message to a partner first, one round of alpha + (beta+gamma) m,
    then the P-process butterfly of Table III follows.  Valid, and every contribution arrives once."""
    A, B, G = 7, 2, 1
    P = 1 << (p.bit_length() - 1)
    n = 4 * P
    ev, off, comp = O.butterfly(p, n, 1, A, B, G)
    L = clog2(P)
    assert comp == (A + (B + G) * n) + 2 * L * A + 2 * (P - 1) * B * n // P + (P - 1) * G * n // P
    assert len(off) == P + 1 and (np.diff(off) == n // P).all()
    rc, last = O.validate(ev, p, np.diff(off), A, B, G, True, tree_rules=False)
    assert rc == 0 and last == comp
    assert O.contributions(ev, p, P) == 0
    x = np.random.default_rng(p).integers(-2**31, 2**31, size=(p, n), dtype=np.int64).astype(np.int32)
    assert (O.reduce(ev, x, off, "max") == x.max(axis=0)).all()


# --------------------------------------------------------------------------- worked examples
def test_fig8_bigreedy_example():
    """16 processes, 5 equal segments, t_comm = 2, t_comp = 1: the time of an optimal broadcast,
    (ceil(log2 16) + 5 - 1) * 3 = 24."""
    ev, comp = O.bi_greedy(16, [1] * 5, 2, 0, 1)
    assert comp == 24
    assert check_valid(ev, 16, [1] * 5, 2, 0, 1, bidir=True) == 24


def test_bigreedy_matches_reverse_optimal_broadcast_everywhere():
    """Conjecture of Section VI-B, Table III: (ceil(log2 p) + q - 1)(alpha + beta s + gamma s)."""
    for p in range(2, 70):
        for q in range(1, 13):
            for (A, B, G) in ((2, 0, 1), (1, 1, 0), (3, 1, 2)):
                _, comp = O.bi_greedy(p, [1] * q, A, B, G, want_events=False)
                assert comp == (clog2(p) + q - 1) * (A + B + G), (p, q, A, B, G)
    for p in (100, 127, 128, 129, 500, 1024):
        for q in (1, 3, 20):
            ev, comp = O.bi_greedy(p, [4] * q, 5, 1, 1)
            assert comp == (clog2(p) + q - 1) * (5 + 4 + 4)
            check_valid(ev, p, [4] * q, 5, 1, 1, bidir=True)


def test_bigreedy_unit_step_equals_event_driven():
    """The printed loop advances t by 1; jumping to the next instant a port frees changes nothing."""
    for p in (2, 3, 4, 7, 16, 21):
        for q in (1, 2, 5):
            for (A, B, G) in ((2, 0, 1), (1, 1, 0), (3, 1, 2)):
                for sizes in ([2] * q, [2] * (q - 1) + [1]):
                    e1, c1 = O.bi_greedy(p, sizes, A, B, G, unit_step=False)
                    e2, c2 = O.bi_greedy(p, sizes, A, B, G, unit_step=True)
                    assert c1 == c2 and (e1 == e2).all()
                    check_valid(e1, p, sizes, A, B, G, bidir=True)


def test_unigreedy_single_segment_is_binomial():
    """With one segment uni-greedy is exactly the binomial algorithm (Section V-B)."""
    for p in range(1, 70):
        for (A, B, G, m) in ((10, 1, 0, 64), (3, 2, 1, 5), (0, 1, 1, 7)):
            ev, comp = O.uni_greedy(p, [m], A, B, G)
            assert comp == clog2(p) * (A + B * m + G * m)
            if p > 1:
                assert check_valid(ev, p, [m], A, B, G, bidir=False, in_order=True) == comp


def test_fig3_example_is_valid_and_in_order():
    """15 processes, 5 equal segments, t_comm = 2, t_comp = 1 (only the parameters are printed)."""
    ev, comp = O.uni_greedy(15, [1] * 5, 2, 0, 1)
    assert check_valid(ev, 15, [1] * 5, 2, 0, 1, bidir=False, in_order=True) == comp


# --------------------------------------------------------------------------- Table II
def test_lower_bounds_table2():
    """No schedule beats the latency, bandwidth and computation bounds taken one at a time."""
    for p in (3, 4, 6, 16, 33, 100):
        for m, s in ((16, 16), (16, 4), (16, 1), (30, 7)):
            sizes = O.equal_sizes(m, s)
            for (A, B, G) in ((5, 0, 0), (0, 1, 0), (0, 0, 1), (2, 1, 1)):
                _, cu = O.uni_greedy(p, sizes, A, B, G, want_events=False)
                _, cb = O.bi_greedy(p, sizes, A, B, G, want_events=False)
                assert cu >= clog2(p) * A
                assert cb >= clog2(p) * A
                assert cu >= 2 * m * B            # unidirectional bandwidth bound, p >= 3
                assert cb >= m * B
                assert cu * p >= (p - 1) * m * G
                assert cb * p >= (p - 1) * m * G


# --------------------------------------------------------------------------- Theorem 5
def brute_force_in_order_optimum(p, sizes, A, B, G):
    """Minimum completion time over ALL schedules that reduce segments in order: per segment any
    sequence of valid send/receive pairs (Lemma 1: sender is not the root, t = max of the two states)."""
    q = len(sizes)

    @lru_cache(maxsize=None)
    def best(j, root, others, remaining_mask):
        # others: tuple of states of processes 1..p-1; remaining_mask: which of them still hold segment j
        if remaining_mask == 0:
            if j + 1 == q:
                return root
            return best(j + 1, root, others, (1 << (p - 1)) - 1)
        tc, tp = A + B * sizes[j], G * sizes[j]
        res = None
        for a in range(p - 1):
            if not (remaining_mask >> a) & 1:
                continue
            # receiver: the root
            t = max(others[a], root)
            o = list(others); o[a] = t + tc
            r = best(j, t + tc + tp, tuple(o), remaining_mask & ~(1 << a))
            res = r if res is None or r < res else res
            for b in range(p - 1):
                if b == a or not (remaining_mask >> b) & 1:
                    continue
                t = max(others[a], others[b])
                o = list(others); o[a] = t + tc; o[b] = t + tc + tp
                r = best(j, root, tuple(o), remaining_mask & ~(1 << a))
                res = r if r < res else res
        return res

    return best(0, 0, tuple([0] * (p - 1)), (1 << (p - 1)) - 1)


@pytest.mark.parametrize("p,sizes", [(2, [1, 1, 1]), (3, [1, 1, 1]), (3, [2, 1, 3]), (4, [1, 1, 1]), (4, [3, 1]),
                                     (4, [1, 2, 1]), (5, [1, 1]), (5, [2, 1]), (5, [1, 1, 1])])
@pytest.mark.parametrize("A,B,G", [(2, 0, 1), (1, 1, 0), (0, 1, 1), (3, 1, 2)])
def test_theorem5_greedy_is_optimal_among_in_order_schedules(p, sizes, A, B, G):
    _, comp = O.uni_greedy(p, sizes, A, B, G, want_events=False)
    assert comp == brute_force_in_order_optimum(p, tuple(sizes), A, B, G)


# --------------------------------------------------------------------------- Table IV
def compositions():
    """Index -> segmentation of 10 units, bit k = a cut after unit k+1 (the oracle's convention)."""
    out = []
    for mask in range(512):
        sizes, run = [], 0
        for u in range(10):
            run += 1
            if u == 9 or (mask >> u) & 1:
                sizes.append(run); run = 0
        out.append(tuple(sizes))
    return out


COMPS = compositions()
# the table's "equi-segmentation" column only ever shows sizes ceil(10/q): 10, 5, 4, 3, 2, 1
EQUI_TABLE = [tuple(O.equal_sizes(10, s)) for s in (1, 2, 3, 4, 5, 10)]
EQUI_ALL = [tuple(O.equal_sizes(10, s)) for s in range(1, 11)]


def load_table4():
    rows = []
    with open(os.path.join(GOLDEN, "table4_unequal_segmentation.txt")) as f:
        for ln in f:
            if ln.startswith("#") or not ln.strip():
                continue
            par, ratio, equi, opts = [c.strip() for c in ln.split("|")]
            p, a, g = map(int, par.split())
            rows.append((p, a, g, ratio, tuple(map(int, equi.split(","))),
                         {tuple(map(int, o.split(","))) for o in opts.split(";")}))
    return rows


TABLE4 = load_table4()


def test_compositions_convention():
    assert len(set(COMPS)) == 512 and all(sum(c) == 10 for c in COMPS)
    t = O.unequal_times(8, 3, 1)
    for idx in (0, 511, 137, 300):
        _, c = O.uni_greedy(8, list(COMPS[idx]), 3, 1, 1, want_events=False)
        assert t[idx] == c


def _row_check(row):
    p, a, g, ratio, equi, opts = row
    t = O.unequal_times(p, a, g)
    by_seg = dict(zip(COMPS, t.tolist()))
    best = int(t.min())
    best_equi = min(by_seg[e] for e in EQUI_TABLE)
    assert "%.4f" % (best_equi / best) == ratio, (row, best_equi, best)
    assert by_seg[equi] == best_equi, (row, "equi-segmentation column")
    assert {c for c in COMPS if by_seg[c] == best} == opts, (row, "optimal segmentations")
    # listed because no equi-segmentation at all is optimal
    assert min(by_seg[e] for e in EQUI_ALL) > best
    return True


def test_table4_all_61_rows():
    """Ratio, best equi-segmentation and the full set of optimal segmentations of every row."""
    assert len(TABLE4) == 61
    with ThreadPoolExecutor(max_workers=os.cpu_count() or 1) as ex:
        assert all(ex.map(_row_check, TABLE4))
    # Section VIII: maximum improvement 7.3 %, mean of the 61 improvements 2.0 %
    ratios = [float(r[3]) for r in TABLE4]
    assert "%.1f" % ((max(ratios) - 1) * 100) == "7.3"
    assert "%.1f" % ((sum(ratios) / len(ratios) - 1) * 100) == "2.0"


def _is_unequal_optimised(args):
    p, a, g = args
    t = O.unequal_times(p, a, g)
    by_seg = dict(zip(COMPS, t.tolist()))
    return min(by_seg[e] for e in EQUI_ALL) > int(t.min())


def test_section8_census_61_of_986():
    """29 values of alpha x 2 of gamma x 17 of p = 986 experiments, 61 of which are optimised only by
    an unequal segmentation, and exactly the 61 the table lists."""
    alphas = list(range(0, 11)) + list(range(20, 101, 10)) + list(range(200, 1001, 100))
    ps = [2 ** k for k in range(2, 11)] + [3 * 2 ** k for k in range(1, 9)]
    exps = [(p, a, g) for p in ps for a in alphas for g in (0, 1)]
    assert len(exps) == 986
    with ThreadPoolExecutor(max_workers=os.cpu_count() or 1) as ex:
        flags = list(ex.map(_is_unequal_optimised, exps))
    found = {e for e, f in zip(exps, flags) if f}
    assert len(found) == 61
    assert found == {(r[0], r[1], r[2]) for r in TABLE4}


# --------------------------------------------------------------------------- the checker itself bites
def test_validator_catches_planted_mistakes():
    p, sizes, A, B, G = 8, [4, 4, 4], 3, 1, 1
    ev, comp = O.uni_greedy(p, sizes, A, B, G)
    assert O.validate(ev, p, sizes, A, B, G, False, True, True) == (0, comp)
    bad = ev.copy(); k = int(np.flatnonzero(bad["dst"] == 0)[0])
    bad["src"][k], bad["dst"][k] = 0, bad["src"][k]                 # the root sends
    assert O.validate(bad, p, sizes, A, B, G, False, True, True)[0] == 2
    bad = ev.copy(); bad["src"][0] = bad["src"][1]                  # someone never sends, someone twice
    assert O.validate(bad, p, sizes, A, B, G, False, True, True)[0] == 3
    bad = ev.copy(); k = int(np.argmax(bad["t_start"])); bad["t_start"][k] -= 1   # starts while still busy
    assert O.validate(bad, p, sizes, A, B, G, False, True, True)[0] in (4, 5)
    bad = ev[::-1].copy()
    assert O.validate(bad, p, sizes, A, B, G, False, True, True) == (0, comp)      # order of the list is free
    # a bidirectional schedule is not a unidirectional one
    evb, _ = O.bi_greedy(p, sizes, A, B, G)
    assert O.validate(evb, p, sizes, A, B, G, True)[0] == 0
    assert O.validate(evb, p, sizes, A, B, G, False)[0] == 4
    # contributions: drop one event, duplicate one
    assert O.contributions(ev[1:], p, 3) != 0
    assert O.contributions(np.concatenate([ev, ev[:1]]), p, 3) != 0
    # in-order rule: swap the segments of two events of one process
    bad = ev.copy()
    first0 = int(np.flatnonzero(bad["seg"] == 0)[0]); first1 = int(np.flatnonzero(bad["seg"] == 1)[0])
    bad["t_start"][first0], bad["t_start"][first1] = bad["t_start"][first1], bad["t_start"][first0]
    assert O.validate(bad, p, sizes, A, B, G, False, True, True)[0] != 0


# --------------------------------------------------------------------------- Section V-B text (soft pins)
def _best_times_p64(m, A=10, B=1, G=0, p=64):
    """Best completion time of each algorithm over all integer segment sizes (the figures of Section V-B
    use each algorithm's optimal segment size; alpha = 10, beta = 1, gamma = 0, p = 64)."""
    greedy = min(O.uni_greedy(p, O.equal_sizes(m, s), A, B, G, want_events=False)[1] for s in range(1, m + 1))
    unit = lambda s: A + (B + G) * s
    N = clog2(p + 1)
    binom = clog2(p) * unit(m)
    pipe = min((p - 1 + 2 * (-(-m // s) - 1)) * unit(s) for s in range(1, m + 1))
    binary = min((2 * (N - 1) + 4 * (-(-m // s) - 1)) * unit(s) for s in range(1, m + 1))
    return greedy, binom, pipe, binary


def test_section5_small_mid_and_large_message_regimes():
    """Small messages: uni-greedy with one segment IS binomial; mid-size: about 50 % faster than the best
    standard algorithm; large: pipeline approaches it."""
    ratios = {}
    for m in (4, 8, 16, 64, 128, 256, 512, 1024, 2048, 4096):
        g, binom, pipe, binary = _best_times_p64(m)
        assert g <= min(binom, pipe, binary)                       # Theorem 5: never worse than an in-order schedule
        ratios[m] = min(binom, pipe, binary) / g
        if m <= 16:
            assert g == binom                                      # same time as binomial
    assert 1.4 <= max(ratios.values()) <= 1.7                      # "approximately 50 % faster" in the middle
    assert max(ratios, key=ratios.get) in (256, 512, 1024)
    assert ratios[4096] < ratios[1024] < ratios[512]               # and the advantage fades for large messages
    g, binom, pipe, binary = _best_times_p64(16384)
    assert pipe == min(binom, pipe, binary) and pipe / g < 1.12    # pipeline approaches uni-greedy
