"""Host logic of the schedule-faithful execution: the per-process action lists, replayed on the CPU
by a small message-passing emulation (flags, slots, rendezvous), must never dead-lock, never
overwrite a slot that is still to be read, and must give the oracle's bits."""
import numpy as np
import pytest

import paper_1310_4645_b200 as rd
from oracle import rd_oracle as O
from helpers import oracle_schedule

M1 = (2e-6, 1e-10, 5e-11)
CASES = [(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI), (rd.RD_BI_GREEDY, rd.RD_PORT_BI), (rd.RD_BINOMIAL, rd.RD_PORT_UNI),
         (rd.RD_PIPELINE, rd.RD_PORT_UNI), (rd.RD_PIPELINE, rd.RD_PORT_BI), (rd.RD_BINARY, rd.RD_PORT_UNI),
         (rd.RD_BINARY, rd.RD_PORT_BI), (rd.RD_BUTTERFLY, rd.RD_PORT_BI)]


def slot_words(off):
    return (max(int(off[j]) % 4 + int(off[j + 1] - off[j]) for j in range(len(off) - 1)) + 3) // 4 * 4


def lane_range(width, lanes, g, seg_start, seg_len, v=4):
    """Slot words [lo, hi) of a segment that block g of a process's G blocks works on (rule stated in
    include/rd.h): a fixed 1/G of the slot, clipped to where the segment sits in it."""
    units = width // v
    lo, hi = units * g // lanes * v, units * (g + 1) // lanes * v
    first, last = seg_start % 4, seg_start % 4 + seg_len
    lo, hi = max(lo, first), min(hi, last)
    return (lo, hi) if lo < hi else (first, first)


def emulate(h, x, op, blocking_send, rng, lanes=1):
    """Runs every process's action list; the (process, lane) agents advance in random order, one action at
    a time.  Lanes have their own flags but share the scratch slots, as on the GPU."""
    if lanes > 1:
        return emulate_lanes(h, x, op, blocking_send, rng, lanes)
    p, n = x.shape
    off = rd.rd_schedule_segments(h).astype(np.int64)
    lists, slots = [], 0
    for i in range(p):
        a, slots = rd.rd_schedule_actions(h, i)
        lists.append(a)
    longest = int(np.diff(off).max()) if len(off) > 1 else 0
    scratch = np.zeros((p, max(slots, 1), max(longest, 1)), dtype=x.dtype)
    out = np.zeros(n, dtype=x.dtype)
    n_events = rd.rd_schedule_info(h)["n_events"]
    posted = np.zeros(n_events, dtype=bool)
    taken = np.zeros(n_events, dtype=bool)
    reads_pending = {}                    # (proc, slot) -> event whose receiver still has to read it
    pc = [0] * p
    waiting_ack = [None] * p

    def combine(held, inc):
        if op == "sum":
            if x.dtype == np.int32:
                return (held.view(np.uint32) + inc.view(np.uint32)).view(np.int32)
            return (held + inc).astype(np.float32)
        return np.where(inc > held, inc, held)

    def value(proc, slot, seg):
        lo, hi = off[seg], off[seg + 1]
        if slot >= 0:
            return scratch[proc, slot, :hi - lo]
        return x[proc, lo:hi] if slot == -1 else out[lo:hi]

    steps = 0
    while any(pc[i] < len(lists[i]) or waiting_ack[i] is not None for i in range(p)):
        progressed = False
        for i in rng.permutation(p):
            if waiting_ack[i] is not None:
                if not taken[waiting_ack[i]]:
                    continue
                waiting_ack[i] = None
                progressed = True
            if pc[i] >= len(lists[i]):
                continue
            seg, peer, kind, slot, peer_slot, first, ev, wait_ev = (int(v) for v in lists[i][pc[i]])
            lo, hi = off[seg], off[seg + 1]
            if kind == 2:
                posted[ev] = True
                if slot >= 0:
                    reads_pending[(i, slot)] = ev
                if blocking_send:
                    waiting_ack[i] = ev
                pc[i] += 1
                progressed = True
                continue
            if wait_ev >= 0 and not taken[wait_ev]:
                continue
            if not posted[ev]:
                continue
            if slot >= 0:
                # the slot must not hold a value some receiver has not read yet
                pend = reads_pending.get((i, slot))
                assert pend is None or taken[pend], "slot overwritten before it was read"
            inc = value(peer, peer_slot, seg).copy()
            held = x[i, lo:hi] if first else value(i, slot, seg)
            res = inc if kind == 1 else combine(held, inc)
            if slot >= 0:
                scratch[i, slot, :hi - lo] = res
            else:
                assert i == 0 and slot == -2
                out[lo:hi] = res
            taken[ev] = True
            pc[i] += 1
            progressed = True
        steps += 1
        assert progressed, "dead-lock in the action lists"
    assert posted.all() and taken.all()
    return out, slots


def emulate_lanes(h, x, op, blocking_send, rng, lanes):
    p, n = x.shape
    off = rd.rd_schedule_segments(h).astype(np.int64)
    lists = [rd.rd_schedule_actions(h, i)[0] for i in range(p)]
    slots = rd.rd_schedule_actions(h, 0)[1]
    longest = int(np.diff(off).max())
    width = slot_words(off)
    scratch = np.zeros((p, max(slots, 1), width), dtype=x.dtype)
    owner = np.full(scratch.shape, -1, dtype=np.int64)      # segment whose value an offset of a slot holds
    out = np.zeros(n, dtype=x.dtype)
    n_events = rd.rd_schedule_info(h)["n_events"]
    posted = np.zeros((n_events, lanes), dtype=bool)
    taken = np.zeros((n_events, lanes), dtype=bool)
    pc = np.zeros((p, lanes), dtype=np.int64)
    waiting = np.full((p, lanes), -1, dtype=np.int64)
    # let some lanes run far ahead of others: a lane is only scheduled with its own probability
    speed = rng.uniform(0.05, 1.0, size=lanes)

    def combine(held, inc):
        if op == "sum":
            if x.dtype == np.int32:
                return (held.view(np.uint32) + inc.view(np.uint32)).view(np.int32)
            return (held + inc).astype(np.float32)
        return np.where(inc > held, inc, held)

    agents = [(i, g) for i in range(p) for g in range(lanes)]
    idle_rounds = 0
    while any(pc[i, g] < len(lists[i]) or waiting[i, g] >= 0 for i, g in agents):
        progressed = False
        for k in rng.permutation(len(agents)):
            i, g = agents[k]
            if rng.random() > speed[g]:
                continue
            if waiting[i, g] >= 0:
                if not taken[waiting[i, g], g]:
                    continue
                waiting[i, g] = -1
                progressed = True
            if pc[i, g] >= len(lists[i]):
                continue
            seg, peer, kind, slot, peer_slot, first, ev, wait_ev = (int(v) for v in lists[i][pc[i, g]])
            seg_len = off[seg + 1] - off[seg]
            lo, hi = lane_range(width, lanes, g, off[seg], seg_len)        # slot words
            base = off[seg] - off[seg] % 4                                 # message word of slot word 0
            if kind == 2:
                posted[ev, g] = True
                if blocking_send:
                    waiting[i, g] = ev
                pc[i, g] += 1
                progressed = True
                continue
            if (wait_ev >= 0 and not taken[wait_ev, g]) or not posted[ev, g]:
                continue
            if peer_slot >= 0:
                assert (owner[peer, peer_slot, lo:hi] == seg).all(), "the sender's slot holds another segment here"
                inc = scratch[peer, peer_slot, lo:hi].copy()
            else:
                inc = (x[peer, base + lo:base + hi] if peer_slot == -1 else out[base + lo:base + hi]).copy()
            if first:
                held = x[i, base + lo:base + hi]
            elif slot >= 0:
                assert (owner[i, slot, lo:hi] == seg).all(), "own slot holds another segment here"
                held = scratch[i, slot, lo:hi]
            else:
                held = out[base + lo:base + hi]
            res = inc if kind == 1 else combine(held, inc)
            if slot >= 0:
                scratch[i, slot, lo:hi] = res
                owner[i, slot, lo:hi] = seg
            else:
                out[base + lo:base + hi] = res
            taken[ev, g] = True
            pc[i, g] += 1
            progressed = True
        idle_rounds = 0 if progressed else idle_rounds + 1
        assert idle_rounds < 200, "dead-lock in the action lists"
    return out, slots


@pytest.mark.parametrize("algo,port", CASES)
@pytest.mark.parametrize("seg", [256, 257, 101])
def test_lanes_that_drift_apart_never_meet_in_a_slot(algo, port, seg):
    """Unequal segments (a short last one; with 257 and 101 they also begin at every position inside a
    128-bit vector), several blocks per process running at very different speeds."""
    p, n = 13, 618
    rng = np.random.default_rng(algo)
    x = (rng.standard_normal((p, n)) * 10.0 ** rng.integers(-4, 5, size=(p, n))).astype(np.float32)
    h = rd.rd_schedule_create(algo, port, p, 4 * n, 4 * seg if algo != rd.RD_BUTTERFLY else 0, *M1)
    try:
        ev, off, _ = oracle_schedule(algo, port, p, 4 * n, 4 * seg if algo != rd.RD_BUTTERFLY else 4 * n, *M1)
        want = O.reduce(ev, x, off, "sum")
        for trial in range(4):
            got, _ = emulate(h, x, "sum", port == rd.RD_PORT_UNI, np.random.default_rng(100 + trial), lanes=5)
            assert got.tobytes() == want.tobytes()
    finally:
        rd.rd_destroy(h)


@pytest.mark.parametrize("algo,port", CASES)
@pytest.mark.parametrize("p", [2, 3, 8, 13, 32])
def test_action_lists_reproduce_the_oracle(algo, port, p):
    n, seg = 96, 16
    rng = np.random.default_rng(7 * p + algo)
    xf = (rng.standard_normal((p, n)) * 10.0 ** rng.integers(-6, 7, size=(p, n))).astype(np.float32)
    xi = rng.integers(-2**31, 2**31, size=(p, n), dtype=np.int64).astype(np.int32)
    h = rd.rd_schedule_create(algo, port, p, 4 * n, 4 * seg, *M1)
    try:
        ev, off, _ = oracle_schedule(algo, port, p, 4 * n, 4 * seg, *M1)
        for x, op in ((xf, "sum"), (xf, "max"), (xi, "sum")):
            for trial in range(3):
                got, slots = emulate(h, x, op, port == rd.RD_PORT_UNI, np.random.default_rng(trial))
                assert got.tobytes() == O.reduce(ev, x, off, op).tobytes()
        if algo == rd.RD_UNI_GREEDY:
            assert slots <= 1            # Section V: in-order reduction needs one partial segment per process
    finally:
        rd.rd_destroy(h)


def test_slots_of_the_named_workloads_are_small():
    for algo, port, p, msg, seg, bound in ((rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, 64, 4 << 20, 16 << 10, 1),
                                           (rd.RD_BI_GREEDY, rd.RD_PORT_BI, 64, 4 << 20, 16 << 10, 8),
                                           (rd.RD_PIPELINE, rd.RD_PORT_BI, 64, 4 << 20, 16 << 10, 2),
                                           (rd.RD_BINARY, rd.RD_PORT_UNI, 64, 4 << 20, 16 << 10, 2)):
        h = rd.rd_schedule_create(algo, port, p, msg, seg, *M1)
        _, slots = rd.rd_schedule_actions(h, 1)
        rd.rd_destroy(h)
        assert 1 <= slots <= bound, (algo, slots)
