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


def emulate(h, x, op, blocking_send, rng):
    """Runs every process's action list; processes advance in random order, one action at a time."""
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


@pytest.mark.parametrize("algo,port", CASES)
@pytest.mark.parametrize("p", [2, 3, 8, 13, 32])
def test_action_lists_reproduce_the_oracle(algo, port, p):
    if algo == rd.RD_BUTTERFLY and p & (p - 1):
        pytest.skip("butterfly needs a power of two")
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
