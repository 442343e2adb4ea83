"""rd_reduce_faithful_static: the schedule-faithful reduction for callers that cannot allocate.

Some users of this library run it inside a process whose device memory is already spoken for --
a serving stack that reserved the whole GPU for its own pool, a job tuned to the last byte -- or
from a loop in which a cudaMalloc (a driver-wide lock) is not acceptable.  For them the library
offers one entry point that keeps all of its scratch (tables, flags, partial-result slots) in a
fixed 32 MiB device array that is part of the library itself.  This test calls it through the C
ABI, always on a schedule nothing else has been called on (so the schedule owns no device tables
the call could lean on), and checks that
  * the result is the oracle's, bit for bit, and the same as the ordinary entry point's, which is
    run afterwards on the same schedule;
  * two and three calls in a row work (the array still holds the previous call's data);
  * the device's free memory as the driver reports it (cudaMemGetInfo, which sees every
    allocation of the process, the library's own cudaMalloc calls included) is the same before
    and after the call, while the ordinary entry point on a schedule of that size visibly lowers it;
  * a schedule too big for the array is refused.

Collected last on purpose (file name): a run that stops at the first failure has then already
run every other test.
"""
import numpy as np
import pytest
import torch

import paper_1310_4645_b200 as rd
from paper_1310_4645_b200.inputs import make_inputs
from oracle import rd_oracle as O
from helpers import oracle_schedule

pytestmark = pytest.mark.gpu

M1 = (2e-6, 1e-10, 5e-11)
OPNAME = {rd.RD_SUM: "sum", rd.RD_MAX: "max"}


def free_bytes():
    torch.cuda.synchronize()
    return torch.cuda.mem_get_info()[0]


@pytest.fixture(autouse=True)
def first_call_is_the_set_up():
    """The first call on a device looks up the array's address (and, in a fresh process, makes the CUDA
    runtime load the library's kernels and set up cooperative launches): do it before anything is measured."""
    x = make_inputs(2, 64, "normal", seed=0, device="cuda")
    out = torch.empty(64, device="cuda")
    h = rd.rd_schedule_create(rd.RD_PIPELINE, rd.RD_PORT_UNI, 2, 256, 128, *M1)
    try:
        rd.rd_reduce_faithful_static(h, x, out, rd.RD_SUM)
    finally:
        rd.rd_destroy(h)
    yield


def both_ways(algo, port, p, n, seg_bytes, dist, op, seed, expect_allocation=False):
    x = make_inputs(p, n, dist, seed=seed, device="cuda")
    ref = torch.full((n,), 5, dtype=x.dtype, device="cuda")
    got = torch.full((n,), 7, dtype=x.dtype, device="cuda")
    tab = rd.PointerTable(x)
    ev, off, _ = oracle_schedule(algo, port, p, 4 * n, seg_bytes if seg_bytes else 4 * n, *M1)
    want = O.reduce(ev, x.cpu().numpy(), off, OPNAME[op])
    h = rd.rd_schedule_create(algo, port, p, 4 * n, seg_bytes, *M1)      # a fresh schedule: never uploaded, never run
    try:
        before = free_bytes()
        st = rd.rd_reduce_faithful_static(h, tab, got, op, want_stats=True)    # the one that allocates nothing
        after = free_bytes()
        rd.rd_reduce(h, tab, ref, op, exec_mode=rd.RD_EXEC_FAITHFUL)          # the existing entry point, which allocates
        later = free_bytes()
    finally:
        rd.rd_destroy(h)
    assert after == before, "the device's free memory changed by %d bytes across the call" % (before - after)
    if expect_allocation:                    # the same measure does see the ordinary entry point's cudaMalloc calls
        assert later < after
    assert st.device_status == 0
    if p > 1:                                # a single process holds the result already: a plain copy
        assert st.n_launches == 1 and st.makespan_ns > 0
    # schedule-ordered results are exact: the oracle's bytes, and the existing entry point's
    assert got.cpu().numpy().tobytes() == want.tobytes()
    assert torch.equal(got.view(torch.int32), ref.view(torch.int32))


def test_two_calls_in_a_row_match_the_oracle_and_the_allocating_entry_point():
    # first call: uni-greedy, fp32 sum; second call: another schedule, shape, dtype and op, so that the
    # array's regions fall differently and stale flags or slots of the first call would show
    both_ways(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, 16, 1 << 15, 4096, "normal", rd.RD_SUM, seed=1)
    both_ways(rd.RD_BI_GREEDY, rd.RD_PORT_BI, 33, 6000, 4000, "int_pm2p20", rd.RD_MAX, seed=2)
    # and the first one again
    both_ways(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, 16, 1 << 15, 4096, "normal", rd.RD_SUM, seed=3)


def test_the_measure_sees_the_other_entry_points_allocations():
    # binomial, one segment of 2 MiB per process: 16 MiB of partial-result slots, which fit the array and which
    # the ordinary entry point has to cudaMalloc
    both_ways(rd.RD_BINOMIAL, rd.RD_PORT_UNI, 8, 1 << 19, 0, "normal", rd.RD_SUM, seed=7, expect_allocation=True)


def test_every_schedule_once():
    for algo, port in ((rd.RD_BINOMIAL, rd.RD_PORT_UNI), (rd.RD_PIPELINE, rd.RD_PORT_BI),
                       (rd.RD_BINARY, rd.RD_PORT_UNI), (rd.RD_BUTTERFLY, rd.RD_PORT_BI)):
        both_ways(algo, port, 8, 3003, 4 * 333, "normal", rd.RD_SUM, seed=4)     # element path too
    both_ways(rd.RD_PIPELINE, rd.RD_PORT_UNI, 1, 1000, 400, "normal", rd.RD_SUM, seed=5)   # single process


def test_a_schedule_beyond_the_array_is_refused():
    p, n = 64, 1 << 20                      # slots alone: 64 processes x 1 MiB segments = 64 MiB > 32 MiB
    x = make_inputs(p, n, "normal", seed=6, device="cuda")
    out = torch.zeros(n, device="cuda")
    h = rd.rd_schedule_create(rd.RD_BINOMIAL, rd.RD_PORT_UNI, p, 4 * n, 0, *M1)
    try:
        with pytest.raises(rd.RdError) as e:
            rd.rd_reduce_faithful_static(h, x, out, rd.RD_SUM)
        assert e.value.status == rd.RD_ERR_TOO_LARGE
        assert "scratch" in str(e.value)
        assert (out == 0).all()              # nothing was launched
    finally:
        rd.rd_destroy(h)
