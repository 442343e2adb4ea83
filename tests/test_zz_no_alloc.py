"""rd_reduce_faithful_static: the schedule-faithful reduction for callers that cannot allocate.

Some users of this library run it inside a process whose device memory is already spoken for --
a serving stack that reserved the whole GPU for its own pool, a job tuned to the last byte -- or
from a loop in which a cudaMalloc (a driver-wide lock) is not acceptable.  For them the library
offers one entry point that keeps all of its scratch (tables, flags, partial-result slots) in a
fixed 32 MiB device array that is part of the library itself.  This test calls it through the C
ABI and checks that it gives exactly the bits of the ordinary entry point, twice in a row (the
array still holds the first call's data when the second one starts), that torch's allocator is
not asked for anything meanwhile, and that a schedule too big for the array is refused.

Collected last on purpose (file name): a run that stops at the first failure has then already
run every other test.
"""
import pytest
import torch

import paper_1310_4645_b200 as rd
from paper_1310_4645_b200.inputs import make_inputs

pytestmark = pytest.mark.gpu

M1 = (2e-6, 1e-10, 5e-11)


def both_ways(algo, port, p, n, seg_bytes, dist, op, seed):
    x = make_inputs(p, n, dist, seed=seed, device="cuda")
    ref = torch.full((n,), 5, dtype=x.dtype, device="cuda")
    got = torch.full((n,), 7, dtype=x.dtype, device="cuda")
    tab = rd.PointerTable(x)
    h = rd.rd_schedule_create(algo, port, p, 4 * n, seg_bytes, *M1)
    try:
        rd.rd_reduce(h, tab, ref, op, exec_mode=rd.RD_EXEC_FAITHFUL)          # the existing entry point
        torch.cuda.synchronize()
        before = torch.cuda.memory_stats()["allocation.all.allocated"]
        st = rd.rd_reduce_faithful_static(h, tab, got, op, want_stats=True)    # the one that allocates nothing
        after = torch.cuda.memory_stats()["allocation.all.allocated"]
    finally:
        rd.rd_destroy(h)
    assert after == before
    assert st.device_status == 0
    if p > 1:                                # a single process holds the result already: a plain copy
        assert st.n_launches == 1 and st.makespan_ns > 0
    # same kernel, same order of combines: the results are identical bit for bit (the tests' tolerance
    # for schedule-ordered results is exactness)
    assert torch.equal(got.view(torch.int32), ref.view(torch.int32))


def test_two_calls_in_a_row_match_the_allocating_entry_point():
    # first call: uni-greedy, fp32 sum; second call: another schedule, shape, dtype and op, so that the
    # array's regions fall differently and stale flags or slots of the first call would show
    both_ways(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, 16, 1 << 15, 4096, "normal", rd.RD_SUM, seed=1)
    both_ways(rd.RD_BI_GREEDY, rd.RD_PORT_BI, 33, 6000, 4000, "int_pm2p20", rd.RD_MAX, seed=2)
    # and the first one again
    both_ways(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, 16, 1 << 15, 4096, "normal", rd.RD_SUM, seed=3)


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
