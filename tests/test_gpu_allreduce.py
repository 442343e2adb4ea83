"""All-reduce (Section III: a reduce followed by a broadcast), reduction towards another root, and calls from
several threads, against the oracle through the C ABI (GPU)."""
import threading

import numpy as np
import pytest
import torch

import paper_1310_4645_b200 as rd
from paper_1310_4645_b200.inputs import make_inputs
from oracle import rd_oracle as O
from helpers import oracle_schedule

pytestmark = pytest.mark.gpu

M1 = (2e-6, 1e-10, 5e-11)
SCHEDULES = [(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI), (rd.RD_BI_GREEDY, rd.RD_PORT_BI), (rd.RD_BINOMIAL, rd.RD_PORT_UNI),
             (rd.RD_PIPELINE, rd.RD_PORT_UNI), (rd.RD_BINARY, rd.RD_PORT_BI), (rd.RD_BUTTERFLY, rd.RD_PORT_BI)]


def oracle_allreduce(algo, port, x, seg_bytes, op):
    """Section III: every process ends up with what the root holds after the reduce."""
    p, n = x.shape
    ev, off, _ = oracle_schedule(algo, port, p, 4 * n, seg_bytes, *M1)
    root = O.reduce(ev, x, off, op)
    return [root] * p


@pytest.mark.parametrize("algo,port", SCHEDULES)
def test_every_process_receives_the_roots_result(algo, port):
    # (p, n, segment elements): whole vectors; a ragged message (element path of the broadcast); one process; more
    # destinations than one broadcast launch carries (256)
    for p, n, seg in [(8, 4096, 512), (13, 6180, 999), (5, 4099, 1000), (1, 5000, 1000), (300, 2048, 1024)]:
        for dist, op in (("normal", "sum"), ("int_pm2p20", "max")):
            x = make_inputs(p, n, dist, seed=p + n, device="cuda")
            outs = torch.full((p, n), 77, dtype=x.dtype, device="cuda")
            h = rd.rd_schedule_create(algo, port, p, 4 * n, 4 * seg, *M1)
            try:
                st = rd.rd_allreduce(h, x, outs, rd.RD_SUM if op == "sum" else rd.RD_MAX, want_stats=True)
            finally:
                rd.rd_destroy(h)
            want = oracle_allreduce(algo, port, x.cpu().numpy(), 4 * seg, op)
            got = outs.cpu().numpy()
            for i in range(p):
                assert got[i].tobytes() == want[i].tobytes(), (p, n, i)
            assert st.device_status == 0
            assert st.bytes_moved == ((p + 1) + (p if p > 1 else 0)) * 4 * n
            vectors = all(x[i].data_ptr() % 16 == 0 for i in range(p)) and outs.data_ptr() % 16 == 0
            tail = 1 if vectors and n % 4 else 0             # the 128-bit path leaves the last n mod 4 elements to a second, tiny launch
            # the broadcast: at most 256 destinations per launch; aligned copies go through the bulk-copy kernel (whole
            # 128-bit vectors) and a word-wise launch for the last n mod 4 words, other copies through the word-wise one
            groups = 0 if p == 1 else (p - 2) // 256 + 1
            aligned = all(outs[i].data_ptr() % 16 == 0 for i in range(p))
            per_group = (1 if n >= 4 else 0) + (1 if n % 4 else 0) if aligned else 1
            assert st.n_launches == 1 + tail + groups * per_group


@pytest.mark.parametrize("p", [16, 40])      # up to 16 destinations: bulk copies through shared memory; more: registers
def test_in_place_and_unaligned_buffers(p):
    wide = make_inputs(p, 6000, "normal", seed=8, device="cuda")                             # every row 16-byte aligned
    big = make_inputs(p, 6002, "normal", seed=9, device="cuda")
    ragged = make_inputs(p, 6004, "normal", seed=11, device="cuda")                          # aligned rows, n mod 4 = 2
    for rows in ([wide[i] for i in range(p)], [big[i, :6001] for i in range(p)], [big[i, 1:] for i in range(p)],
                 [ragged[i, :6002] for i in range(p)]):
        n = rows[0].numel()
        keep = torch.stack(rows).cpu().numpy()
        h = rd.rd_schedule_create(rd.RD_BI_GREEDY, rd.RD_PORT_BI, p, 4 * n, 4 * 1000, *M1)
        try:
            rd.rd_allreduce(h, rows, rows, rd.RD_SUM)                                     # every copy over its own input
            torch.cuda.synchronize()
        finally:
            rd.rd_destroy(h)
        want = oracle_allreduce(rd.RD_BI_GREEDY, rd.RD_PORT_BI, keep, 4 * 1000, "sum")
        for i in range(p):
            assert rows[i].cpu().numpy().tobytes() == want[i].tobytes()
        big = make_inputs(p, 6002, "normal", seed=10, device="cuda")


def test_sixteen_bit_elements():
    p, n = 12, 8192
    x = torch.randn(p, n, device="cuda", generator=torch.Generator("cuda").manual_seed(3)).to(torch.bfloat16)
    outs = torch.zeros_like(x)
    h = rd.rd_schedule_create(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, p, 2 * n, 2 * 2048, *M1)
    try:
        rd.rd_allreduce(h, x, outs, rd.RD_SUM)
        torch.cuda.synchronize()
    finally:
        rd.rd_destroy(h)
    ev, off, _ = oracle_schedule(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, p, 2 * n, 2 * 2048, *M1)
    bits = lambda t: t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    want = O.reduce(ev, bits(x), off * 2, "sum", half="bf16")
    for i in range(p):
        assert bits(outs[i]).tobytes() == want.tobytes()


def test_overlapping_copies_are_refused():
    p, n = 4, 1024
    x = make_inputs(p, n, "normal", seed=1, device="cuda")
    outs = torch.empty_like(x)
    h = rd.rd_schedule_create(rd.RD_PIPELINE, rd.RD_PORT_UNI, p, 4 * n, 4 * 256, *M1)
    try:
        for bad in ([outs[0], outs[1], outs[1], outs[3]],           # two copies in one place
                    [outs[0], x[2], outs[2], outs[3]],               # process 1's copy over process 2's input
                    [x[1], outs[1], outs[2], outs[3]]):              # the root's copy over another process's input
            with pytest.raises(rd.RdError) as e:
                rd.rd_allreduce(h, x, bad, rd.RD_SUM)
            assert e.value.status == rd.RD_ERR_INVALID_ARG
    finally:
        rd.rd_destroy(h)


@pytest.mark.parametrize("algo,port", SCHEDULES)
def test_reduction_towards_another_root(algo, port):
    """The processes are interchangeable (Section II: homogeneous, fully connected), so reducing towards process r
    is the schedule with the processes relabelled: the pointer array is passed with buffer r first (here r and 0
    swap their roles).  The result is the oracle's for the relabelled inputs, exactly; as an integer sum it is the
    order-free sum; as an fp32 sum it is a different association from the one towards root 0."""
    p, n, seg, r = 13, 3 * 2048 + 36, 2048 + 520, 5
    perm = list(range(p))
    perm[0], perm[r] = perm[r], perm[0]
    for dist in ("normal", "int_pm2p20"):
        x = make_inputs(p, n, dist, seed=77, device="cuda")
        if dist == "normal":
            x *= 10.0 ** torch.randint(-4, 5, x.shape, device="cuda", generator=torch.Generator("cuda").manual_seed(1))
        h = rd.rd_schedule_create(algo, port, p, 4 * n, 4 * seg, *M1)
        try:
            out_r, out_0 = torch.empty(n, dtype=x.dtype, device="cuda"), torch.empty(n, dtype=x.dtype, device="cuda")
            rd.rd_reduce(h, [x[k] for k in perm], out_r, rd.RD_SUM)
            rd.rd_reduce(h, x, out_0, rd.RD_SUM)
            torch.cuda.synchronize()
        finally:
            rd.rd_destroy(h)
        ev, off, _ = oracle_schedule(algo, port, p, 4 * n, 4 * seg, *M1)
        xh = x.cpu().numpy()
        want = O.reduce(ev, np.ascontiguousarray(xh[perm]), off, "sum")         # process k of the schedule holds buffer perm[k]
        assert out_r.cpu().numpy().tobytes() == want.tobytes()
        if dist == "int_pm2p20":
            assert torch.equal(out_r, out_0)
        else:
            assert not torch.equal(out_r, out_0)                                # another association of the same terms
            ref, mag = O.reference_f64(xh, "sum")
            assert (np.abs(out_r.cpu().numpy().astype(np.float64) - ref) <= 1e-5 * mag).all()


def test_threads_with_their_own_schedules_launch_concurrently():
    """Distinct schedules may be used from distinct threads: four threads, each with its own schedule, stream and
    ring shape (stack depths 0 to 6, two or three thread blocks per SM, packed pointers and a pointer table),
    launch at the same time; every result is the oracle's."""
    cases = [(rd.RD_PIPELINE, rd.RD_PORT_UNI, 9, 2048 * 1500 + 36, 4 * (2048 + 520)), (rd.RD_BINOMIAL, rd.RD_PORT_UNI, 128, 2048 * 40, 4 * 4096),
             (rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, 5, 2048 * 37 + 8, 4 * 3000), (rd.RD_BI_GREEDY, rd.RD_PORT_BI, 300, 2048 * 6, 4 * 2048)]
    xs = [make_inputs(p, n, "normal", seed=60 + k, device="cuda") for k, (_, _, p, n, _) in enumerate(cases)]
    wants = []
    for (algo, port, p, n, seg), x in zip(cases, xs):
        ev, off, _ = oracle_schedule(algo, port, p, 4 * n, seg, *M1)
        wants.append(O.reduce(ev, x.cpu().numpy(), off, "sum"))
    torch.cuda.synchronize()
    errors = []
    gate = threading.Barrier(len(cases))

    def work(k):
        try:
            algo, port, p, n, seg = cases[k]
            torch.cuda.set_device(0)
            stream = torch.cuda.Stream()
            out = torch.empty(n, device="cuda")
            h = rd.rd_schedule_create(algo, port, p, 4 * n, seg, *M1)
            try:
                gate.wait()
                for rep in range(10):
                    with torch.cuda.stream(stream):
                        out.zero_()
                        rd.rd_reduce(h, xs[k], out, rd.RD_SUM, stream=stream)
                    stream.synchronize()
                    assert out.cpu().numpy().tobytes() == wants[k].tobytes(), (k, rep)
                assert rd.rd_schedule_status(h) == 0
            finally:
                rd.rd_destroy(h)
        except BaseException as e:          # noqa: BLE001 - reported by the main thread
            errors.append(repr(e))
            try:
                gate.abort()
            except Exception:
                pass

    threads = [threading.Thread(target=work, args=(k,)) for k in range(len(cases))]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
