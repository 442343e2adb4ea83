"""The compiled combine programs: interpreted on the host (by an interpreter written from the
header's description) they give the oracle evaluator's bits for every schedule, dtype and op."""
import numpy as np
import pytest

import paper_1310_4645_b200 as rd
from oracle import rd_oracle as O
from helpers import oracle_schedule, run_program

M1 = (2e-6, 1e-10, 5e-11)
CASES = [(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI), (rd.RD_BI_GREEDY, rd.RD_PORT_BI), (rd.RD_BINOMIAL, rd.RD_PORT_UNI),
         (rd.RD_PIPELINE, rd.RD_PORT_UNI), (rd.RD_PIPELINE, rd.RD_PORT_BI), (rd.RD_BINARY, rd.RD_PORT_UNI),
         (rd.RD_BINARY, rd.RD_PORT_BI), (rd.RD_BUTTERFLY, rd.RD_PORT_BI)]


def wide_floats(rng, shape):
    return (rng.standard_normal(shape) * 10.0 ** rng.integers(-6, 7, size=shape)).astype(np.float32)


@pytest.mark.parametrize("algo,port", CASES)
@pytest.mark.parametrize("p", [1, 2, 3, 8, 21, 64])
def test_programs_reproduce_the_oracle(algo, port, p):
    msg, seg = 4 * 96, 4 * 16
    n = msg // 4
    rng = np.random.default_rng(1000 * algo + p)
    xf = wide_floats(rng, (p, n))
    xf[:, :8] = np.where(rng.random((p, 8)) < 0.5, 0.0, -0.0)           # signed zeros for max
    xi = rng.integers(-2**31, 2**31, size=(p, n), dtype=np.int64).astype(np.int32)
    h = rd.rd_schedule_create(algo, port, p, msg, seg, *M1)
    try:
        info = rd.rd_schedule_info(h)
        off = rd.rd_schedule_segments(h).astype(np.int64)
        oev, ooff, _ = oracle_schedule(algo, port, p, msg, seg, *M1)
        assert info["stack_depth"] <= max(1, int(np.ceil(np.log2(max(p, 2)))))
        xp = (rng.uniform(0.5, 2.0, size=(p, n)) * rng.choice([-1.0, 1.0], size=(p, n))).astype(np.float32)
        for x, ops_ in ((xf, ("sum", "max", "min")), (xi, ("sum", "max", "min", "prod")), (xp, ("prod",))):
            for op in ops_:
                want = O.reduce(oev, x, ooff, op)
                got = np.empty_like(want)
                for j in range(info["q"]):
                    ops = rd.rd_schedule_program(h, j)
                    assert sorted(int(w) & 0xFFF for w in ops) == list(range(p))     # every process exactly once
                    depth, depth_plain = [], []
                    got[off[j]:off[j + 1]] = run_program(ops, x[:, off[j]:off[j + 1]], op, depth_out=depth)
                    # bits 30 / 31 are hints: one plain stack gives the same bits, one level deeper at most
                    plain = run_program(ops, x[:, off[j]:off[j + 1]], op, use_hints=False, depth_out=depth_plain)
                    assert plain.tobytes() == got[off[j]:off[j + 1]].tobytes()
                    assert depth_plain[0] <= info["stack_depth"] and depth[0] <= max(depth_plain[0] - 1, 0)
                assert got.tobytes() == want.tobytes(), (op, x.dtype)
    finally:
        rd.rd_destroy(h)


def test_stack_depth_of_the_named_workloads():
    """Partial results kept besides the running one stay within log2 p."""
    for algo, port, p, msg, seg in ((rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, 64, 4 << 20, 16 << 10),
                                    (rd.RD_BI_GREEDY, rd.RD_PORT_BI, 256, 16 << 20, 64 << 10),
                                    (rd.RD_BUTTERFLY, rd.RD_PORT_BI, 256, 16 << 20, 0),
                                    (rd.RD_BINOMIAL, rd.RD_PORT_UNI, 1024, 1 << 20, 0),
                                    (rd.RD_PIPELINE, rd.RD_PORT_UNI, 1024, 1 << 20, 1 << 12)):
        h = rd.rd_schedule_create(algo, port, p, msg, seg, *M1)
        d = rd.rd_schedule_info(h)["stack_depth"]
        rd.rd_destroy(h)
        assert d <= int(np.log2(p)), (algo, d)
        if algo == rd.RD_PIPELINE:
            assert d == 0                      # a chain needs no stack at all
