"""The sweep workload at each schedule's own optimal segment size (Sections V-B and VII: every algorithm is
compared at its tuned segment size), against the oracle, bit for bit, through the C ABI (GPU).

A thinned grid of the sweep: p in {2, 16, 128, 1024} x message in {8 B, 4 KiB, 1 MiB, 64 MiB} x the six
schedules x {int32, fp32} x {sum, max}.  The library is asked for `seg_bytes = 0`, i.e. the segment size
rd_optimal_segment returns for the schedule; the oracle's own simulator then builds the schedule for that
segment size and its evaluator gives the expected bytes.  Where p * m is at most 256 MiB the whole message is
compared; above that, at least eight segments (the first two, the last three -- the last one is the
ragged one whenever the segment size does not divide the message -- and three in between) are: whole when
the segment's p operands fit in 64 MiB, else on its first, middle and last 16 MiB / 4p elements (the oracle
replays the segment's events on those element ranges; elements do not depend on each other).
Inputs: uniform random numbers from seed 4 (integers in [-2^20, 2^20], floats in [-1, 1)), as in the sweep.
"""
import numpy as np
import pytest
import torch

import paper_1310_4645_b200 as rd
from paper_1310_4645_b200.sweep import SCHEDULES, fill_arena, ALPHA, BETA, GAMMA
from oracle import rd_oracle as O
from helpers import oracle_schedule

pytestmark = pytest.mark.gpu

MODEL = (ALPHA, BETA, GAMMA)
OPS = {"sum": rd.RD_SUM, "max": rd.RD_MAX}
WHOLE_LIMIT = 256 << 20
SEGMENT_LIMIT = 64 << 20          # a picked segment is checked whole when its p operands are at most this many bytes
SLICE_BYTES = 16 << 20            # ... else on three slices of this many operand bytes each


def picked_segments(q):
    return sorted({0, 1, q // 3, q // 2, (2 * q) // 3, q - 3, q - 2, q - 1} & set(range(q)))


def run_case(p, m, x, out, name, algo, port, ops):
    n = m // 4
    seg = rd.rd_optimal_segment(algo, port, p, m, *MODEL)
    assert seg % 4 == 0 and 4 <= seg <= m
    h = rd.rd_schedule_create(algo, port, p, m, 0, *MODEL)                  # 0: the schedule's own optimum
    try:
        info = rd.rd_schedule_info(h)
        ev, off, comp = oracle_schedule(algo, port, p, m, seg, *MODEL)     # the oracle's schedule at that size
        assert info["predicted_ticks"] == comp, (name, p, m, seg)
        assert (rd.rd_schedule_segments(h).astype(np.int64) == off).all()
        q = len(off) - 1
        if algo != rd.RD_BUTTERFLY:
            assert q == -(-m // seg)
        whole = p * m <= WHOLE_LIMIT
        xh = x.cpu().numpy() if whole else None
        for opname in ops:
            out.fill_(77)
            rd.rd_reduce(h, x, out, OPS[opname])
            torch.cuda.synchronize()
            if whole:
                want = O.reduce(ev, xh, off, opname)
                assert out.cpu().numpy().tobytes() == want.tobytes(), (name, p, m, seg, opname, str(x.dtype))
                continue
            picks = [j for j in picked_segments(q) if off[j + 1] > off[j]]
            assert len(picks) >= min(8, q)
            for j in picks:
                lo, hi = int(off[j]), int(off[j + 1])
                sel = ev[ev["seg"] == j].copy()
                sel["seg"] = 0
                if (hi - lo) * p * 4 <= SEGMENT_LIMIT:
                    spans = [(lo, hi)]
                else:
                    w = max(4, SLICE_BYTES // (4 * p))
                    mid = lo + (hi - lo - w) // 2
                    spans = [(lo, lo + w), (mid, mid + w), (hi - w, hi)]
                for a, b in spans:
                    want = O.reduce(sel, x[:, a:b].cpu().numpy(), [0, b - a], opname)
                    assert out[a:b].cpu().numpy().tobytes() == want.tobytes(), (name, p, m, seg, opname, j, a)
            # and order free over the whole message: the maximum is the maximum
            if opname == "max":
                assert torch.equal(out, x.amax(dim=0))
    finally:
        rd.rd_destroy(h)
    return seg


@pytest.mark.parametrize("p", [2, 16, 128, 1024])
@pytest.mark.parametrize("m", [8, 4 << 10, 1 << 20, 64 << 20])
def test_sweep_cells_at_the_optimal_segment_size(p, m):
    free_b, _ = torch.cuda.mem_get_info()
    if free_b < p * m + m + (2 << 30):
        pytest.skip("needs %.1f GiB of device memory" % (p * m / 2**30))
    n = m // 4
    chosen = {}
    for dtype in (torch.int32, torch.float32):
        x = fill_arena(p * n, dtype, "cuda").view(p, n)
        out = torch.empty(n, dtype=dtype, device="cuda")
        for name, algo, port in SCHEDULES:
            chosen[name] = run_case(p, m, x, out, name, algo, port, ("sum", "max"))
        del x, out
        torch.cuda.empty_cache()
    # the tuned sizes are what the paper's protocol gives: one segment for binomial and the butterfly, and for
    # everything when the message is tiny; pipelined schedules cut large messages into many segments
    assert chosen["binomial"] == m and chosen["butterfly"] == m
    if m == 8:
        assert all(s == m for s in chosen.values())
    if m >= (1 << 20) and p >= 16:
        assert chosen["pipeline"] < m and chosen["uni_greedy"] < m and chosen["bi_greedy"] < m
