"""Shared helpers of the tests (no method arithmetic of the library, no oracle internals)."""
import numpy as np

import paper_1310_4645_b200 as rd
from oracle import rd_oracle as O

TICK = 1e-15
ORDER = ["t_start", "seg", "src", "dst"]


def ticks(alpha, beta, gamma, tick=TICK):
    return int(round(alpha / tick)), int(round(beta / tick)), int(round(gamma / tick))


def oracle_schedule(algo, port, p, msg_bytes, seg_bytes, alpha, beta, gamma, sizes=None):
    """(events sorted like the library's export, segment offsets in elements, completion ticks)."""
    A, B, G = ticks(alpha, beta, gamma)
    bidir = port == rd.RD_PORT_BI
    if algo == rd.RD_BUTTERFLY:
        ev, off, comp = O.butterfly(p, msg_bytes // 4, 4, A, B, G)
        return np.sort(ev, order=ORDER), off, comp
    if sizes is None:
        sizes = O.equal_sizes(msg_bytes, min(seg_bytes, msg_bytes)) if msg_bytes else []
    if algo == rd.RD_UNI_GREEDY:
        ev, comp = O.uni_greedy(p, sizes, A, B, G)
    elif algo == rd.RD_BI_GREEDY:
        ev, comp = O.bi_greedy(p, sizes, A, B, G)
    elif algo == rd.RD_BINOMIAL:
        ev, comp = O.binomial(p, sizes, A, B, G)
    elif algo == rd.RD_PIPELINE:
        ev, comp = O.pipeline(p, sizes, A, B, G, bidir)
    elif algo == rd.RD_BINARY:
        ev, comp = O.binary(p, sizes, A, B, G, bidir)
    else:
        raise ValueError(algo)
    off = np.concatenate([[0], np.cumsum(np.asarray(sizes, dtype=np.int64) // 4)])
    return np.sort(ev, order=ORDER), off, comp


def run_program(ops, x, op, use_hints=True, depth_out=None):
    """Reference interpreter of one compiled combine program (format documented in include/rd.h).
    x: [p, len] array; returns the root's value.  Written from the header's description only.
    use_hints: honour bits 30 / 31 (sub-expressions that need no stack run in a second accumulator);
    depth_out: a list that receives the deepest the stack got."""
    x = np.asarray(x)

    def combine(held, incoming):
        if op == "sum":
            if x.dtype == np.int32:
                return (held.view(np.uint32) + incoming.view(np.uint32)).view(np.int32)
            return (held + incoming).astype(np.float32)
        if op == "prod":
            if x.dtype == np.int32:
                return (held.view(np.uint32) * incoming.view(np.uint32)).view(np.int32)
            return (held * incoming).astype(np.float32)
        if op == "min":
            return np.where(incoming < held, incoming, held)
        return np.where(incoming > held, incoming, held)

    stack, top, second = [], None, None
    loads = deepest = 0
    for w in ops:
        w = int(w)
        proc, kind, npop, roles = w & 0xFFF, (w >> 12) & 3, (w >> 14) & 0xF, (w >> 18) & 0xFFF
        aside, last = (w >> 30) & 1, (w >> 31) & 1
        v = x[proc]
        loads += 1
        assert not last or (aside and npop >= 1)
        first_pop = 0
        if aside and use_hints:
            # a sub-expression that needs no stack, evaluated in a second accumulator
            if kind == 1:
                assert second is None
                second = v.copy()
            else:
                assert kind in (2, 3) and second is not None
                second = combine(second, v) if kind == 2 else combine(v, second)
            assert npop == 0 or last                         # nothing is popped inside it
            if last:
                top = combine(top, second) if roles & 1 else combine(second, top)
                second, first_pop = None, 1
        else:
            assert second is None or not use_hints           # nothing else happens while one is under way
            if kind == 0:
                top = v.copy()
            elif kind == 1:
                stack.append(top)
                deepest = max(deepest, len(stack))
                top = v.copy()
            elif kind == 2:
                top = combine(top, v)
            else:
                top = combine(v, top)
        for k in range(first_pop, npop):
            y = stack.pop()
            top = combine(y, top) if (roles >> k) & 1 else combine(top, y)
    assert not stack and second is None and loads == x.shape[0]
    if depth_out is not None:
        depth_out.append(deepest)
    return top


M1_64 = (2e-6, 1e-10, 5e-11)
OPS64 = {"sum": rd.RD_SUM, "max": rd.RD_MAX, "min": rd.RD_MIN, "prod": rd.RD_PROD}


def check64(algo, port, x_dev, seg_bytes, op, exec_mode=0, rows=None, out=None, variant=None):
    """8-byte elements: the schedule counts in 4-byte words, the oracle in elements."""
    import torch
    p, n = x_dev.shape
    h = rd.rd_schedule_create(algo, port, p, 8 * n, seg_bytes, *M1_64)
    try:
        if variant is not None:
            rd.rd_schedule_set_tree_variant(h, variant)
        out = torch.full((n,), 77, dtype=x_dev.dtype, device=x_dev.device) if out is None else out
        rd.rd_reduce(h, rows if rows is not None else x_dev, out, OPS64[op], exec_mode=exec_mode, want_stats=exec_mode != rd.RD_EXEC_TREE)
        torch.cuda.synchronize()
    finally:
        rd.rd_destroy(h)
    ev, off, _ = oracle_schedule(algo, port, p, 8 * n, seg_bytes if seg_bytes else 8 * n, *M1_64)
    assert (off % 2 == 0).all()
    x = x_dev.cpu().numpy()
    want = O.reduce(ev, x, off // 2, op)
    got = out.cpu().numpy()
    assert got.tobytes() == want.tobytes()
    return got, x


def inputs64(p, n, kind, seed):
    import torch
    g = torch.Generator("cuda").manual_seed(seed)
    if kind == "int64":
        return torch.randint(-2**62, 2**62, (p, n), dtype=torch.int64, device="cuda", generator=g)
    if kind == "int64_small":
        return torch.randint(-3, 4, (p, n), dtype=torch.int64, device="cuda", generator=g) * 2 + 1
    x = torch.empty((p, n), dtype=torch.float64, device="cuda")
    if kind == "near_one":
        x.uniform_(0.5, 2.0, generator=g)
        return x * (torch.randint(0, 2, x.shape, device="cuda", generator=g) * 2.0 - 1.0)
    x.normal_(generator=g)
    return x * 10.0 ** torch.randint(-12, 13, x.shape, device="cuda", generator=g)
