"""Parity of the tree kernel with the oracle, element by element, through the C ABI (GPU)."""
import numpy as np
import pytest
import torch

import paper_1310_4645_b200 as rd
from paper_1310_4645_b200.inputs import make_inputs, WORKLOADS
from oracle import rd_oracle as O
from helpers import oracle_schedule, check64, inputs64

pytestmark = pytest.mark.gpu

M1 = (2e-6, 1e-10, 5e-11)
SCHEDULES = [("uni_greedy", rd.RD_UNI_GREEDY, rd.RD_PORT_UNI), ("bi_greedy", rd.RD_BI_GREEDY, rd.RD_PORT_BI),
             ("binomial", rd.RD_BINOMIAL, rd.RD_PORT_UNI), ("pipeline", rd.RD_PIPELINE, rd.RD_PORT_UNI),
             ("binary", rd.RD_BINARY, rd.RD_PORT_BI), ("butterfly", rd.RD_BUTTERFLY, rd.RD_PORT_BI)]
OPS = {"sum": rd.RD_SUM, "max": rd.RD_MAX, "min": rd.RD_MIN, "prod": rd.RD_PROD}


def gpu_reduce(algo, port, x_dev, seg_bytes, op, model=M1, out=None, rows=None, variant=None):
    p, n = x_dev.shape
    h = rd.rd_schedule_create(algo, port, p, 4 * n, seg_bytes, *model)
    try:
        if variant is not None:
            rd.rd_schedule_set_tree_variant(h, variant)
        out = torch.full((n,), 77, dtype=x_dev.dtype, device=x_dev.device) if out is None else out
        rd.rd_reduce(h, rows if rows is not None else x_dev, out, OPS[op])
        torch.cuda.synchronize()
    finally:
        rd.rd_destroy(h)
    return out


def check(algo, port, x_dev, seg_bytes, op, model=M1, variant=None):
    p, n = x_dev.shape
    got = gpu_reduce(algo, port, x_dev, seg_bytes, op, model, variant=variant).cpu().numpy()
    x = x_dev.cpu().numpy()
    ev, off, _ = oracle_schedule(algo, port, p, 4 * n, seg_bytes if seg_bytes else 4 * n, *model)
    want = O.reduce(ev, x, off, op)
    assert got.tobytes() == want.tobytes()
    return got, x


# (p, n, segment elements): several tiles (2048 elements each on the 128-bit path), ragged tails,
# segments shorter and longer than a tile, non-power-of-two process counts
SHAPES = [(8, 4096, 512), (5, 10000, 2500), (13, 3 * 2048 + 36, 2048 + 520), (64, 8192, 1024), (2, 4100, 4100),
          (33, 6000, 1000), (16, 128, 8), (1, 5000, 1000),
          # segments that start and end inside a 128-bit vector (the message itself is whole vectors)
          (8, 3000, 333), (16, 4100, 4100), (13, 6180, 999), (4, 64, 3), (8, 4096, 6), (32, 8192, 2049),
          # message lengths that are not whole vectors: the last elements go through the element kernel
          (8, 4099, 1000), (16, 2050, 2050), (5, 7, 2), (3, 3, 1), (8, 6151, 333),
          # one and two processes (the direct kernel by default): ragged tiles, segments off the vector boundary
          (2, 3 * 2048 + 36, 2048 + 520), (2, 6151, 333), (1, 4099, 1000), (2, 12288, 2048)]


@pytest.mark.parametrize("name,algo,port", SCHEDULES)
@pytest.mark.parametrize("dist,op", [("int_pm2p20", "sum"), ("int_pm2p20", "max"), ("normal", "sum"), ("normal", "max")])
def test_parity_small_shapes(name, algo, port, dist, op):
    for p, n, seg in SHAPES:
        x = make_inputs(p, n, dist, seed=p * 1000 + n, device="cuda")
        if dist == "normal":
            x *= 10.0 ** torch.randint(-4, 5, x.shape, device="cuda", generator=torch.Generator("cuda").manual_seed(1))
        check(algo, port, x, 4 * seg, op)


@pytest.mark.parametrize("name,algo,port", SCHEDULES)
@pytest.mark.parametrize("dist,op", [("int_pm2p20", "sum"), ("normal", "sum"), ("normal", "max")])
def test_parity_small_shapes_on_the_direct_kernel(name, algo, port, dist, op):
    """The library picks the streaming kernel by itself (the test above); here every shape with at most 8
    processes goes through the direct kernel.  Same bits."""
    for p, n, seg in SHAPES:
        if p > 8:
            continue
        x = make_inputs(p, n, dist, seed=p * 1000 + n, device="cuda")
        check(algo, port, x, 4 * seg, op, variant=rd.RD_TREE_DIRECT)


@pytest.mark.parametrize("name,algo,port", SCHEDULES)
@pytest.mark.parametrize("dist,op", [("int_pm2p20", "sum"), ("normal", "sum"), ("normal", "max")])
def test_parity_small_shapes_with_two_operand_tiles_per_stage(name, algo, port, dist, op):
    """The streaming kernel on tiles of 1024 words, two operands to a ring stage (what the 16-bit types use
    by default), asked for here with 4-byte elements: odd process counts leave the last stage of a tile half
    full, p = 1 and p = 2 have a single stage per tile.  Same bits."""
    for p, n, seg in SHAPES:
        x = make_inputs(p, n, dist, seed=p * 1000 + n, device="cuda")
        check(algo, port, x, 4 * seg, op, variant=rd.RD_TREE_STREAM_PAIRED)


def test_two_operand_tiles_per_stage_deep_stacks_and_many_tiles():
    """Many tiles per thread block, stacks up to depth 8 (binomial, p = 300), eight-byte elements."""
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    for p, n, seg, (name, algo, port) in [(9, 1024 * 7 * sms + 100, 3 * 1024 + 520, SCHEDULES[0]), (300, 1024 * 40 + 8, 4096, SCHEDULES[2]),
                                          (128, 1024 * 5 * sms, 4096, SCHEDULES[1]), (3, 1024 * 9 * sms + 8, 2048 + 520, SCHEDULES[5])]:
        x = make_inputs(p, n, "normal", seed=p + n, device="cuda")
        h = rd.rd_schedule_create(algo, port, p, 4 * n, 4 * seg, *M1)
        try:
            rd.rd_schedule_set_tree_variant(h, rd.RD_TREE_STREAM_PAIRED)
            shape = rd.rd_schedule_tree_shape(h)
        finally:
            rd.rd_destroy(h)
        assert shape["variant"] == rd.RD_TREE_STREAM_PAIRED and shape["n_tiles"] >= n // 1024
        check(algo, port, x, 4 * seg, "sum", variant=rd.RD_TREE_STREAM_PAIRED)
    for kind, op in (("int64", "sum"), ("fp64", "sum"), ("fp64", "max")):
        x = inputs64(13, 3 * 2048 + 36, kind, seed=21)
        check64(rd.RD_BI_GREEDY, rd.RD_PORT_BI, x, 8 * (1024 + 260), op, variant=rd.RD_TREE_STREAM_PAIRED)


def test_launch_shapes_two_and_three_blocks_per_sm():
    """The streaming kernel runs two or three thread blocks per SM depending on the number of tiles and on
    the stack depth; the direct kernel runs when asked for.  Every shape, element by element."""
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    seen = set()
    # (p, n, segment elements, schedule): few tiles; between two and three blocks' worth of tiles; many tiles
    # with ragged segments; a deep stack (binomial, p = 128) with many tiles; one or two processes
    cases = [(5, 2048 * 40 + 36, 2048 + 520, SCHEDULES[0]), (5, 2048 * (2 * sms + 40) + 36, 4096, SCHEDULES[3]),
             (9, 2048 * 7 * sms + 100, 3 * 2048 + 520, SCHEDULES[0]), (128, 2048 * 5 * sms, 4096, SCHEDULES[2]),
             (2, 2048 * 9 * sms + 8, 2048 + 520, SCHEDULES[1]), (1, 2048 * 3 + 4, 1000, SCHEDULES[3])]
    for p, n, seg, (name, algo, port) in cases:
        x = make_inputs(p, n, "normal", seed=p + n, device="cuda")
        variant = rd.RD_TREE_DIRECT if p <= 2 else None
        h = rd.rd_schedule_create(algo, port, p, 4 * n, 4 * seg, *M1)
        try:
            if variant is not None:
                rd.rd_schedule_set_tree_variant(h, variant)
            shape = rd.rd_schedule_tree_shape(h)
        finally:
            rd.rd_destroy(h)
        seen.add((shape["variant"], shape["blocks_per_sm"]))
        assert shape["n_tiles"] >= n // 2048
        assert (shape["variant"] == rd.RD_TREE_DIRECT) == (p <= 2)
        assert shape["ring_stages"] >= 3 or shape["variant"] == rd.RD_TREE_DIRECT
        check(algo, port, x, 4 * seg, "sum", variant=variant)
        check(algo, port, x, 4 * seg, "sum")                          # and the library's own choice
    assert (rd.RD_TREE_STREAM, 2) in seen and (rd.RD_TREE_STREAM, 3) in seen and (rd.RD_TREE_DIRECT, 4) in seen


def test_direct_kernel_limits():
    """The direct kernel holds all operands of an element in registers: at most 8 processes."""
    h = rd.rd_schedule_create(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, 9, 4096, 1024, *M1)
    try:
        with pytest.raises(rd.RdError) as e:
            rd.rd_schedule_set_tree_variant(h, rd.RD_TREE_DIRECT)
        assert e.value.status == rd.RD_ERR_UNSUPPORTED
        with pytest.raises(rd.RdError) as e:
            rd.rd_schedule_set_tree_variant(h, 7)
        assert e.value.status == rd.RD_ERR_INVALID_ARG
        rd.rd_schedule_set_tree_variant(h, rd.RD_TREE_STREAM)
        rd.rd_schedule_set_tree_variant(h, rd.RD_TREE_AUTO)
    finally:
        rd.rd_destroy(h)
    # every process count the direct kernel serves, every schedule, with both kernels on the same inputs
    for p in range(1, 9):
        n = 2048 * 3 + 4 * p
        x = make_inputs(p, n, "normal", seed=p, device="cuda")
        for name, algo, port in SCHEDULES:
            a = gpu_reduce(algo, port, x, 4 * 1000, "sum", variant=rd.RD_TREE_DIRECT)
            b = gpu_reduce(algo, port, x, 4 * 1000, "sum", variant=rd.RD_TREE_STREAM)
            assert torch.equal(a.view(torch.int32), b.view(torch.int32)), (p, name)
            check(algo, port, x, 4 * 1000, "max", variant=rd.RD_TREE_DIRECT)


@pytest.mark.parametrize("name,algo,port", SCHEDULES)
@pytest.mark.parametrize("dist,op", [("int_pm2p20", "min"), ("int_pm2p20", "prod"), ("normal", "min"), ("near_one", "prod")])
def test_parity_min_and_product(name, algo, port, dist, op):
    """Integer results are also checked against the order-free value; fp32 products use factors with
    magnitude in [0.5, 2) so that no partial product overflows to a NaN-producing inf * 0."""
    for p, n, seg in SHAPES:
        if dist == "near_one":
            g = torch.Generator("cuda").manual_seed(p * 1000 + n)
            x = torch.empty((p, n), device="cuda").uniform_(0.5, 2.0, generator=g)
            x *= torch.randint(0, 2, x.shape, device="cuda", generator=g) * 2.0 - 1.0
        else:
            x = make_inputs(p, n, dist, seed=p * 1000 + n, device="cuda")
        got, xh = check(algo, port, x, 4 * seg, op)
        if op == "min":
            assert (got == xh.min(axis=0)).all()
        elif dist == "int_pm2p20":
            want = np.multiply.reduce(xh.view(np.uint32), axis=0, dtype=np.uint32).view(np.int32)
            assert (got == want).all()


# (p, n, segment elements) for 8-byte elements: tiles hold 1024 of them; segments that begin 8 bytes
# into a 128-bit vector; message lengths that are not whole vectors
SHAPES64 = [(8, 4096, 512), (5, 10000, 2500), (13, 3 * 1024 + 18, 1024 + 261), (64, 4096, 512), (2, 2050, 2050),
            (33, 3000, 501), (16, 64, 4), (1, 2500, 500), (8, 1501, 333), (3, 3, 1), (8, 3077, 167)]


@pytest.mark.parametrize("name,algo,port", [s for s in SCHEDULES if s[0] != "butterfly"])
@pytest.mark.parametrize("kind,op", [("int64", "sum"), ("int64", "max"), ("int64", "min"), ("int64_small", "prod"),
                                     ("normal64", "sum"), ("normal64", "max"), ("normal64", "min"), ("near_one", "prod")])
def test_parity_eight_byte_elements(name, algo, port, kind, op):
    for p, n, seg in SHAPES64:
        x = inputs64(p, n, kind, seed=p * 1000 + n)
        got, xh = check64(algo, port, x, 8 * seg, op)
        if kind.startswith("int64") and op in ("sum", "max", "min"):
            want = {"sum": lambda: x.sum(dim=0), "max": lambda: x.amax(dim=0), "min": lambda: x.amin(dim=0)}[op]()
            assert (got == want.cpu().numpy()).all()                   # torch's int64 sum wraps as well


def test_eight_byte_elements_on_the_direct_kernel():
    for name, algo, port in SCHEDULES[:5]:
        for p, n, seg in SHAPES64:
            if p > 8:
                continue
            v = rd.RD_TREE_DIRECT
            check64(algo, port, inputs64(p, n, "normal64", seed=p + n), 8 * seg, "sum", variant=v)
            check64(algo, port, inputs64(p, n, "int64", seed=p + n), 8 * seg, "max", variant=v)
            check64(algo, port, inputs64(p, n, "near_one", seed=p + n), 8 * seg, "prod", variant=v)


def test_eight_byte_elements_butterfly_and_odd_boundaries():
    """Halving keeps chunk boundaries on elements when n is a multiple of the power of two below p;
    otherwise a boundary would fall inside an element and the call is refused."""
    for p, n in ((8, 4096), (13, 1024 + 8), (32, 2048 + 32)):
        check64(rd.RD_BUTTERFLY, rd.RD_PORT_BI, inputs64(p, n, "normal64", seed=p), 0, "sum")
        check64(rd.RD_BUTTERFLY, rd.RD_PORT_BI, inputs64(p, n, "int64", seed=p), 0, "max")
    x = inputs64(8, 4099, "normal64", seed=1)
    with pytest.raises(rd.RdError) as e:
        check64(rd.RD_BUTTERFLY, rd.RD_PORT_BI, x, 0, "sum")
    assert e.value.status == rd.RD_ERR_INVALID_ARG
    with pytest.raises(rd.RdError) as e:
        check64(rd.RD_PIPELINE, rd.RD_PORT_UNI, x, 12, "sum")           # 12-byte segments split elements
    assert e.value.status == rd.RD_ERR_INVALID_ARG


def test_eight_byte_elements_off_the_vector_boundary():
    """Buffers that start 8 bytes into a 128-bit vector take the element path (one element per thread)."""
    p, n = 8, 3003
    big = inputs64(p, n + 1, "normal64", seed=6)
    rows = [big[i, 1:] for i in range(p)]
    assert rows[0].data_ptr() % 16 == 8
    out_big = torch.zeros(n + 1, dtype=torch.float64, device="cuda")
    check64(rd.RD_BI_GREEDY, rd.RD_PORT_BI, big[:, 1:], 8 * 512, "sum", rows=rows, out=out_big[1:])
    assert out_big[0].item() == 0.0


def test_fp64_keeps_what_fp32_would_lose():
    """2^30 + 1 + ... : exact in fp64 for any order, and different from an fp32 evaluation."""
    p, n = 16, 4096
    x = torch.ones((p, n), dtype=torch.float64, device="cuda")
    x[0] = 2.0 ** 40
    got, _ = check64(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, x, 8 * 512, "sum")
    assert (got == 2.0 ** 40 + 15).all()


def test_config1_bit_exact_and_order_free():
    """p = 8, 4096 int32, 8 segments of 512, uni-greedy, wrapping sum."""
    w = WORKLOADS["config1"]
    x = make_inputs(w["p"], w["n"], w["dist"], w["seed"], device="cuda")
    got, xh = check(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, x, w["seg_bytes"], "sum", (w["alpha"], w["beta"], w["gamma"]))
    assert (got == xh.astype(np.int64).sum(axis=0).astype(np.int32)).all()


def test_int32_sum_wraps():
    x = torch.full((8, 4096), 2**30, dtype=torch.int32, device="cuda")
    got, _ = check(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, x, 2048, "sum")
    assert (got == 0).all()            # 8 * 2^30 = 2^33 = 0 mod 2^32


@pytest.mark.parametrize("name,algo,port", SCHEDULES)
def test_element_path_for_unaligned_segments_and_buffers(name, algo, port):
    """Segment sizes that are not multiples of 16 bytes, and buffers that start 4 bytes off a 16-byte
    boundary, take the one-element-per-lane path."""
    p, n = 8, 3003
    x = make_inputs(p, n, "normal", seed=5, device="cuda")
    check(algo, port, x, 4 * 333, "sum")
    # misaligned views: row i starts at element 1 of a longer buffer
    big = make_inputs(p, n + 1, "normal", seed=6, device="cuda")
    rows = [big[i, 1:] for i in range(p)]
    assert rows[0].data_ptr() % 16 == 4
    out_big = torch.zeros(n + 1, dtype=torch.float32, device="cuda")
    gpu_reduce(algo, port, big[:, 1:], 4 * 1024, "sum", out=out_big[1:], rows=rows)
    ev, off, _ = oracle_schedule(algo, port, p, 4 * n, 4 * 1024, *M1)
    want = O.reduce(ev, big[:, 1:].cpu().numpy().copy(), off, "sum")
    assert out_big[1:].cpu().numpy().tobytes() == want.tobytes()
    assert out_big[0].item() == 0.0                                    # nothing written before the view


def test_signed_zero_and_inf_follow_the_held_incoming_rule():
    p, n = 16, 4096
    g = torch.Generator("cuda").manual_seed(3)
    choices = torch.tensor([0.0, -0.0, 1.0, -1.0, float("inf"), -float("inf")], device="cuda")
    x = choices[torch.randint(0, 6, (p, n), device="cuda", generator=g)].contiguous()
    for name, algo, port in SCHEDULES:
        check(algo, port, x, 4 * 512, "max")
    x = choices[torch.randint(0, 5, (p, n), device="cuda", generator=g)].contiguous()     # no -inf: inf - inf is NaN
    for name, algo, port in SCHEDULES:
        check(algo, port, x, 4 * 512, "sum")


def test_denormals_are_not_flushed():
    p, n = 4, 2048
    tiny = np.float32(2.0 ** -149)                                             # smallest subnormal
    x = torch.full((p, n), float(tiny), dtype=torch.float32, device="cuda")
    got, _ = check(rd.RD_BINOMIAL, rd.RD_PORT_UNI, x, 0, "sum")
    assert (got == np.float32(2.0 ** -147)).all() and got[0] > 0


def test_output_may_alias_the_roots_input():
    p, n = 8, 8192
    x = make_inputs(p, n, "normal", seed=9, device="cuda")
    keep = x.clone()
    gpu_reduce(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, x, 4096, "sum", out=x[0])
    ev, off, _ = oracle_schedule(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, p, 4 * n, 4096, *M1)
    want = O.reduce(ev, keep.cpu().numpy(), off, "sum")
    assert x[0].cpu().numpy().tobytes() == want.tobytes()
    assert torch.equal(x[1:], keep[1:])                                # inputs are never written


def test_many_processes_use_the_pointer_table():
    """More processes than fit in the kernel's parameter block."""
    p, n = 300, 4096
    x = make_inputs(p, n, "uniform_pm1", seed=2, device="cuda")
    for _ in range(3):                                                 # cycles the table slots
        check(rd.RD_BI_GREEDY, rd.RD_PORT_BI, x, 4096, "sum")
    p, n = 1024, 2048
    x = make_inputs(p, n, "uniform_pm1", seed=2, device="cuda")
    check(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, x, 2048, "sum")
    check(rd.RD_BUTTERFLY, rd.RD_PORT_BI, x, 0, "max")


def test_empty_message_and_stats():
    x = torch.zeros((4, 0), dtype=torch.float32, device="cuda")
    h = rd.rd_schedule_create(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, 4, 0, 16, *M1)
    rd.rd_reduce(h, x, torch.zeros(0, device="cuda"), rd.RD_SUM)
    rd.rd_destroy(h)
    x = make_inputs(8, 1 << 16, "normal", seed=1, device="cuda")
    out = torch.empty(1 << 16, device="cuda")
    h = rd.rd_schedule_create(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, 8, 4 << 16, 4096, *M1)
    assert rd.rd_schedule_status(h) == 0                         # nothing has run yet
    st = rd.rd_reduce(h, x, out, rd.RD_SUM, want_stats=True)
    assert rd.rd_schedule_status(h) == 0
    assert st.kernel_ms > 0 and st.bytes_moved == 9 * (4 << 16) and st.n_launches == 1
    assert abs(st.predicted_s - rd.rd_schedule_info(h)["predicted_seconds"]) < 1e-12
    with pytest.raises(rd.RdError) as e:
        rd.rd_reduce(h, x[:, :100].contiguous(), out[:100], rd.RD_SUM)
    assert e.value.status == rd.RD_ERR_SIZE_MISMATCH
    rd.rd_destroy(h)


def test_reduce_host_round_trip():
    p, n = 8, 10000
    x = make_inputs(p, n, "normal", seed=4, device="cpu").pin_memory()
    out = torch.empty(n, dtype=torch.float32).pin_memory()
    staging = torch.empty((p + 1) * n, dtype=torch.float32, device="cuda")
    h = rd.rd_schedule_create(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, p, 4 * n, 4000, *M1)
    rd.rd_reduce_host(h, x, out, staging, rd.RD_SUM)
    ev, off, _ = oracle_schedule(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, p, 4 * n, 4000, *M1)
    want = O.reduce(ev, x.numpy(), off, "sum").tobytes()
    assert out.numpy().tobytes() == want
    # rows of one array travel in one copy; rows scattered over the host (here: in reverse order of address,
    # and two of them in buffers of their own) are copied one by one
    back = torch.empty((p, n), dtype=torch.float32).pin_memory()
    rows = [back[p - 1 - i] for i in range(p)]
    rows[2], rows[5] = torch.empty(n).pin_memory(), torch.empty(n, dtype=torch.float32)        # one of them pageable
    for i in range(p):
        rows[i].copy_(x[i])
    out.zero_()
    rd.rd_reduce_host(h, rows, out, staging, rd.RD_SUM)
    rd.rd_destroy(h)
    assert out.numpy().tobytes() == want


@pytest.mark.parametrize("name,algo,port", SCHEDULES[:5])
def test_config2_shape_full_size(name, algo, port):
    """p = 64, n = 2^20 fp32 N(0,1), 16 KB segments: bit-exact against the oracle on every element of
    sampled segments, and within 1e-5 * sum|x_i| of the fp64 sum everywhere."""
    w = WORKLOADS["config2"]
    model = (w["alpha"], w["beta"], w["gamma"])
    x = make_inputs(w["p"], w["n"], w["dist"], w["seed"], device="cuda")
    got = gpu_reduce(algo, port, x, w["seg_bytes"], "sum", model).cpu().numpy()
    xh = x.cpu().numpy()
    ev, off, _ = oracle_schedule(algo, port, w["p"], 4 * w["n"], w["seg_bytes"], *model)
    q = len(off) - 1
    for j in sorted(set([0, 1, q // 3, q // 2, q - 2, q - 1])):
        sel = ev[ev["seg"] == j].copy()
        sel["seg"] = 0
        sl = slice(int(off[j]), int(off[j + 1]))
        want = O.reduce(sel, np.ascontiguousarray(xh[:, sl]), [0, sl.stop - sl.start], "sum")
        assert got[sl].tobytes() == want.tobytes(), j
    ref, mag = O.reference_f64(xh, "sum")
    assert (np.abs(got.astype(np.float64) - ref) <= 1e-5 * mag).all()
    assert np.abs(got - ref).max() / np.abs(ref).max() <= 1e-5


@pytest.mark.parametrize("mode", [rd.RD_EXEC_TREE, rd.RD_EXEC_FAITHFUL])
def test_unequal_segmentation_end_to_end(mode):
    """Section VIII: segments of different sizes, e.g. (5,3,2) and (3,2,2,2,1) tenths of the message;
    both kernels execute the uni-greedy / bi-greedy / pipeline schedules built for them, bit for bit."""
    from helpers import ticks
    p = 12
    for parts in ((5, 3, 2), (3, 2, 2, 2, 1), (2, 2, 1, 1, 1, 1, 1, 1), (10,)):
        unit = 412                                           # elements per tenth: segments are not vector aligned
        sizes = [4 * unit * k for k in parts]
        n = unit * 10
        x = make_inputs(p, n, "normal", seed=sum(parts) + len(parts), device="cuda")
        x *= 10.0 ** torch.randint(-4, 5, x.shape, device="cuda", generator=torch.Generator("cuda").manual_seed(2))
        for algo, port in ((rd.RD_UNI_GREEDY, rd.RD_PORT_UNI), (rd.RD_BI_GREEDY, rd.RD_PORT_BI), (rd.RD_PIPELINE, rd.RD_PORT_BI)):
            h = rd.rd_schedule_create_segments(algo, port, p, sizes, *M1)
            out = torch.empty(n, device="cuda")
            rd.rd_reduce(h, x, out, rd.RD_SUM, exec_mode=mode)
            torch.cuda.synchronize()
            rd.rd_destroy(h)
            ev, off, _ = oracle_schedule(algo, port, p, 4 * n, 0, *M1, sizes=sizes)
            want = O.reduce(ev, x.cpu().numpy(), off, "sum")
            assert out.cpu().numpy().tobytes() == want.tobytes(), (parts, algo)


def _device_fp64_bound(x, out):
    """|r - r64| <= 1e-5 * sum_i |x_i| on EVERY element, the fp64 sums taken on the device slab by slab; returns
    the largest error relative to the largest |r64| as well."""
    n = out.numel()
    slab = max(1 << 16, (1 << 27) // x.shape[0])          # 1 GiB of fp64 operands at a time
    worst, biggest = 0.0, 0.0
    for lo in range(0, n, slab):
        xs = x[:, lo:lo + slab].double()
        ref, mag = xs.sum(dim=0), xs.abs().sum(dim=0)
        err = (out[lo:lo + slab].double() - ref).abs()
        assert bool((err <= 1e-5 * mag).all()), lo
        worst, biggest = max(worst, float(err.max())), max(biggest, float(ref.abs().max()))
    assert worst / biggest <= 1e-5
    return worst / biggest


def _full_size_parity(wname, schedules, ops, n_samples=16, whole_message_for=()):
    """A full-size workload in the launch configuration the benchmark uses (one rd_reduce call per schedule and
    operation on the resident arena).  What is compared, and on which fraction of the output elements:
      * bit for bit against the oracle -- its own simulator's schedule, its evaluator -- on n_samples whole
        segments per schedule and operation (the first two, the last four, which are the tiles handed out last,
        and others spread evenly): n_samples / q of the elements; for the schedules in `whole_message_for`
        on every element (fraction 1.0);
      * `max`: equal to the order-free maximum taken on the device, on every element (fraction 1.0);
      * `sum`: within 1e-5 * sum|x_i| of the fp64 sum taken on the device, on every element (fraction 1.0).
    Returns the fractions so that the callers can state them."""
    w = WORKLOADS[wname]
    model = (w["alpha"], w["beta"], w["gamma"])
    p, n = w["p"], w["n"]
    x = make_inputs(p, n, w["dist"], w["seed"], device="cuda")
    tab = rd.PointerTable(x)
    out = torch.empty(n, device="cuda")
    want_max = x.amax(dim=0) if "max" in ops else None
    fractions = {}
    for algo, port in schedules:
        h = rd.rd_schedule_create(algo, port, p, 4 * n, w["seg_bytes"], *model)
        oev, off, comp = oracle_schedule(algo, port, p, 4 * n, w["seg_bytes"], *model)     # the oracle's own events
        assert rd.rd_schedule_info(h)["predicted_ticks"] == comp
        assert (rd.rd_schedule_segments(h).astype(np.int64) == off).all()
        q = len(off) - 1
        picks = {0, 1, q - 4, q - 3, q - 2, q - 1} & set(range(q))
        for j in np.linspace(2, q - 5, max(n_samples - 6, 0) * 2).astype(int):     # others, spread evenly
            if len(picks) < min(n_samples, q) and 0 <= j < q:
                picks.add(int(j))
        picks = sorted(picks)
        assert len(picks) >= min(n_samples, q)
        xh = x.cpu().numpy() if algo in whole_message_for else None
        for op in ops:
            out.fill_(7.0)
            rd.rd_reduce(h, tab, out, OPS[op])
            torch.cuda.synchronize()
            covered = 0
            if xh is not None:
                want = O.reduce(oev, xh, off, op)
                assert out.cpu().numpy().tobytes() == want.tobytes(), (wname, algo, op)
                covered = n
            else:
                for j in picks:
                    lo, hi = int(off[j]), int(off[j + 1])
                    if hi == lo:
                        continue
                    sel = oev[oev["seg"] == j].copy()
                    sel["seg"] = 0
                    want = O.reduce(sel, x[:, lo:hi].cpu().numpy(), [0, hi - lo], op)
                    assert out[lo:hi].cpu().numpy().tobytes() == want.tobytes(), (wname, algo, op, j)
                    covered += hi - lo
            fractions[(algo, op, "oracle")] = covered / n
            if op == "max":
                assert torch.equal(out, want_max), (wname, algo)
                fractions[(algo, op, "order_free")] = 1.0
            if op == "sum":
                _device_fp64_bound(x, out)
                fractions[(algo, op, "fp64_bound")] = 1.0
        del xh
        rd.rd_destroy(h)
    return fractions


def test_config3_full_size():
    """p = 256, n = 2^22 fp32 uniform [-1, 1), 64 KiB segments, two ports: bi-greedy, butterfly and the trees.
    bi-greedy is evaluated by the oracle end to end (every element, 4 GiB of inputs on the host); the other
    four schedules on 16 of their 256 segments (butterfly: of its 256 chunks); the fp64 bound on every element
    for all five."""
    fr = _full_size_parity("config3", [(rd.RD_BI_GREEDY, rd.RD_PORT_BI), (rd.RD_BUTTERFLY, rd.RD_PORT_BI),
                                        (rd.RD_BINOMIAL, rd.RD_PORT_BI), (rd.RD_PIPELINE, rd.RD_PORT_BI),
                                        (rd.RD_BINARY, rd.RD_PORT_BI)], ["sum"], n_samples=16,
                            whole_message_for=(rd.RD_BI_GREEDY,))
    assert fr[(rd.RD_BI_GREEDY, "sum", "oracle")] == 1.0
    assert all(v >= 16 / 256 for k, v in fr.items() if k[2] == "oracle")
    assert all(v == 1.0 for k, v in fr.items() if k[2] != "oracle")


def test_config4_full_size():
    """p = 32, n = 2^28 fp32 N(0,1) (32 GiB), 1 MiB segments: uni- and bi-greedy, sum and max.  The oracle sees
    16 of the 1024 segments per schedule and operation (1/64 of the elements, among them the last four);
    the maximum and the fp64 bound are checked on every element."""
    free_b, _ = torch.cuda.mem_get_info()
    if free_b < (48 << 30):
        pytest.skip("needs 40 GiB of device memory")
    fr = _full_size_parity("config4", [(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI), (rd.RD_BI_GREEDY, rd.RD_PORT_BI)], ["sum", "max"],
                            n_samples=16)
    assert all(v >= 16 / 1024 for k, v in fr.items() if k[2] == "oracle")
    assert all(v == 1.0 for k, v in fr.items() if k[2] != "oracle")


def test_tree_mode_launches_can_be_replayed_from_a_cuda_graph():
    """Small messages are launch bound; after one ordinary call per schedule (which uploads its tables and
    configures the kernel) a tree-mode rd_reduce with at most 256 processes is a single kernel launch and
    can be recorded into a CUDA graph and replayed."""
    p, n = 8, 4096
    xs = [make_inputs(p, n, "normal", seed=s, device="cuda") for s in range(3)]
    outs = [torch.zeros(n, device="cuda") for _ in range(3)]
    tabs = [rd.PointerTable(x) for x in xs]
    hs = [rd.rd_schedule_create(a, pt, p, 4 * n, 2048, *M1) for a, pt in
          ((rd.RD_UNI_GREEDY, rd.RD_PORT_UNI), (rd.RD_BINOMIAL, rd.RD_PORT_UNI), (rd.RD_BI_GREEDY, rd.RD_PORT_BI))]
    want = []
    for h, t, o in zip(hs, tabs, outs):
        rd.rd_reduce(h, t, o, rd.RD_SUM)                 # ordinary call first
    torch.cuda.synchronize()
    want = [o.clone() for o in outs]
    for o in outs:
        o.zero_()
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            for _ in range(4):
                for h, t, o in zip(hs, tabs, outs):
                    rd.rd_reduce(h, t, o, rd.RD_SUM, stream=stream)
    graph.replay()
    torch.cuda.synchronize()
    for o, w in zip(outs, want):
        assert torch.equal(o, w)
    # the same for a batch that fits the kernel's parameters (one launch, nothing copied ahead of it) and for
    # the direct kernel (two processes)
    h2 = rd.rd_schedule_create(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, 2, 4 * n, 2048, *M1)
    o2, w2 = torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")
    batch = rd.Batch([(h, t, o) for h, t, o in zip(hs, tabs, outs)])
    rd.rd_schedule_set_tree_variant(h2, rd.RD_TREE_DIRECT)
    rd.rd_reduce_batch(batch, rd.RD_SUM)                 # ordinary calls first
    rd.rd_reduce(h2, xs[0][:2], w2, rd.RD_SUM)
    torch.cuda.synchronize()
    assert rd.rd_schedule_tree_shape(h2)["variant"] == rd.RD_TREE_DIRECT
    for o, w in zip(outs, want):
        assert torch.equal(o, w)
        o.zero_()
    graph2 = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph2, stream=stream):
            for _ in range(3):
                rd.rd_reduce_batch(batch, rd.RD_SUM, stream=stream)
                rd.rd_reduce(h2, xs[0][:2], o2, rd.RD_SUM, stream=stream)
    graph2.replay()
    torch.cuda.synchronize()
    for o, w in zip(outs, want):
        assert torch.equal(o, w)
    assert torch.equal(o2, w2)
    for h in hs + [h2]:
        rd.rd_destroy(h)


def test_largest_process_count():
    """p = 4096, the boundary's maximum: the tree kernel runs it (deepest stacks, pointer table); the
    schedule-faithful kernel cannot keep that many processes resident and says so."""
    p, n = 4096, 512
    x = make_inputs(p, n, "int_pm2p20", seed=8, device="cuda")
    for algo, port, seg in ((rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, 1024), (rd.RD_BINOMIAL, rd.RD_PORT_BI, 0),
                            (rd.RD_BINARY, rd.RD_PORT_UNI, 512)):
        check(algo, port, x, seg, "sum")
    h = rd.rd_schedule_create(rd.RD_BINOMIAL, rd.RD_PORT_UNI, p, 4 * n, 0, *M1)
    out = torch.empty(n, dtype=torch.int32, device="cuda")
    with pytest.raises(rd.RdError) as e:
        rd.rd_reduce(h, x, out, rd.RD_SUM, exec_mode=rd.RD_EXEC_FAITHFUL)
    assert e.value.status == rd.RD_ERR_UNSUPPORTED
    rd.rd_destroy(h)


def test_randomized_shapes_order_free_results():
    """200 seeded random shapes (process counts, message lengths and segment sizes with no regard for vector
    or tile boundaries, every schedule): int32 sum and max do not depend on the combine order, so torch's own
    reductions are an exact reference at any size."""
    rng = np.random.default_rng(12345)
    for case in range(200):
        name, algo, port = SCHEDULES[case % len(SCHEDULES)]
        p = int(rng.choice([2, 3, 5, 8, 17, 40, 64, 100, 257, 300]))
        n = int(rng.integers(1, 30000))
        seg = int(rng.integers(1, n + 1)) if rng.random() < 0.5 else int(rng.integers(1, 600))
        x = make_inputs(p, n, "int_pm2p20", seed=case, device="cuda")
        x = x * int(rng.integers(1, 5000))                        # let sums wrap now and then
        h = rd.rd_schedule_create(algo, port, p, 4 * n, 4 * seg, *M1)
        out = torch.empty(n, dtype=torch.int32, device="cuda")
        try:
            for op, want in ((rd.RD_SUM, x.sum(dim=0, dtype=torch.int64)), (rd.RD_MAX, x.amax(dim=0))):
                out.fill_(-7)
                rd.rd_reduce(h, x, out, op)
                if op == rd.RD_SUM:
                    want = ((want + (1 << 31)) % (1 << 32) - (1 << 31)).to(torch.int32)
                assert torch.equal(out, want), (case, name, p, n, seg, op)
        finally:
            rd.rd_destroy(h)


def test_randomized_shapes_types_and_operations_against_the_oracle():
    """150 seeded random cases over every element type, operation and schedule, with process counts, message
    lengths and segment sizes that respect no vector or tile boundary: the oracle's bytes, exactly.  A third of the
    fp32 cases carry signed zeros, subnormals and the smallest normal number among their inputs (no infinities:
    inf - inf would be a NaN, whose bit pattern is the machine's own)."""
    rng = np.random.default_rng(4645)
    special = torch.tensor([0.0, -0.0, 1.0, -1.0, 2.0 ** -149, -(2.0 ** -149), 2.0 ** -126, 0.5, 1.5, -2.5], device="cuda")
    esizes = {"fp32": 4, "int32": 4, "bf16": 2, "fp16": 2, "fp64": 8, "int64": 8}
    done = 0
    for case in range(150):
        _, algo, port = SCHEDULES[int(rng.integers(len(SCHEDULES)))]
        p = int(rng.choice([1, 2, 3, 4, 5, 8, 9, 16, 17, 33, 64, 100, 128, 257, 300]))
        dt = str(rng.choice(list(esizes)))
        esize = esizes[dt]
        words = int(rng.integers(1, 20000))                       # 4-byte words of a message
        n = words * (4 // esize) if esize <= 4 else words // 2 + 1
        seg_words = int(rng.integers(1, words + 1)) if rng.random() < 0.5 else int(rng.integers(1, 700))
        if esize == 8:
            seg_words = max(2, seg_words // 2 * 2)                # no segment may begin inside an element
        msg_bytes, op = n * esize, str(rng.choice(list(OPS)))
        seg_bytes = min(seg_words * 4, msg_bytes)
        g = torch.Generator("cuda").manual_seed(case)
        if dt in ("int32", "int64"):
            x = torch.randint(-(1 << 20), 1 << 20, (p, n), device="cuda", generator=g, dtype=torch.int32 if dt == "int32" else torch.int64)
            if op == "prod":
                x = x % 7 - 3
        else:
            x = torch.randn(p, n, device="cuda", generator=g, dtype=torch.float64 if dt == "fp64" else torch.float32)
            if op == "prod":
                x = x.abs() * 0.5 + 0.75                           # magnitudes around 1: no overflow, no inf * 0
            else:
                x = x * 10.0 ** torch.randint(-4, 5, x.shape, device="cuda", generator=g)
                if dt == "fp32" and rng.random() < 0.33:
                    pick = torch.rand(x.shape, device="cuda", generator=g) < 0.3
                    x = torch.where(pick, special[torch.randint(0, len(special), x.shape, device="cuda", generator=g)], x)
            if dt == "bf16":
                x = x.to(torch.bfloat16)
            if dt == "fp16":
                x = x.clamp(-6e4, 6e4).to(torch.float16)
        x = x.contiguous()
        out = torch.empty(n, dtype=x.dtype, device="cuda")
        try:
            h = rd.rd_schedule_create(algo, port, p, msg_bytes, seg_bytes, *M1)
        except rd.RdError:
            continue                                               # (a butterfly whose halving would cut an 8-byte element)
        try:
            rd.rd_reduce(h, x, out, OPS[op])
            torch.cuda.synchronize()
        except rd.RdError as e:
            assert e.status == rd.RD_ERR_INVALID_ARG and esize == 8, (case, e.status)
            continue
        finally:
            rd.rd_destroy(h)
        ev, off, _ = oracle_schedule(algo, port, p, msg_bytes, seg_bytes, *M1)
        off = off // 2 if esize == 8 else off * (4 // esize)       # boundaries in elements of the type
        if dt in ("bf16", "fp16"):
            want = O.reduce(ev, x.view(torch.int16).cpu().numpy().view(np.uint16), off, op, half=dt)
            got = out.view(torch.int16).cpu().numpy().view(np.uint16)
        else:
            want, got = O.reduce(ev, x.cpu().numpy(), off, op), out.cpu().numpy()
        assert got.tobytes() == want.tobytes(), (case, algo, p, dt, op, n, seg_bytes)
        done += 1
    assert done >= 130


def test_batch_equals_separate_calls_and_keeps_stream_order():
    """Independent jobs issued together: bit-identical to one rd_reduce per job; what follows the batch on
    the stream sees every result, what precedes it is seen by every job."""
    p, n = 64, 1 << 18
    specs = [(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, 16 << 10), (rd.RD_BINOMIAL, rd.RD_PORT_UNI, 16 << 10),
             (rd.RD_PIPELINE, rd.RD_PORT_UNI, 16 << 10), (rd.RD_BINARY, rd.RD_PORT_UNI, 16 << 10),
             (rd.RD_BI_GREEDY, rd.RD_PORT_BI, 64 << 10), (rd.RD_BUTTERFLY, rd.RD_PORT_BI, 0)]
    hs = [rd.rd_schedule_create(a, pt, p, 4 * n, seg, *M1) for a, pt, seg in specs]
    try:
        x = torch.empty((p, n), device="cuda")
        outs = [torch.empty(n, device="cuda") for _ in hs]
        batch = rd.Batch([(h, x, o) for h, o in zip(hs, outs)])
        for trial in range(5):
            g = torch.Generator("cuda").manual_seed(trial)
            x.normal_(generator=g)                                  # written on the stream just before the batch
            x *= 10.0 ** torch.randint(-4, 5, x.shape, device="cuda", generator=g)
            for o in outs:
                o.fill_(-1.0)
            rd.rd_reduce_batch(batch, rd.RD_SUM)
            sums = torch.stack([o.double().sum() for o in outs])    # read on the stream just after it
            ref = []
            for h in hs:
                r = torch.empty(n, device="cuda")
                rd.rd_reduce(h, x, r, rd.RD_SUM)
                ref.append(r)
            torch.cuda.synchronize()
            for o, r in zip(outs, ref):
                assert torch.equal(o, r)
            assert torch.equal(sums, torch.stack([r.double().sum() for r in ref]))
        xh = x.cpu().numpy()
        ev, off, _ = oracle_schedule(specs[0][0], specs[0][1], p, 4 * n, specs[0][2], *M1)
        assert outs[0].cpu().numpy().tobytes() == O.reduce(ev, xh, off, "sum").tobytes()
    finally:
        for h in hs:
            rd.rd_destroy(h)


def test_batch_of_unlike_jobs():
    """Jobs of different sizes and process counts, one with a ragged length (two launches), one with more
    processes than travel as kernel parameters, and one whose output is its own root input."""
    shapes = [(8, 4096, 2048), (13, 6151, 4 * 333), (300, 4096, 4096), (5, 10000, 4 * 2500), (2, 4100, 4 * 4100)]
    hs, xs, outs = [], [], []
    for k, (p, n, seg) in enumerate(shapes):
        hs.append(rd.rd_schedule_create(rd.RD_BI_GREEDY, rd.RD_PORT_BI, p, 4 * n, seg, *M1))
        xs.append(make_inputs(p, n, "int_pm2p20", seed=k, device="cuda"))
        outs.append(torch.empty(n, dtype=torch.int32, device="cuda"))
    keep = xs[0].clone()
    outs[0] = xs[0][0]                                              # aliases its own root input
    try:
        rd.rd_reduce_batch([(h, x, o) for h, x, o in zip(hs, xs, outs)], rd.RD_SUM)
        torch.cuda.synchronize()
        xs[0] = keep
        for x, o in zip(xs, outs):
            want = ((x.sum(dim=0, dtype=torch.int64) + (1 << 31)) % (1 << 32) - (1 << 31)).to(torch.int32)
            assert torch.equal(o, want)
        with pytest.raises(rd.RdError) as e:                        # job 1 would write job 0's inputs
            rd.rd_reduce_batch([(hs[1], xs[1], outs[1]), (hs[1], xs[1], xs[1][3])], rd.RD_SUM)
        assert e.value.status == rd.RD_ERR_INVALID_ARG
    finally:
        for h in hs:
            rd.rd_destroy(h)


def test_batch_as_one_launch_of_unlike_jobs():
    """Whole-vector, 16-byte aligned jobs run as ONE launch of the streaming kernel whatever their shapes:
    different process counts (one, two, more than travel as kernel parameters), lengths, segmentations with
    boundaries inside a vector, stack depths, a schedule that serves two jobs, an output that aliases its own
    root input.  Called more often than the library keeps per-call tables in flight; every call bit-identical
    to separate rd_reduce calls, integer results also to the order-free value."""
    shapes = [(8, 4096, 2048), (13, 6152, 4 * 333), (300, 4096, 4096), (5, 10000, 4 * 2500), (2, 4100, 4 * 4100),
              (1, 2048 * 3 + 4, 4 * 1000), (64, 2048 * 40, 16 << 10), (33, 2048 * 7 + 12, 4 * 999)]
    for dist, op, dt in (("int_pm2p20", rd.RD_SUM, torch.int32), ("normal", rd.RD_SUM, torch.float32), ("normal", rd.RD_MAX, torch.float32)):
        hs, xs, outs = [], [], []
        for k, (p, n, seg) in enumerate(shapes):
            algo, port = [(rd.RD_BI_GREEDY, rd.RD_PORT_BI), (rd.RD_UNI_GREEDY, rd.RD_PORT_UNI), (rd.RD_BINOMIAL, rd.RD_PORT_UNI)][k % 3]
            hs.append(rd.rd_schedule_create(algo, port, p, 4 * n, seg, *M1))
            xs.append(make_inputs(p, n, dist, seed=k, device="cuda"))
            outs.append(torch.empty(n, dtype=dt, device="cuda"))
        hs.append(hs[1]); xs.append(make_inputs(13, 6152, dist, seed=99, device="cuda")); outs.append(torch.empty(6152, dtype=dt, device="cuda"))
        keep = xs[0].clone()
        outs[0] = xs[0][0]                                          # aliases its own root input
        try:
            for h in hs:                                            # the comparison below must see this kernel, not the direct one
                rd.rd_schedule_set_tree_variant(h, rd.RD_TREE_STREAM)
                assert rd.rd_schedule_tree_shape(h)["n_tiles"] >= 1
            for call in range(7):
                xs[0].copy_(keep)
                for o in outs[1:]:
                    o.zero_()
                rd.rd_reduce_batch([(h, x, o) for h, x, o in zip(hs, xs, outs)], op)
                got = [o.clone() for o in outs]
                xs[0].copy_(keep)
                for h, x, o, g in zip(hs, xs, outs, got):
                    r = torch.empty_like(g)
                    rd.rd_reduce(h, x, r, op)
                    assert torch.equal(r.view(torch.int32), g.view(torch.int32))
                    if dt == torch.int32:
                        want = ((x.sum(dim=0, dtype=torch.int64) + (1 << 31)) % (1 << 32) - (1 << 31)).to(torch.int32)
                        assert torch.equal(g, want)
                    elif op == rd.RD_MAX:
                        assert torch.equal(g, x.amax(dim=0))
        finally:
            for h in hs[:-1]:
                rd.rd_destroy(h)


def test_batch_too_large_for_the_kernel_parameters():
    """More than 16 jobs (or 1024 input pointers): descriptors and pointers reach the device through the
    library's pinned ring, which has four slots and grows on demand: many calls in a row, then a larger batch."""
    def make(k, p, n, seg):
        hs = [rd.rd_schedule_create([rd.RD_UNI_GREEDY, rd.RD_PIPELINE, rd.RD_BINARY][j % 3], rd.RD_PORT_UNI, p, 4 * n, seg, *M1)
              for j in range(k)]
        xs = [make_inputs(p, n, "int_pm2p20", seed=100 * k + j, device="cuda") for j in range(k)]
        outs = [torch.empty(n, dtype=torch.int32, device="cuda") for _ in range(k)]
        return hs, xs, outs
    def run(hs, xs, outs, calls):
        batch = rd.Batch([(h, x, o) for h, x, o in zip(hs, xs, outs)])
        for call in range(calls):
            for o in outs:
                o.fill_(call)
            rd.rd_reduce_batch(batch, rd.RD_SUM)
            for x, o in zip(xs, outs):
                want = ((x.sum(dim=0, dtype=torch.int64) + (1 << 31)) % (1 << 32) - (1 << 31)).to(torch.int32)
                assert torch.equal(o, want)
    small = make(20, 7, 2048 * 3 + 8, 4 * 1000)          # 20 jobs
    wide = make(3, 400, 4096, 4 * 1024)                    # 1200 pointers
    big = make(40, 300, 2048 + 4, 4 * 512)                 # 12000 pointers: the ring has to grow
    try:
        run(*small, calls=9)
        run(*wide, calls=2)
        run(*big, calls=6)
        run(*small, calls=2)
        # fp32 in the order of each job's schedule
        p, n, seg = 7, 2048 * 3 + 8, 4 * 1000
        xs = [make_inputs(p, n, "normal", seed=j, device="cuda") for j in range(20)]
        outs = [torch.empty(n, device="cuda") for _ in range(20)]
        rd.rd_reduce_batch([(h, x, o) for h, x, o in zip(small[0], xs, outs)], rd.RD_SUM)
        for j in (0, 1, 2, 19):
            algo = [rd.RD_UNI_GREEDY, rd.RD_PIPELINE, rd.RD_BINARY][j % 3]
            ev, off, _ = oracle_schedule(algo, rd.RD_PORT_UNI, p, 4 * n, seg, *M1)
            assert outs[j].cpu().numpy().tobytes() == O.reduce(ev, xs[j].cpu().numpy(), off, "sum").tobytes()
    finally:
        for hs in (small[0], wide[0], big[0]):
            for h in hs:
                rd.rd_destroy(h)


def test_config2_over_two_streams_as_the_benchmark_issues_it():
    """The four schedules of config2 alternate over two CUDA streams (launches overlap each other's tail):
    every output is bit-identical to the same reduction issued alone, and sampled segments of it to the oracle."""
    w = WORKLOADS["config2"]
    model = (w["alpha"], w["beta"], w["gamma"])
    p, n = w["p"], w["n"]
    arenas = [make_inputs(p, n, w["dist"], w["seed"] + 1000 * a, device="cuda") for a in range(3)]
    tabs = [rd.PointerTable(a) for a in arenas]
    algos = [rd.RD_UNI_GREEDY, rd.RD_BINOMIAL, rd.RD_PIPELINE, rd.RD_BINARY]
    hs = [rd.rd_schedule_create(a, rd.RD_PORT_UNI, p, 4 * n, w["seg_bytes"], *model) for a in algos]
    try:
        outs = [torch.empty(n, device="cuda") for _ in hs]
        streams = [torch.cuda.Stream(), torch.cuda.Stream()]
        torch.cuda.synchronize()
        c = 0
        for step in range(6):
            for i, h in enumerate(hs):
                rd.rd_reduce(h, tabs[c % 3], outs[i], rd.RD_SUM, stream=streams[i % 2])
                c += 1
        torch.cuda.synchronize()
        # the last step read arenas (20, 21, 22, 23) mod 3
        for i, h in enumerate(hs):
            alone = torch.empty(n, device="cuda")
            rd.rd_reduce(h, tabs[(20 + i) % 3], alone, rd.RD_SUM)
            torch.cuda.synchronize()
            assert torch.equal(outs[i], alone)
            assert rd.rd_schedule_status(h) == 0
        ev = rd.rd_schedule_events(hs[0])
        off = rd.rd_schedule_segments(hs[0]).astype(np.int64)
        oev = np.zeros(len(ev), dtype=O.EVENT_DTYPE)
        for f in ("t_start", "seg", "src", "dst", "kind"):
            oev[f] = ev[f]
        for j in (0, 100, 255):
            lo, hi = int(off[j]), int(off[j + 1])
            sel = oev[oev["seg"] == j].copy()
            sel["seg"] = 0
            want = O.reduce(sel, arenas[20 % 3][:, lo:hi].cpu().numpy(), [0, hi - lo], "sum")
            assert outs[0][lo:hi].cpu().numpy().tobytes() == want.tobytes()
    finally:
        for h in hs:
            rd.rd_destroy(h)


def test_config2_as_batches_over_two_streams_as_the_benchmark_issues_it():
    """The benchmark's step: the four schedules of config2, each on its own messages, as ONE rd_reduce_batch
    call (one launch); steps alternate over two CUDA streams and two sets of messages.  Every output is
    bit-identical to the same reduction issued alone, and sampled segments of every job to the oracle run on
    the oracle's own schedule."""
    w = WORKLOADS["config2"]
    model = (w["alpha"], w["beta"], w["gamma"])
    p, n = w["p"], w["n"]
    specs = [("uni_greedy", rd.RD_UNI_GREEDY), ("binomial", rd.RD_BINOMIAL), ("pipeline", rd.RD_PIPELINE), ("binary", rd.RD_BINARY)]
    hs = [rd.rd_schedule_create(a, rd.RD_PORT_UNI, p, 4 * n, w["seg_bytes"], *model) for _, a in specs]
    try:
        arenas = [[make_inputs(p, n, w["dist"], w["seed"] + 1000 * (4 * s + j), device="cuda") for j in range(4)] for s in range(2)]
        outs = [[torch.full((n,), -3.0, device="cuda") for _ in hs] for _ in range(2)]
        batches = [rd.Batch([(h, x, o) for h, x, o in zip(hs, arenas[s], outs[s])]) for s in range(2)]
        streams = [torch.cuda.Stream(), torch.cuda.Stream()]
        torch.cuda.synchronize()
        for step in range(6):
            rd.rd_reduce_batch(batches[step % 2], rd.RD_SUM, stream=streams[step % 2])
        torch.cuda.synchronize()
        assert rd.rd_schedule_status(hs[0]) == 0
        for s in range(2):
            for j, (h, (name, algo)) in enumerate(zip(hs, specs)):
                alone = torch.empty(n, device="cuda")
                rd.rd_reduce(h, arenas[s][j], alone, rd.RD_SUM)
                torch.cuda.synchronize()
                assert torch.equal(outs[s][j].view(torch.int32), alone.view(torch.int32)), (s, name)
                ev, off, _ = oracle_schedule(algo, rd.RD_PORT_UNI, p, 4 * n, w["seg_bytes"], *model)
                for seg in (0, 77 + j, 255):
                    lo, hi = int(off[seg]), int(off[seg + 1])
                    sel = ev[ev["seg"] == seg].copy()
                    sel["seg"] = 0
                    want = O.reduce(sel, arenas[s][j][:, lo:hi].cpu().numpy(), [0, hi - lo], "sum")
                    assert outs[s][j][lo:hi].cpu().numpy().tobytes() == want.tobytes(), (s, name, seg)
    finally:
        for h in hs:
            rd.rd_destroy(h)


# ---------------------------------------------------------------------------------------------
# bf16 elements combined in fp32 (tree mode): every schedule and operation against the oracle's
# bit patterns; the oracle widens, combines in fp32 in schedule order and rounds once at the root.
# ---------------------------------------------------------------------------------------------
def bf16_inputs(p, n, kind, seed, dtype=torch.bfloat16):
    g = torch.Generator("cuda").manual_seed(seed)
    if kind == "small_int":
        return torch.randint(-3, 4, (p, n), device="cuda", generator=g).to(dtype)
    x = torch.empty((p, n), device="cuda")
    if kind == "near_one":
        x.uniform_(0.5, 2.0, generator=g)
        x *= torch.randint(0, 2, x.shape, device="cuda", generator=g) * 2.0 - 1.0
    else:
        x.normal_(generator=g)
        span = 4 if dtype == torch.bfloat16 else 2                    # fp16: sums of 300 such values stay finite
        x *= 10.0 ** torch.randint(-span, span + 1, x.shape, device="cuda", generator=g)
    return x.to(dtype)


def bits(t):
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def check_bf16(algo, port, x, seg_bytes, op, rows=None, out=None, variant=None):
    p, n = x.shape                                                   # n 16-bit elements = 2 n bytes
    h = rd.rd_schedule_create(algo, port, p, 2 * n, seg_bytes, *M1)
    try:
        if variant is not None:
            rd.rd_schedule_set_tree_variant(h, variant)
        out = torch.full((n,), 7.0, dtype=x.dtype, device="cuda") if out is None else out
        rd.rd_reduce(h, rows if rows is not None else x, out, OPS[op])
        torch.cuda.synchronize()
    finally:
        rd.rd_destroy(h)
    ev, off, _ = oracle_schedule(algo, port, p, 2 * n, seg_bytes if seg_bytes else 2 * n, *M1)
    want = O.reduce(ev, bits(x), off * 2, op, half="bf16" if x.dtype == torch.bfloat16 else "fp16")   # the schedule counts 4-byte words
    assert bits(out).tobytes() == want.tobytes()
    return out


# (p, n bf16 elements, segment in bf16 elements): tiles hold 2048 or 4096 of them; ragged tails; segments that
# begin inside a 128-bit vector (multiples of 2 elements); lengths that are not whole vectors
SHAPES_BF16 = [(8, 8192, 1024), (5, 20000, 5000), (13, 3 * 4096 + 72, 4096 + 1040), (64, 16384, 2048), (2, 8200, 8200),
               (33, 12000, 2000), (16, 256, 16), (1, 10000, 2000), (8, 6000, 666), (4, 128, 6), (32, 16384, 4098),
               (8, 8198, 2000), (5, 14, 4), (3, 6, 2), (8, 12302, 666), (128, 8192, 1024), (300, 4096, 4096)]


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16])
@pytest.mark.parametrize("name,algo,port", SCHEDULES)
@pytest.mark.parametrize("kind,op", [("normal", "sum"), ("normal", "max"), ("normal", "min"), ("near_one", "prod"), ("small_int", "sum")])
def test_bf16_parity(name, algo, port, kind, op, dtype):
    for p, n, seg in SHAPES_BF16:
        if dtype == torch.float16 and op == "prod" and p > 16:
            continue                                                 # products of many factors leave fp16's range
        x = bf16_inputs(p, n, kind, seed=p * 1000 + n, dtype=dtype)
        out = check_bf16(algo, port, x, 2 * seg, op)
        if kind == "small_int":                                      # exact for any order
            assert torch.equal(out.float(), x.float().sum(dim=0))
        elif op in ("max", "min"):
            assert torch.equal(out, x.amax(dim=0) if op == "max" else x.amin(dim=0))


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16])
@pytest.mark.parametrize("name,algo,port", SCHEDULES)
def test_bf16_parity_with_one_operand_tile_per_stage(name, algo, port, dtype):
    """The 16-bit types run two operand tiles of 2048 elements per ring stage by default (the test above); on
    request one tile of 4096 elements per stage, with stack levels twice as large.  Same bits."""
    for p, n, seg in SHAPES_BF16:
        x = bf16_inputs(p, n, "normal", seed=p * 1000 + n, dtype=dtype)
        for op in ("sum", "max"):
            check_bf16(algo, port, x, 2 * seg, op, variant=rd.RD_TREE_STREAM)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16])
def test_sixteen_bit_extrema_of_zeros_subnormals_and_infinities(dtype):
    """max and min of 16-bit elements are taken on the packed 16-bit values themselves; the oracle widens to fp32,
    compares there and rounds at the end.  Same bits, also where it is delicate: +0 against -0 (the held value
    survives a tie, so the order of the schedule decides the sign), subnormals (never flushed), infinities, and
    neighbouring values that differ in the last bit."""
    info = torch.finfo(dtype)
    tiny_sub = 2.0 ** (-133 if dtype == torch.bfloat16 else -24)                   # the smallest subnormal
    palette = torch.tensor([0.0, -0.0, tiny_sub, -tiny_sub, 3 * tiny_sub, -3 * tiny_sub, info.tiny, -info.tiny,
                            info.tiny * (1 - info.eps), 1.0, 1.0 + info.eps, -1.0, -1.0 - info.eps, info.max, -info.max,
                            float("inf"), float("-inf"), 0.5, -0.5], dtype=torch.float64).to(dtype).cuda()
    assert (palette[2].float() > 0) and (palette[2].float() < info.tiny)            # really a subnormal of the type
    g = torch.Generator("cuda").manual_seed(11)
    for p, n, seg in [(8, 8192, 1024), (13, 3 * 4096 + 72, 4096 + 1040), (64, 16384, 2048), (5, 14, 4), (200, 4096, 4096)]:
        idx = torch.randint(0, len(palette), (p, n), device="cuda", generator=g)
        idx[:, : n // 4] = torch.randint(0, 2, (p, n // 4), device="cuda", generator=g)       # a stretch of nothing but +0 and -0
        x = palette[idx]
        for name, algo, port in SCHEDULES:
            for op in ("max", "min"):
                out = check_bf16(algo, port, x, 2 * seg, op)
                assert torch.equal(out.float(), (x.float().amax(dim=0) if op == "max" else x.float().amin(dim=0)))  # as numbers
        rows = [x[i, 2:] for i in range(p)]                                        # 4 bytes off a vector: the element kernel
        if n > 16:
            check_bf16(rd.RD_BI_GREEDY, rd.RD_PORT_BI, x[:, 2:].contiguous(), 2 * 1000, "max")
            big_out = torch.zeros(n, dtype=dtype, device="cuda")
            check_bf16(rd.RD_BI_GREEDY, rd.RD_PORT_BI, x[:, 2:], 2 * 1000, "max", rows=rows, out=big_out[2:])


def test_bf16_partial_results_stay_in_fp32_and_ties_round_to_even():
    """1 + 2^-9 + 2^-9 + 2^-9 through a pipeline: 1 + 2^-7 when the partial sums are fp32 (1 if they were
    rounded to bf16 each time); 1 + 2 * 2^-9 is a tie and goes to the even neighbour 1."""
    n = 4096 * 3
    x = torch.full((4, n), 2.0 ** -9, dtype=torch.bfloat16, device="cuda")
    x[3] = 1.0
    out = check_bf16(rd.RD_PIPELINE, rd.RD_PORT_UNI, x, 2 * 4096, "sum")
    assert (out.float() == 1 + 2.0 ** -7).all()
    out = check_bf16(rd.RD_PIPELINE, rd.RD_PORT_UNI, x[1:].contiguous(), 2 * 4096, "sum")
    assert (out.float() == 1.0).all()
    # the same for fp16, whose spacing at 1 is 2^-10, and its overflow to infinity
    y = torch.full((4, n), 2.0 ** -12, dtype=torch.float16, device="cuda")
    y[3] = 1.0
    out = check_bf16(rd.RD_PIPELINE, rd.RD_PORT_UNI, y, 2 * 4096, "sum")
    assert (out.float() == 1 + 2.0 ** -10).all()
    out = check_bf16(rd.RD_PIPELINE, rd.RD_PORT_UNI, y[1:].contiguous(), 2 * 4096, "sum")
    assert (out.float() == 1.0).all()
    z = torch.full((3, n), 30000.0, dtype=torch.float16, device="cuda")
    out = check_bf16(rd.RD_BINOMIAL, rd.RD_PORT_UNI, z, 2 * 4096, "sum")
    assert torch.isinf(out.float()).all()
    out = check_bf16(rd.RD_BINOMIAL, rd.RD_PORT_UNI, z[:2].contiguous(), 2 * 4096, "sum")
    assert (out.float() == 60000.0).all()                             # 60000 is below fp16's largest value 65504


def test_bf16_buffers_off_the_vector_boundary_and_batches():
    """Buffers 4 bytes into a 128-bit vector take the element path; a batch of bf16 jobs is one launch."""
    p, n = 8, 6006
    big = bf16_inputs(p, n + 2, "normal", seed=5)
    rows = [big[i, 2:] for i in range(p)]
    assert rows[0].data_ptr() % 16 == 4
    out_big = torch.zeros(n + 2, dtype=torch.bfloat16, device="cuda")
    check_bf16(rd.RD_BI_GREEDY, rd.RD_PORT_BI, big[:, 2:], 2 * 1024, "sum", rows=rows, out=out_big[2:])
    assert out_big[0].item() == 0.0 and out_big[1].item() == 0.0
    with pytest.raises(rd.RdError) as e:                             # 2 bytes off a word: refused
        check_bf16(rd.RD_PIPELINE, rd.RD_PORT_UNI, big[:, 1:-1], 2 * 1024, "sum", rows=[big[i, 1:-1] for i in range(p)],
                   out=out_big[1:-1])
    assert e.value.status == rd.RD_ERR_INVALID_ARG
    shapes = [(8, 8192, 1024), (13, 12304, 2 * 333), (64, 4096 * 5, 4096), (2, 8200, 8200)]
    hs = [rd.rd_schedule_create(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, p, 2 * n, 2 * seg, *M1) for p, n, seg in shapes]
    try:
        xs = [bf16_inputs(p, n, "normal", seed=k) for k, (p, n, seg) in enumerate(shapes)]
        outs = [torch.empty(n, dtype=torch.bfloat16, device="cuda") for p, n, seg in shapes]
        rd.rd_reduce_batch([(h, x, o) for h, x, o in zip(hs, xs, outs)], rd.RD_SUM)
        torch.cuda.synchronize()
        for (p, n, seg), x, o in zip(shapes, xs, outs):
            ev, off, _ = oracle_schedule(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, p, 2 * n, 2 * seg, *M1)
            assert bits(o).tobytes() == O.reduce(ev, bits(x), off * 2, "sum").tobytes()
        with pytest.raises(rd.RdError) as e:                         # no schedule-faithful execution for bf16
            rd.rd_reduce(hs[0], xs[0], outs[0], rd.RD_SUM, exec_mode=rd.RD_EXEC_FAITHFUL)
        assert e.value.status == rd.RD_ERR_UNSUPPORTED
    finally:
        for h in hs:
            rd.rd_destroy(h)


def test_tiles_on_demand_over_many_launches_and_streams():
    """The streaming kernel's thread blocks take their tiles from a counter that the launch's last block puts
    back to zero.  Hundreds of launches of unlike shapes (different numbers of thread blocks and tiles per
    block, single reductions and batches), alternating over three streams, must all give the bits of a launch
    issued alone, and no launch may report a wait that gave up."""
    shapes = [(5, 2048 * 37 + 8, 4 * 3000), (64, 2048 * 300, 16 << 10), (9, 2048 * 1500 + 36, 4 * (2048 + 520)), (3, 2048 * 2, 4096)]
    hs, xs, refs = [], [], []
    for k, (p, n, seg) in enumerate(shapes):
        algo, port = SCHEDULES[k % 4][1:]
        hs.append(rd.rd_schedule_create(algo, port, p, 4 * n, seg, *M1))
        xs.append(make_inputs(p, n, "normal", seed=50 + k, device="cuda"))
        r = torch.empty(n, device="cuda")
        rd.rd_reduce(hs[-1], xs[-1], r, rd.RD_SUM)
        refs.append(r)
    torch.cuda.synchronize()
    try:
        streams = [torch.cuda.Stream() for _ in range(3)]
        outs = [[torch.zeros_like(r) for r in refs] for _ in streams]
        batch = [rd.Batch([(hs[0], xs[0], o[0]), (hs[3], xs[3], o[3])]) for o in outs]
        for it in range(120):
            si = it % 3
            with torch.cuda.stream(streams[si]):
                for o in outs[si]:
                    o.zero_()
                rd.rd_reduce(hs[1], xs[1], outs[si][1], rd.RD_SUM, stream=streams[si])
                rd.rd_reduce_batch(batch[si], rd.RD_SUM, stream=streams[si])
                rd.rd_reduce(hs[2], xs[2], outs[si][2], rd.RD_SUM, stream=streams[si])
            if it % 30 == 29:
                torch.cuda.synchronize()
                for o in outs:
                    for got, want in zip(o, refs):
                        assert torch.equal(got.view(torch.int32), want.view(torch.int32))
        for h in hs:
            assert rd.rd_schedule_status(h) == 0
    finally:
        for h in hs:
            rd.rd_destroy(h)
