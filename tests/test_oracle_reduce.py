"""Pins of the oracle's reduction evaluator (O2): special cases with a plain definition."""
import numpy as np
import pytest

from oracle import rd_oracle as O

f32 = np.float32


def schedules(p, sizes, A=3, B=1, G=1):
    """Every tree schedule for (p, sizes) as (name, events)."""
    out = [("uni", O.uni_greedy(p, sizes, A, B, G)[0]),
           ("pipe", O.pipeline(p, sizes, A, B, G, False)[0]),
           ("binary", O.binary(p, sizes, A, B, G, True)[0]),
           ("binomial", O.binomial(p, sizes, A, B, G)[0])]
    if p >= 2:
        out.append(("bi", O.bi_greedy(p, sizes, A, B, G)[0]))
    return out


def seg_off(sizes):
    return np.concatenate([[0], np.cumsum(sizes)])


@pytest.mark.parametrize("p", [2, 3, 8, 13, 64])
def test_integer_results_do_not_depend_on_the_order(p):
    rng = np.random.default_rng(p)
    sizes = [5, 5, 5, 2]
    n = sum(sizes)
    x = rng.integers(-2**31, 2**31, size=(p, n), dtype=np.int64).astype(np.int32)   # wraps on purpose
    want_sum = (x.astype(np.int64).sum(axis=0) & 0xFFFFFFFF).astype(np.uint32).view(np.int32)
    want_max = x.max(axis=0)
    for name, ev in schedules(p, sizes):
        assert (O.reduce(ev, x, seg_off(sizes), "sum") == want_sum).all(), name
        assert (O.reduce(ev, x, seg_off(sizes), "max") == want_max).all(), name
    ev, off, _ = O.butterfly(p, n, 4, 3, 1, 1)
    assert (O.reduce(ev, x, off, "sum") == want_sum).all()
    assert (O.reduce(ev, x, off, "max") == want_max).all()


@pytest.mark.parametrize("p", [2, 3, 8, 13, 64])
def test_integer_min_and_wrapping_product_do_not_depend_on_the_order(p):
    """min is the plain minimum; the product is the product of the residues modulo 2^32."""
    rng = np.random.default_rng(50 + p)
    sizes = [5, 5, 5, 2]
    n = sum(sizes)
    x = rng.integers(-2**31, 2**31, size=(p, n), dtype=np.int64).astype(np.int32)
    x[:, :6] = rng.integers(-3, 4, size=(p, 6)) * 2 + 1            # small odd factors: the product stays non-zero
    want_prod = np.array([int(np.prod([int(v) for v in x[:, e]], dtype=object)) & 0xFFFFFFFF for e in range(n)],
                         dtype=np.uint64).astype(np.uint32).view(np.int32)
    assert (want_prod[:6] != 0).all()
    for name, ev in schedules(p, sizes):
        assert (O.reduce(ev, x, seg_off(sizes), "min") == x.min(axis=0)).all(), name
        assert (O.reduce(ev, x, seg_off(sizes), "prod") == want_prod).all(), name
    ev, off, _ = O.butterfly(p, n, 4, 3, 1, 1)
    assert (O.reduce(ev, x, off, "min") == x.min(axis=0)).all()
    assert (O.reduce(ev, x, off, "prod") == want_prod).all()


@pytest.mark.parametrize("p", [2, 5, 16, 33])
def test_fp32_min_is_the_minimum_and_powers_of_two_multiply_exactly(p):
    rng = np.random.default_rng(150 + p)
    sizes = [7, 7, 3]
    x = rng.standard_normal((p, 17)).astype(f32)
    e = rng.integers(-3, 4, size=(p, 17))
    pw = (np.ldexp(1.0, e) * rng.choice([-1.0, 1.0], size=(p, 17))).astype(f32)      # products are exact in any order
    want = np.ldexp(1.0, e.sum(axis=0)) * np.prod(np.sign(pw), axis=0)
    for name, ev in schedules(p, sizes):
        assert (O.reduce(ev, x, seg_off(sizes), "min") == x.min(axis=0)).all(), name
        assert (O.reduce(ev, pw, seg_off(sizes), "prod") == want.astype(f32)).all(), name


def test_fp32_product_two_processes_is_one_multiply_and_min_keeps_the_held_zero():
    rng = np.random.default_rng(8)
    x = (rng.standard_normal((2, 1000)) * 10.0 ** rng.integers(-8, 8, size=(2, 1000))).astype(f32)
    ev, _ = O.uni_greedy(2, [600, 400], 1, 1, 1)
    assert (O.reduce(ev, x, [0, 600, 1000], "prod") == x[0] * x[1]).all()
    z = np.array([[0.0], [-0.0]], dtype=f32)                          # incoming -0 is not less than held +0
    ev, _ = O.uni_greedy(2, [1], 1, 1, 1)
    assert np.signbit(O.reduce(ev, z, [0, 1], "min"))[0] == False
    assert np.signbit(O.reduce(ev, z[::-1].copy(), [0, 1], "min"))[0] == True


def test_fp32_product_pipeline_is_a_running_product_from_the_far_end():
    p = 9
    rng = np.random.default_rng(p)
    x = rng.uniform(0.5, 2.0, size=(p, 64)).astype(f32)
    want = x[p - 1].copy()
    for k in range(p - 2, -1, -1):
        want = (x[k] * want).astype(f32)
    ev, _ = O.pipeline(p, [32, 32], 3, 1, 1, False)
    assert O.reduce(ev, x, [0, 32, 64], "prod").tobytes() == want.tobytes()


@pytest.mark.parametrize("p", [2, 5, 16, 33])
def test_fp32_max_is_the_maximum(p):
    rng = np.random.default_rng(100 + p)
    sizes = [7, 7, 3]
    x = rng.standard_normal((p, 17)).astype(f32)
    for name, ev in schedules(p, sizes):
        assert (O.reduce(ev, x, seg_off(sizes), "max") == x.max(axis=0)).all(), name


def test_fp32_max_keeps_the_held_value_on_ties():
    """incoming > held ? incoming : held -- with +0 and -0 the held one survives."""
    x = np.array([[0.0], [-0.0]], dtype=f32)           # root holds +0, receives -0
    ev, _ = O.uni_greedy(2, [1], 1, 1, 1)
    assert np.signbit(O.reduce(ev, x, [0, 1], "max"))[0] == False
    x = np.array([[-0.0], [0.0]], dtype=f32)           # root holds -0, receives +0: not greater
    assert np.signbit(O.reduce(ev, x, [0, 1], "max"))[0] == True


def test_fp32_sum_two_processes_is_one_add():
    rng = np.random.default_rng(7)
    x = (rng.standard_normal((2, 1000)) * 10.0 ** rng.integers(-8, 8, size=(2, 1000))).astype(f32)
    ev, _ = O.uni_greedy(2, [600, 400], 1, 1, 1)
    assert (O.reduce(ev, x, [0, 600, 1000], "sum") == x[0] + x[1]).all()


@pytest.mark.parametrize("p", [3, 4, 9, 32])
def test_fp32_sum_pipeline_is_a_running_sum_from_the_far_end(p):
    """Process k combines what it holds with what k+1 sends: x_0 + (x_1 + (... + x_{p-1}))."""
    rng = np.random.default_rng(p)
    x = (rng.standard_normal((p, 64)) * 10.0 ** rng.integers(-4, 5, size=(p, 64))).astype(f32)
    want = x[p - 1].copy()
    for k in range(p - 2, -1, -1):
        want = (x[k] + want).astype(f32)
    for bidir in (False, True):
        ev, _ = O.pipeline(p, [16] * 4, 2, 1, 1, bidir)
        assert (O.reduce(ev, x, [0, 16, 32, 48, 64], "sum") == want).all()


def test_fp32_sum_binomial_and_binary_association():
    """Association order matters in fp32.  p = 4, each tree written out from its definition:
    binomial  round 0: 1->0, 3->2; round 1: 2->0         =>  (x0 + x1) + (x2 + x3)
    pipeline  3->2->1->0                                  =>  x0 + (x1 + (x2 + x3))
    binary    heap order, left child first: 3->1, 1->0, 2->0  =>  (x0 + (x1 + x3)) + x2
    and on inputs with a wide exponent range the three differ from each other."""
    rng = np.random.default_rng(11)
    n = 256
    x = (rng.standard_normal((4, n)) * 10.0 ** rng.integers(-6, 7, size=(4, n))).astype(f32)
    x0, x1, x2, x3 = x
    forms = {
        "binomial": ((x0 + x1).astype(f32) + (x2 + x3).astype(f32)).astype(f32),
        "pipeline": (x0 + (x1 + (x2 + x3).astype(f32)).astype(f32)).astype(f32),
        "binary": ((x0 + (x1 + x3).astype(f32)).astype(f32) + x2).astype(f32),
    }
    got = {
        "binomial": O.reduce(O.binomial(4, [n], 1, 1, 1)[0], x, [0, n], "sum"),
        "pipeline": O.reduce(O.pipeline(4, [n], 1, 1, 1, False)[0], x, [0, n], "sum"),
        "binary": O.reduce(O.binary(4, [n], 1, 1, 1, False)[0], x, [0, n], "sum"),
    }
    for a in forms:
        assert (got[a] == forms[a]).all(), a
        for b in forms:
            if a != b:
                assert (got[a] != forms[b]).any(), (a, b)
    # a hand-checkable instance: 2^24 + 1 + 1 + 1
    big, one = f32(2.0 ** 24), f32(1.0)
    y = np.array([[big], [one], [one], [one]], dtype=f32)
    assert O.reduce(O.binomial(4, [1], 1, 1, 1)[0], y, [0, 1], "sum")[0] == f32(2.0 ** 24 + 2)   # (2^24+1 -> 2^24) + 2
    assert O.reduce(O.pipeline(4, [1], 1, 1, 1, False)[0], y, [0, 1], "sum")[0] == f32(2.0 ** 24 + 4)  # 2^24 + 3 -> even


def test_fp32_sum_butterfly_association():
    """p = 4: chunk c is reduced by V(c) = (x_c + x_{c^2}) + (x_{c^1} + x_{c^3})."""
    rng = np.random.default_rng(3)
    n = 8
    x = (rng.standard_normal((4, n)) * 10.0 ** rng.integers(-6, 7, size=(4, n))).astype(f32)
    ev, off, _ = O.butterfly(4, n, 4, 1, 1, 1)
    got = O.reduce(ev, x, off, "sum")
    assert list(off) == [0, 2, 4, 6, 8]
    for c in range(4):
        sl = slice(off[c], off[c + 1])
        want = (x[c, sl] + x[c ^ 2, sl]).astype(f32) + (x[c ^ 1, sl] + x[c ^ 3, sl]).astype(f32)
        assert (got[sl] == want.astype(f32)).all()


@pytest.mark.parametrize("p,dist", [(8, "normal"), (64, "normal"), (256, "uniform")])
def test_fp32_sum_is_close_to_fp64(p, dist):
    """Any association of p fp32 numbers is within (p-1) * 2^-24 * sum|x_i| of the exact sum."""
    rng = np.random.default_rng(p)
    sizes = [100, 100, 56]
    n = 256
    x = (rng.standard_normal((p, n)) if dist == "normal" else rng.uniform(-1, 1, (p, n))).astype(f32)
    ref, mag = O.reference_f64(x, "sum")
    assert np.allclose(ref, x.astype(np.float64).sum(axis=0), rtol=1e-13, atol=1e-13)
    assert np.allclose(mag, np.abs(x.astype(np.float64)).sum(axis=0), rtol=1e-13)
    for name, ev in schedules(p, sizes):
        got = O.reduce(ev, x, seg_off(sizes), "sum").astype(np.float64)
        assert (np.abs(got - ref) <= (p - 1) * 2.0 ** -24 * mag).all(), name
        assert (np.abs(got - ref) <= 1e-5 * mag).all(), name


def test_segments_use_their_own_trees():
    """Uni-greedy builds a different tree per segment: replaying segment j's events on segment k's data
    must in general change fp32 bits, while each segment alone matches a replay restricted to it."""
    p, sizes = 16, [8, 8, 8, 8]
    rng = np.random.default_rng(0)
    x = (rng.standard_normal((p, 32)) * 10.0 ** rng.integers(-3, 4, size=(p, 32))).astype(f32)
    ev, _ = O.uni_greedy(p, sizes, 2, 0, 1)
    full = O.reduce(ev, x, seg_off(sizes), "sum")
    for j in range(4):
        only = ev[ev["seg"] == j].copy()
        only["seg"] = 0
        part = O.reduce(only, x[:, 8 * j:8 * j + 8].copy(), [0, 8], "sum")
        assert (part == full[8 * j:8 * j + 8]).all()


def test_empty_segments_and_single_process():
    x = np.arange(12, dtype=np.int32).reshape(1, 12)
    ev, _ = O.uni_greedy(1, [4, 8], 1, 1, 1)
    assert len(ev) == 0
    assert (O.reduce(ev, x, [0, 4, 12], "sum") == x[0]).all()
    x = np.ones((4, 3), dtype=np.int32)
    ev, off, _ = O.butterfly(4, 3, 4, 1, 1, 1)          # fewer elements than processes: empty chunks
    assert (O.reduce(ev, x, off, "sum") == 4).all()


# ---- 8-byte element types ---------------------------------------------------------------------------------

@pytest.mark.parametrize("p", [2, 3, 8, 13, 64])
def test_int64_results_do_not_depend_on_the_order(p):
    """Sum and product modulo 2^64 (computed here with Python integers), max and min exactly."""
    rng = np.random.default_rng(300 + p)
    sizes = [5, 5, 5, 2]
    n = sum(sizes)
    x = rng.integers(-2**63, 2**63, size=(p, n), dtype=np.int64)
    x[:, :6] = rng.integers(-3, 4, size=(p, 6)) * 2 + 1
    cols = [[int(v) for v in x[:, e]] for e in range(n)]
    wrap = lambda v: np.array([c & 0xFFFFFFFFFFFFFFFF for c in v], dtype=np.uint64).view(np.int64)
    want_sum = wrap([sum(c) for c in cols])
    want_prod = wrap([int(np.prod(np.array(c, dtype=object))) for c in cols])
    assert (want_prod[:6] != 0).all()
    for name, ev in schedules(p, sizes):
        assert (O.reduce(ev, x, seg_off(sizes), "sum") == want_sum).all(), name
        assert (O.reduce(ev, x, seg_off(sizes), "prod") == want_prod).all(), name
        assert (O.reduce(ev, x, seg_off(sizes), "max") == x.max(axis=0)).all(), name
        assert (O.reduce(ev, x, seg_off(sizes), "min") == x.min(axis=0)).all(), name
    ev, off, _ = O.butterfly(p, n, 8, 3, 1, 1)
    assert (O.reduce(ev, x, off, "sum") == want_sum).all()


def test_fp64_two_processes_is_one_operation_and_the_pipeline_a_running_sum():
    rng = np.random.default_rng(9)
    x = rng.standard_normal((2, 1000)) * 10.0 ** rng.integers(-30, 30, size=(2, 1000))
    ev, _ = O.uni_greedy(2, [600, 400], 1, 1, 1)
    assert (O.reduce(ev, x, [0, 600, 1000], "sum") == x[0] + x[1]).all()
    assert (O.reduce(ev, x, [0, 600, 1000], "prod") == x[0] * x[1]).all()
    p = 9
    x = rng.standard_normal((p, 64)) * 10.0 ** rng.integers(-8, 9, size=(p, 64))
    want = x[p - 1].copy()
    for k in range(p - 2, -1, -1):
        want = x[k] + want
    ev, _ = O.pipeline(p, [32, 32], 3, 1, 1, False)
    assert O.reduce(ev, x, [0, 32, 64], "sum").tobytes() == want.tobytes()


@pytest.mark.parametrize("p", [2, 5, 16, 33])
def test_fp64_extrema_and_exact_sums(p):
    """Integers below 2^40 add exactly in fp64 whatever the order; the same values do not in fp32, so a
    reduction that went through fp32 anywhere would fail here."""
    rng = np.random.default_rng(400 + p)
    sizes = [7, 7, 3]
    x = rng.standard_normal((p, 17))
    k = rng.integers(-2**40, 2**40, size=(p, 17)).astype(np.float64)
    for name, ev in schedules(p, sizes):
        assert (O.reduce(ev, x, seg_off(sizes), "max") == x.max(axis=0)).all(), name
        assert (O.reduce(ev, x, seg_off(sizes), "min") == x.min(axis=0)).all(), name
        assert (O.reduce(ev, k, seg_off(sizes), "sum") == k.sum(axis=0)).all(), name
    z = np.array([[0.0], [-0.0]])
    ev, _ = O.uni_greedy(2, [1], 1, 1, 1)
    assert np.signbit(O.reduce(ev, z, [0, 1], "max"))[0] == False
    assert np.signbit(O.reduce(ev, z[::-1].copy(), [0, 1], "max"))[0] == True


# ---------------------------------------------------------------------------------------------
# bf16 elements combined in fp32: inputs widened exactly, fp32 partial results in the schedule's
# order, one rounding to bf16 (nearest, ties to even) of what the root holds at the end.
# The pins use torch's CPU conversion as the independent statement of "round an fp32 to bf16".
# ---------------------------------------------------------------------------------------------
def bf16_bits(a):
    """fp32 array -> uint16 bf16 bit patterns, rounded by torch (library routine, not the oracle's)."""
    import torch
    return torch.from_numpy(np.ascontiguousarray(a, dtype=f32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def bf16_value(bits):
    return (bits.astype(np.uint32) << 16).view(f32)


def test_bf16_two_processes_is_one_fp32_add_rounded_once():
    rng = np.random.default_rng(11)
    x = bf16_bits(rng.standard_normal((2, 4000)) * 10.0 ** rng.integers(-6, 7, size=(2, 4000)))
    ev, _ = O.uni_greedy(2, [2400, 1600], 1, 1, 1)
    got = O.reduce(ev, x, [0, 2400, 4000], "sum")
    assert got.dtype == np.uint16
    assert (got == bf16_bits(bf16_value(x[0]) + bf16_value(x[1]))).all()
    prod = O.reduce(ev, x, [0, 2400, 4000], "prod")
    assert (prod == bf16_bits(bf16_value(x[0]) * bf16_value(x[1]))).all()


def test_bf16_rounding_ties_go_to_the_even_neighbour_and_the_rest_to_the_nearest():
    """1 + k * 2^-9 for k = 0..8 around the bf16 neighbours 1, 1 + 2^-7, 1 + 2^-6 (spacing 2^-7): a single
    process pair adds 1 and k * 2^-9 exactly in fp32."""
    ks = np.arange(0, 9)
    x = np.stack([bf16_bits(np.ones(9)), bf16_bits(ks * 2.0 ** -9)])
    ev, _ = O.uni_greedy(2, [9], 1, 1, 1)
    got = bf16_value(O.reduce(ev, x, [0, 9], "sum"))
    # k: 0 1 -> 1; 2 is the tie between 1 (even mantissa) and 1 + 2^-7 -> 1; 3 4 5 -> 1 + 2^-7;
    # 6 is the tie between 1 + 2^-7 (odd) and 1 + 2^-6 (even) -> 1 + 2^-6; 7 8 -> 1 + 2^-6
    want = 1 + np.array([0, 0, 0, 1, 1, 1, 2, 2, 2]) * 2.0 ** -7
    assert (got == want.astype(f32)).all()


def test_bf16_partial_results_stay_in_fp32():
    """Pipeline of 4: 1 + 2^-9 + 2^-9 + 2^-9.  Kept in fp32 the sum is 1 + 3 * 2^-9, above the half-way point,
    and rounds to 1 + 2^-7; rounding every partial result to bf16 would give 1."""
    x = np.stack([bf16_bits(np.full(8, v)) for v in (2.0 ** -9, 2.0 ** -9, 2.0 ** -9, 1.0)])
    ev, _ = O.pipeline(4, [8], 1, 1, 1, False)
    got = bf16_value(O.reduce(ev, x, [0, 8], "sum"))
    assert (got == f32(1 + 2.0 ** -7)).all()


@pytest.mark.parametrize("p", [2, 5, 16, 64])
def test_bf16_small_integers_sum_exactly_and_extrema_are_order_free(p):
    """Integers up to 256 in magnitude are bf16 values, so sums that stay there are exact for any order; max and
    min pick one of the inputs, which is a bf16 value already."""
    rng = np.random.default_rng(p)
    n, sizes = 96, [40, 40, 16]
    xi = rng.integers(-3, 4, size=(p, n))
    x = bf16_bits(xi.astype(f32))
    y = bf16_bits(rng.standard_normal((p, n)) * 10.0 ** rng.integers(-5, 6, size=(p, n)))
    for name, ev in schedules(p, sizes):
        assert (bf16_value(O.reduce(ev, x, seg_off(sizes), "sum")) == xi.sum(axis=0)).all(), name
        assert (bf16_value(O.reduce(ev, y, seg_off(sizes), "max")) == bf16_value(y).max(axis=0)).all(), name
        assert (bf16_value(O.reduce(ev, y, seg_off(sizes), "min")) == bf16_value(y).min(axis=0)).all(), name


@pytest.mark.parametrize("p", [3, 9, 32])
def test_bf16_sum_is_the_fp32_schedule_sum_rounded(p):
    """The same events on the widened inputs through the fp32 evaluator (pinned above), then one rounding."""
    rng = np.random.default_rng(100 + p)
    n, sizes = 200, [64, 64, 72]
    x = bf16_bits(rng.standard_normal((p, n)) * 10.0 ** rng.integers(-3, 4, size=(p, n)))
    for name, ev in schedules(p, sizes):
        wide = O.reduce(ev, bf16_value(x), seg_off(sizes), "sum")
        assert (O.reduce(ev, x, seg_off(sizes), "sum") == bf16_bits(wide)).all(), name
        # and close to the order-free fp64 sum: one bf16 rounding (8 significant bits: 2^-8 relative) on top of the fp32 bound
        ref = bf16_value(x).astype(np.float64).sum(axis=0)
        mag = np.abs(bf16_value(x).astype(np.float64)).sum(axis=0)
        got = bf16_value(O.reduce(ev, x, seg_off(sizes), "sum")).astype(np.float64)
        assert (np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref) + p * 2.0 ** -23 * mag + 1e-30).all(), name


# fp16 (IEEE binary16) elements, combined in fp32 like bf16.
def f16_bits(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a, dtype=f32)).to(torch.float16).view(torch.int16).numpy().view(np.uint16)


def f16_value(bits):
    return bits.view(np.float16).astype(f32)


def test_fp16_two_processes_is_one_fp32_operation_rounded_once():
    rng = np.random.default_rng(12)
    x = f16_bits(rng.standard_normal((2, 4000)) * 10.0 ** rng.integers(-3, 3, size=(2, 4000)))
    ev, _ = O.uni_greedy(2, [2400, 1600], 1, 1, 1)
    got = O.reduce(ev, x, [0, 2400, 4000], "sum", half="fp16")
    assert (got == f16_bits(f16_value(x[0]) + f16_value(x[1]))).all()
    prod = O.reduce(ev, x, [0, 2400, 4000], "prod", half="fp16")
    assert (prod == f16_bits(f16_value(x[0]) * f16_value(x[1]))).all()
    # overflow goes to infinity, tiny products to subnormals and zero: whatever torch's conversion says
    y = f16_bits(np.array([[60000.0, 6e-5, 6e-8, -60000.0], [60000.0, 6e-5, 0.5, 2.0]]))
    ev, _ = O.uni_greedy(2, [4], 1, 1, 1)
    assert (O.reduce(ev, y, [0, 4], "sum", half="fp16") == f16_bits(f16_value(y[0]) + f16_value(y[1]))).all()
    assert (O.reduce(ev, y, [0, 4], "prod", half="fp16") == f16_bits(f16_value(y[0]) * f16_value(y[1]))).all()


def test_fp16_ties_to_even_and_fp32_partial_results():
    """Spacing of fp16 at 1 is 2^-10: 1 + k * 2^-12 for k = 0..8; and 1 + 3 * 2^-12 through a pipeline of four."""
    ks = np.arange(0, 9)
    x = np.stack([f16_bits(np.ones(9)), f16_bits(ks * 2.0 ** -12)])
    ev, _ = O.uni_greedy(2, [9], 1, 1, 1)
    got = f16_value(O.reduce(ev, x, [0, 9], "sum", half="fp16"))
    want = 1 + np.array([0, 0, 0, 1, 1, 1, 2, 2, 2]) * 2.0 ** -10
    assert (got == want.astype(f32)).all()
    x = np.stack([f16_bits(np.full(8, v)) for v in (2.0 ** -12, 2.0 ** -12, 2.0 ** -12, 1.0)])
    ev, _ = O.pipeline(4, [8], 1, 1, 1, False)
    assert (f16_value(O.reduce(ev, x, [0, 8], "sum", half="fp16")) == f32(1 + 2.0 ** -10)).all()


@pytest.mark.parametrize("p", [2, 5, 16, 64])
def test_fp16_small_integers_sum_exactly_and_extrema_are_order_free(p):
    rng = np.random.default_rng(p)
    n, sizes = 96, [40, 40, 16]
    xi = rng.integers(-3, 4, size=(p, n))
    x = f16_bits(xi.astype(f32))
    y = f16_bits(rng.standard_normal((p, n)) * 10.0 ** rng.integers(-3, 4, size=(p, n)))
    for name, ev in schedules(p, sizes):
        assert (f16_value(O.reduce(ev, x, seg_off(sizes), "sum", half="fp16")) == xi.sum(axis=0)).all(), name
        assert (f16_value(O.reduce(ev, y, seg_off(sizes), "max", half="fp16")) == f16_value(y).max(axis=0)).all(), name
        assert (f16_value(O.reduce(ev, y, seg_off(sizes), "min", half="fp16")) == f16_value(y).min(axis=0)).all(), name
        wide = O.reduce(ev, f16_value(y), seg_off(sizes), "sum")
        assert (O.reduce(ev, y, seg_off(sizes), "sum", half="fp16") == f16_bits(wide)).all(), name


def test_openmp_build_gives_the_bits_of_the_plain_build():
    """The second build of the oracle (-fopenmp, timed by the benchmark on all cores) splits every segment's
    elements over the threads; nothing else changes, so the results are identical bit for bit."""
    rng = np.random.default_rng(7)
    p, sizes = 13, [1000, 1000, 1000, 37]
    n = sum(sizes)
    assert O.threads(openmp=False) == 1 and O.threads(openmp=True) >= 1
    xf = (rng.standard_normal((p, n)) * 10.0 ** rng.integers(-4, 5, size=(p, n))).astype(np.float32)
    xi = rng.integers(-2**31, 2**31, size=(p, n), dtype=np.int64).astype(np.int32)
    for name, ev in schedules(p, sizes):
        for op in ("sum", "max", "min", "prod"):
            for x in (xf, xi):
                a = O.reduce(ev, x, seg_off(sizes), op)
                b = O.reduce(ev, x, seg_off(sizes), op, openmp=True)
                assert a.tobytes() == b.tobytes(), (name, op, x.dtype)
    ev, off, _ = O.butterfly(p, n, 4, 3, 1, 1)
    assert O.reduce(ev, xf, off, "sum").tobytes() == O.reduce(ev, xf, off, "sum", openmp=True).tobytes()
