"""ctypes access to the CPU oracle (rd_oracle.c).  TEST INFRASTRUCTURE ONLY.

Nothing of the product imports this module: it exists for the tests, the smoke
check and the benchmark's CPU-baseline leg.  It holds no arithmetic of its own;
every function marshals numpy arrays into the C oracle and back.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rd_oracle.c")
_LIB = os.path.join(_HERE, "librd_oracle.so")
_LIB_OMP = os.path.join(_HERE, "librd_oracle_omp.so")       # the same source built with -fopenmp (benchmark only)
CFLAGS = ["-O2", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC"]

EVENT_DTYPE = np.dtype(
    [("seg", "<i4"), ("src", "<i4"), ("dst", "<i4"), ("kind", "<i4"), ("t_start", "<i8")], align=True
)
assert EVENT_DTYPE.itemsize == 24


def build(force: bool = False, openmp: bool = False) -> str:
    """Compile rd_oracle.c with gcc when the shared object is missing or stale.  openmp: the second build,
    in which the threads of an OpenMP team share the elements of the int32 and fp32 evaluators."""
    path = _LIB_OMP if openmp else _LIB
    if force or not os.path.exists(path) or os.path.getmtime(path) < os.path.getmtime(_SRC):
        tmp = path + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", *CFLAGS, *(["-fopenmp"] if openmp else []), "-o", tmp, _SRC])
        os.replace(tmp, path)
    return path


_lib = None
_lib_omp = None


def lib(openmp: bool = False):
    global _lib, _lib_omp
    if openmp:
        if _lib_omp is None:
            _lib_omp = C.CDLL(build(openmp=True))
        return _lib_omp
    if _lib is None:
        _lib = C.CDLL(build())
    return _lib


def threads(openmp: bool = False) -> int:
    """Threads the evaluators of the chosen build run on."""
    return int(lib(openmp).orc_threads())


def _i64(a):
    return np.ascontiguousarray(a, dtype=np.int64)


def _p(a, t):
    return a.ctypes.data_as(C.POINTER(t))


def _check(rc, what):
    if rc != 0:
        raise RuntimeError("oracle %s failed with code %d" % (what, rc))


def ceil_log2(v: int) -> int:
    return int(lib().orc_ceil_log2(C.c_int64(int(v))))


def uni_greedy(p, sizes, A, B, G, want_events=True):
    """Algorithm 1.  Returns (events or None, completion ticks)."""
    sizes = _i64(sizes)
    q = len(sizes)
    ev = np.zeros((p - 1) * q, dtype=EVENT_DTYPE) if want_events else None
    comp = C.c_int64(0)
    rc = lib().orc_uni_greedy(C.c_int(p), C.c_int(q), _p(sizes, C.c_int64), C.c_int64(A), C.c_int64(B),
                              C.c_int64(G), C.c_void_p(ev.ctypes.data) if want_events else None, C.byref(comp))
    _check(rc, "uni_greedy")
    return ev, comp.value


def bi_greedy(p, sizes, A, B, G, unit_step=False, want_events=True):
    """Algorithm 2.  Returns (events or None, completion ticks)."""
    sizes = _i64(sizes)
    q = len(sizes)
    ev = np.zeros((p - 1) * q, dtype=EVENT_DTYPE) if want_events else None
    comp = C.c_int64(0)
    rc = lib().orc_bi_greedy(C.c_int(p), C.c_int(q), _p(sizes, C.c_int64), C.c_int64(A), C.c_int64(B),
                             C.c_int64(G), C.c_int(1 if unit_step else 0),
                             C.c_void_p(ev.ctypes.data) if want_events else None, C.byref(comp))
    _check(rc, "bi_greedy")
    return ev, comp.value


def _tree(fn, p, sizes, A, B, G, *extra):
    sizes = _i64(sizes)
    q = len(sizes)
    ev = np.zeros(max((p - 1) * q, 1), dtype=EVENT_DTYPE)
    comp = C.c_int64(0)
    rc = fn(C.c_int(p), C.c_int(q), _p(sizes, C.c_int64), C.c_int64(A), C.c_int64(B), C.c_int64(G),
            *extra, C.c_void_p(ev.ctypes.data), C.byref(comp))
    _check(rc, "tree schedule")
    return ev[: (p - 1) * q], comp.value


def binomial(p, sizes, A, B, G):
    return _tree(lib().orc_binomial, p, sizes, A, B, G)


def pipeline(p, sizes, A, B, G, bidir):
    return _tree(lib().orc_pipeline, p, sizes, A, B, G, C.c_int(1 if bidir else 0))


def binary(p, sizes, A, B, G, bidir):
    return _tree(lib().orc_binary, p, sizes, A, B, G, C.c_int(1 if bidir else 0))


def butterfly(p, n, esize, A, B, G):
    """Reduce-scatter/gather.  Returns (events, chunk_off[P+1] in elements, completion); P = the largest
    power of two not above p (the other p - P processes are folded in first)."""
    P = 1
    while 2 * P <= p:
        P *= 2
    L = ceil_log2(P)
    count = P * (P - 1) + (P // 2) * L + (p - P) * P
    ev = np.zeros(max(count, 1), dtype=EVENT_DTYPE)
    off = np.zeros(P + 1, dtype=np.int64)
    comp = C.c_int64(0)
    rc = lib().orc_butterfly(C.c_int(p), C.c_int64(n), C.c_int64(esize), C.c_int64(A), C.c_int64(B),
                             C.c_int64(G), C.c_void_p(ev.ctypes.data), _p(off, C.c_int64), C.byref(comp))
    _check(rc, "butterfly")
    return ev[:count], off, comp.value


def validate(events, p, sizes, A, B, G, bidir, tree_rules=True, in_order=False):
    """Returns (rule broken or 0, end of the last activity)."""
    sizes = _i64(sizes)
    events = np.ascontiguousarray(events, dtype=EVENT_DTYPE)
    last = C.c_int64(0)
    rc = lib().orc_validate(C.c_void_p(events.ctypes.data), C.c_int64(len(events)), C.c_int(p),
                            C.c_int(len(sizes)), _p(sizes, C.c_int64), C.c_int64(A), C.c_int64(B),
                            C.c_int64(G), C.c_int(1 if bidir else 0), C.c_int(1 if tree_rules else 0),
                            C.c_int(1 if in_order else 0), C.byref(last))
    return int(rc), last.value


def contributions(events, p, q):
    """0 when the root ends every segment holding each process's data exactly once."""
    events = np.ascontiguousarray(events, dtype=EVENT_DTYPE)
    return int(lib().orc_contributions(C.c_void_p(events.ctypes.data), C.c_int64(len(events)), C.c_int(p),
                                       C.c_int(q)))


def reduce(events, x, seg_off, op, half="bf16", openmp=False):
    """O2.  x: array [p, n] of int32, float32, int64, float64, or uint16 holding bf16 (half="bf16") or IEEE
    binary16 (half="fp16") bit patterns (C-contiguous); seg_off in elements of x; op 'sum', 'max', 'min' or 'prod'.
    openmp: run the OpenMP build (int32 and float32 only; same bits, used by the benchmark's all-cores leg)."""
    events = np.ascontiguousarray(events, dtype=EVENT_DTYPE)
    x = np.ascontiguousarray(x)
    p, n = x.shape
    seg_off = _i64(seg_off)
    q = len(seg_off) - 1
    assert seg_off[0] == 0 and seg_off[-1] == n
    out = np.empty(n, dtype=x.dtype)
    ptrs = (C.c_void_p * p)(*[x[i].ctypes.data for i in range(p)])
    opc = {"sum": 0, "max": 1, "min": 2, "prod": 3}[op]
    if x.dtype == np.int32:
        fn = lib(openmp).orc_reduce_i32
    elif x.dtype == np.float32:
        fn = lib(openmp).orc_reduce_f32
    elif openmp:
        raise TypeError("the OpenMP build serves int32 and float32 only")
    elif x.dtype == np.int64:
        fn = lib().orc_reduce_i64
    elif x.dtype == np.float64:
        fn = lib().orc_reduce_f64
    elif x.dtype == np.uint16:                 # 16-bit patterns: combined in fp32, rounded once at the end
        fn = lib().orc_reduce_bf16 if half == "bf16" else lib().orc_reduce_f16
    else:
        raise TypeError(x.dtype)
    rc = fn(C.c_void_p(events.ctypes.data), C.c_int64(len(events)), C.c_int(p), C.c_int(q),
            _p(seg_off, C.c_int64), ptrs, C.c_void_p(out.ctypes.data), C.c_int(opc))
    _check(rc, "reduce")
    return out


def reference_f64(x, op):
    """Order-free fp64 result and sum of magnitudes per element."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    p, n = x.shape
    ref = np.empty(n, dtype=np.float64)
    mag = np.empty(n, dtype=np.float64)
    ptrs = (C.c_void_p * p)(*[x[i].ctypes.data for i in range(p)])
    rc = lib().orc_reference_f64(C.c_int(p), C.c_int64(n), ptrs, C.c_void_p(ref.ctypes.data),
                                 C.c_void_p(mag.ctypes.data), C.c_int({"sum": 0, "max": 1}[op]))
    _check(rc, "reference_f64")
    return ref, mag


def unequal_times(p, A, G):
    """Section VIII: uni-greedy completion time of all 512 segmentations of 10 units (beta = 1)."""
    t = np.zeros(512, dtype=np.int64)
    _check(lib().orc_unequal_times(C.c_int(p), C.c_int64(A), C.c_int64(G), _p(t, C.c_int64)), "unequal_times")
    return t


def equal_sizes(m, s):
    """Equi-segmentation of m units: segments of s, the last possibly smaller (Section II)."""
    q = -(-m // s)
    sizes = [s] * q
    sizes[-1] = m - s * (q - 1)
    return sizes
