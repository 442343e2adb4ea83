"""Thin ctypes binding of librd.so: the same names as include/rd.h, argument marshalling only.

Nothing is computed here.  When the shared library is missing (not built) every call fails with
an ImportError-derived exception: there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "librd.so")

RD_OK = 0
RD_ERR_INVALID_ARG, RD_ERR_UNSUPPORTED, RD_ERR_NOMEM, RD_ERR_CUDA = -1, -2, -3, -4
RD_ERR_TIMEOUT, RD_ERR_SIZE_MISMATCH, RD_ERR_INTERNAL, RD_ERR_TOO_SMALL = -5, -6, -7, -8
RD_ERR_TOO_LARGE = -9
RD_UNI_GREEDY, RD_BI_GREEDY, RD_BINOMIAL, RD_PIPELINE, RD_BINARY, RD_BUTTERFLY = range(6)
RD_PORT_UNI, RD_PORT_BI = 0, 1
RD_SUM, RD_MAX, RD_MIN, RD_PROD = 0, 1, 2, 3
RD_INT32, RD_FP32, RD_INT64, RD_FP64, RD_BF16, RD_FP16 = 0, 1, 2, 3, 4, 5
RD_EXEC_TREE, RD_EXEC_FAITHFUL = 0, 1
RD_TREE_AUTO, RD_TREE_STREAM, RD_TREE_DIRECT, RD_TREE_STREAM_PAIRED = 0, 1, 2, 3

ALGOS = {"uni_greedy": RD_UNI_GREEDY, "bi_greedy": RD_BI_GREEDY, "binomial": RD_BINOMIAL,
         "pipeline": RD_PIPELINE, "binary": RD_BINARY, "butterfly": RD_BUTTERFLY}

EXPORTS = ("rd_schedule_create", "rd_schedule_create_segments", "rd_optimal_segment", "rd_schedule_info",
           "rd_schedule_events", "rd_schedule_segments", "rd_schedule_program", "rd_reduce",
           "rd_schedule_upload", "rd_reduce_host", "rd_destroy", "rd_strerror", "rd_schedule_set_wait_budget",
           "rd_schedule_trace", "rd_schedule_faithful_shape", "rd_schedule_actions", "rd_reduce_faithful_static", "rd_search_segmentation", "rd_schedule_status",
           "rd_reduce_batch", "rd_schedule_set_tree_variant", "rd_schedule_tree_shape", "rd_allreduce")


class rd_model_t(C.Structure):
    _fields_ = [("alpha", C.c_double), ("beta", C.c_double), ("gamma", C.c_double), ("tick", C.c_double)]


class rd_stats_t(C.Structure):
    _fields_ = [("kernel_ms", C.c_double), ("gbytes_per_s", C.c_double), ("makespan_ns", C.c_double),
                ("predicted_s", C.c_double), ("bytes_moved", C.c_uint64), ("device_status", C.c_int32),
                ("n_launches", C.c_int32)]


EVENT_DTYPE = np.dtype(
    [("seg", "<i4"), ("src", "<i4"), ("dst", "<i4"), ("kind", "<i4"), ("t_start", "<i8")], align=True)


class RdError(RuntimeError):
    def __init__(self, status, what):
        self.status = status
        super().__init__("%s: %s (%d)" % (what, rd_strerror(status), status))


class LibraryMissing(ImportError):
    pass


_lib = None


def lib():
    """The loaded library.  Raises LibraryMissing when librd.so has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise LibraryMissing("librd.so not found at %s: build it with `python -m paper_1310_4645_b200.build`"
                                 % LIB_PATH)
        L = C.CDLL(LIB_PATH)
        vp, sz, i32 = C.c_void_p, C.c_size_t, C.c_int
        L.rd_schedule_create.argtypes = [C.POINTER(vp), i32, i32, i32, sz, sz, C.POINTER(rd_model_t)]
        L.rd_schedule_create_segments.argtypes = [C.POINTER(vp), i32, i32, i32, C.POINTER(sz), sz, C.POINTER(rd_model_t)]
        L.rd_optimal_segment.argtypes = [i32, i32, i32, sz, C.POINTER(rd_model_t), C.POINTER(sz)]
        L.rd_schedule_info.argtypes = [vp, C.POINTER(i32), C.POINTER(sz), C.POINTER(sz), C.POINTER(C.c_double),
                                       C.POINTER(C.c_int64), C.POINTER(i32)]
        L.rd_schedule_events.argtypes = [vp, vp, sz]
        L.rd_schedule_segments.argtypes = [vp, vp, sz]
        L.rd_schedule_program.argtypes = [vp, sz, vp, sz]
        L.rd_reduce.argtypes = [vp, C.POINTER(vp), vp, sz, i32, i32, i32, vp, C.POINTER(rd_stats_t)]
        L.rd_schedule_upload.argtypes = [vp]
        L.rd_allreduce.argtypes = [vp, C.POINTER(vp), C.POINTER(vp), sz, i32, i32, vp, C.POINTER(rd_stats_t)]
        L.rd_reduce_host.argtypes = [vp, C.POINTER(vp), vp, vp, sz, i32, i32, vp]
        L.rd_schedule_set_wait_budget.argtypes = [vp, C.c_double]
        L.rd_schedule_set_tree_variant.argtypes = [vp, i32]
        L.rd_schedule_tree_shape.argtypes = [vp, C.POINTER(i32), C.POINTER(i32), C.POINTER(i32), C.POINTER(sz)]
        L.rd_schedule_trace.argtypes = [vp, vp, sz]
        L.rd_schedule_faithful_shape.argtypes = [vp, C.POINTER(i32), C.POINTER(i32), C.POINTER(sz)]
        L.rd_schedule_actions.argtypes = [vp, i32, vp, sz, C.POINTER(sz), C.POINTER(i32)]
        L.rd_reduce_faithful_static.argtypes = [vp, C.POINTER(vp), vp, sz, i32, i32, vp, C.POINTER(rd_stats_t)]
        L.rd_search_segmentation.argtypes = [i32, sz, sz, C.POINTER(rd_model_t), C.POINTER(sz), sz, C.POINTER(sz),
                                             C.POINTER(C.c_int64)]
        L.rd_schedule_status.argtypes = [vp, C.POINTER(i32)]
        L.rd_reduce_batch.argtypes = [sz, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), C.POINTER(sz), i32, i32, vp]
        L.rd_destroy.argtypes = [vp]
        L.rd_destroy.restype = None
        L.rd_strerror.argtypes = [i32]
        L.rd_strerror.restype = C.c_char_p
        for name in EXPORTS:
            if name not in ("rd_destroy", "rd_strerror"):
                getattr(L, name).restype = i32
        _lib = L
    return _lib


def rd_strerror(status: int) -> str:
    return lib().rd_strerror(int(status)).decode()


def _check(status, what):
    if status != RD_OK:
        raise RdError(status, what)


def _model(alpha, beta, gamma, tick=0.0):
    return rd_model_t(float(alpha), float(beta), float(gamma), float(tick))


def rd_schedule_create(algo, port, p, msg_bytes, seg_bytes, alpha, beta, gamma, tick=0.0):
    """Returns an opaque schedule handle (int).  Release with rd_destroy."""
    h = C.c_void_p()
    m = _model(alpha, beta, gamma, tick)
    _check(lib().rd_schedule_create(C.byref(h), int(algo), int(port), int(p), int(msg_bytes), int(seg_bytes),
                                    C.byref(m)), "rd_schedule_create")
    return h.value


def rd_schedule_create_segments(algo, port, p, seg_bytes, alpha, beta, gamma, tick=0.0):
    h = C.c_void_p()
    m = _model(alpha, beta, gamma, tick)
    arr = (C.c_size_t * len(seg_bytes))(*[int(s) for s in seg_bytes])
    _check(lib().rd_schedule_create_segments(C.byref(h), int(algo), int(port), int(p), arr, len(seg_bytes),
                                             C.byref(m)), "rd_schedule_create_segments")
    return h.value


def rd_optimal_segment(algo, port, p, msg_bytes, alpha, beta, gamma, tick=0.0) -> int:
    out = C.c_size_t(0)
    m = _model(alpha, beta, gamma, tick)
    _check(lib().rd_optimal_segment(int(algo), int(port), int(p), int(msg_bytes), C.byref(m), C.byref(out)),
           "rd_optimal_segment")
    return out.value


def rd_schedule_info(h) -> dict:
    p, q, ne, sec, ticks, depth = C.c_int(), C.c_size_t(), C.c_size_t(), C.c_double(), C.c_int64(), C.c_int()
    _check(lib().rd_schedule_info(h, C.byref(p), C.byref(q), C.byref(ne), C.byref(sec), C.byref(ticks),
                                  C.byref(depth)), "rd_schedule_info")
    return dict(p=p.value, q=q.value, n_events=ne.value, predicted_seconds=sec.value,
                predicted_ticks=ticks.value, stack_depth=depth.value)


def rd_schedule_events(h) -> np.ndarray:
    n = rd_schedule_info(h)["n_events"]
    ev = np.zeros(n, dtype=EVENT_DTYPE)
    _check(lib().rd_schedule_events(h, ev.ctypes.data, n), "rd_schedule_events")
    return ev


def rd_schedule_segments(h) -> np.ndarray:
    q = rd_schedule_info(h)["q"]
    off = np.zeros(q + 1, dtype=np.uint64)
    _check(lib().rd_schedule_segments(h, off.ctypes.data, q + 1), "rd_schedule_segments")
    return off


def rd_schedule_program(h, seg) -> np.ndarray:
    p = rd_schedule_info(h)["p"]
    ops = np.zeros(p, dtype=np.uint32)
    _check(lib().rd_schedule_program(h, int(seg), ops.ctypes.data, p), "rd_schedule_program")
    return ops


def rd_schedule_upload(h) -> None:
    _check(lib().rd_schedule_upload(h), "rd_schedule_upload")


def _dtype_code(t):
    import torch
    if t.dtype == torch.int32:
        return RD_INT32
    if t.dtype == torch.float32:
        return RD_FP32
    if t.dtype == torch.int64:
        return RD_INT64
    if t.dtype == torch.float64:
        return RD_FP64
    if t.dtype == torch.bfloat16:
        return RD_BF16
    if t.dtype == torch.float16:
        return RD_FP16
    raise TypeError("int32, float32, int64, float64, bfloat16 or float16 expected, got %s" % t.dtype)


class PointerTable:
    """The host array of p device (or host) pointers rd_reduce takes, built once and reusable.

    `inputs` is either one contiguous [p, n] tensor (row i = process i) or a sequence of p contiguous
    1-D tensors.  The table keeps the tensors alive."""

    def __init__(self, inputs):
        import torch
        if isinstance(inputs, torch.Tensor):
            if inputs.dim() != 2 or not inputs.is_contiguous():
                raise ValueError("a [p, n] contiguous tensor is expected")
            self.p, self.n = int(inputs.shape[0]), int(inputs.shape[1])
            addr = inputs.data_ptr() + np.arange(self.p, dtype=np.uint64) * np.uint64(self.n * inputs.element_size())
            self.dtype, self.is_cuda, self.device = inputs.dtype, inputs.is_cuda, inputs.device
        else:
            rows = list(inputs)
            if not rows:
                raise ValueError("at least one process is needed")
            self.p, self.n = len(rows), int(rows[0].numel())
            for r in rows:
                if not r.is_contiguous() or r.numel() != self.n or r.dtype != rows[0].dtype or r.is_cuda != rows[0].is_cuda:
                    raise ValueError("every input must be contiguous, of the same length, dtype and placement")
            addr = np.array([r.data_ptr() for r in rows], dtype=np.uint64)
            self.dtype, self.is_cuda, self.device = rows[0].dtype, rows[0].is_cuda, rows[0].device
        self._keep = inputs
        self._addr = np.ascontiguousarray(addr)
        self.array = C.cast(self._addr.ctypes.data, C.POINTER(C.c_void_p))


def rd_reduce(h, inputs, out, op, exec_mode=RD_EXEC_TREE, stream=None, want_stats=False):
    """inputs: a PointerTable, a [p, n] CUDA tensor or a list of p CUDA tensors; out: CUDA tensor of n
    elements.  stream: a torch.cuda.Stream (default: the current one).  Returns rd_stats_t or None."""
    import torch
    tab = inputs if isinstance(inputs, PointerTable) else PointerTable(inputs)
    n = out.numel()
    if not tab.is_cuda or tab.n != n or tab.dtype != out.dtype:
        raise ValueError("every input must be a contiguous CUDA tensor with the output's dtype and length")
    if not out.is_cuda or not out.is_contiguous():
        raise ValueError("out must be a contiguous CUDA tensor")
    s = stream if stream is not None else torch.cuda.current_stream(out.device)
    stats = rd_stats_t() if want_stats else None
    prev = torch.cuda.current_device()
    if out.device.index != prev:
        torch.cuda.set_device(out.device)
    try:
        _check(lib().rd_reduce(h, tab.array, out.data_ptr(), n, _dtype_code(out), int(op), int(exec_mode),
                               s.cuda_stream, C.byref(stats) if want_stats else None), "rd_reduce")
    finally:
        if out.device.index != prev:
            torch.cuda.set_device(prev)
    return stats


def rd_allreduce(h, inputs, outs, op, stream=None, want_stats=False):
    """inputs, outs: each a PointerTable, a [p, n] CUDA tensor or a list of p CUDA tensors; outs[i] receives
    process i's copy of the result and may be inputs[i] itself.  Returns rd_stats_t or None."""
    import torch
    tab = inputs if isinstance(inputs, PointerTable) else PointerTable(inputs)
    otab = outs if isinstance(outs, PointerTable) else PointerTable(outs)
    if not tab.is_cuda or not otab.is_cuda or tab.n != otab.n or tab.p != otab.p or tab.dtype != otab.dtype or tab.device != otab.device:
        raise ValueError("inputs and outs must be p contiguous CUDA tensors each, of one dtype, length and device")
    s = stream if stream is not None else torch.cuda.current_stream(tab.device)
    stats = rd_stats_t() if want_stats else None
    with torch.cuda.device(tab.device):
        _check(lib().rd_allreduce(h, tab.array, otab.array, tab.n, _dtype_code(tab), int(op), s.cuda_stream,
                                  C.byref(stats) if want_stats else None), "rd_allreduce")
    return stats


class Batch:
    """Marshalled arguments of rd_reduce_batch, built once and reused: jobs = [(schedule, inputs, out)], inputs
    a PointerTable, a [p, n] CUDA tensor or a list of p CUDA tensors."""

    def __init__(self, jobs):
        self.tables = [t if isinstance(t, PointerTable) else PointerTable(t) for _, t, _ in jobs]
        self.outs = [o for _, _, o in jobs]
        k = len(jobs)
        for tab, out in zip(self.tables, self.outs):
            if not out.is_cuda or not out.is_contiguous() or not tab.is_cuda or tab.n != out.numel() or tab.dtype != out.dtype:
                raise ValueError("every input must be a contiguous CUDA tensor with its output's dtype and length")
            if out.dtype != self.outs[0].dtype or out.device != self.outs[0].device:
                raise ValueError("all jobs of a batch share the element type and the device")
        self.k = k
        self.schedules = (C.c_void_p * k)(*[h for h, _, _ in jobs])
        self.inputs = (C.c_void_p * k)(*[C.cast(t.array, C.c_void_p).value for t in self.tables])
        self.out_ptrs = (C.c_void_p * k)(*[o.data_ptr() for o in self.outs])
        self.n_elems = (C.c_size_t * k)(*[o.numel() for o in self.outs])
        self.dtype = _dtype_code(self.outs[0]) if k else RD_FP32
        self.device = self.outs[0].device if k else None


def rd_reduce_batch(jobs, op, stream=None):
    """jobs: a Batch, or a list of (schedule, inputs, out).  Independent reductions issued together."""
    import torch
    b = jobs if isinstance(jobs, Batch) else Batch(jobs)
    if b.k == 0:
        return
    s = stream if stream is not None else torch.cuda.current_stream(b.device)
    prev = torch.cuda.current_device()
    if b.device.index != prev:
        torch.cuda.set_device(b.device)
    try:
        _check(lib().rd_reduce_batch(b.k, b.schedules, b.inputs, b.out_ptrs, b.n_elems, b.dtype, int(op), s.cuda_stream),
               "rd_reduce_batch")
    finally:
        if b.device.index != prev:
            torch.cuda.set_device(prev)


def rd_reduce_faithful_static(h, inputs, out, op, stream=None, want_stats=False):
    """The schedule-faithful reduction without any device allocation (scratch in the library's fixed
    32 MiB device array).  Same arguments as rd_reduce; see include/rd.h for who needs this and for the
    rules (one call at a time, first call per device outside stream capture)."""
    import torch
    tab = inputs if isinstance(inputs, PointerTable) else PointerTable(inputs)
    n = out.numel()
    if not tab.is_cuda or tab.n != n or tab.dtype != out.dtype:
        raise ValueError("every input must be a contiguous CUDA tensor with the output's dtype and length")
    if not out.is_cuda or not out.is_contiguous():
        raise ValueError("out must be a contiguous CUDA tensor")
    s = stream if stream is not None else torch.cuda.current_stream(out.device)
    stats = rd_stats_t() if want_stats else None
    with torch.cuda.device(out.device):
        _check(lib().rd_reduce_faithful_static(h, tab.array, out.data_ptr(), n, _dtype_code(out), int(op),
                                               s.cuda_stream, C.byref(stats) if want_stats else None),
               "rd_reduce_faithful_static")
    return stats


def rd_reduce_host(h, inputs, out, staging, op, stream=None):
    """inputs: a PointerTable, a [p, n] host tensor or a list of p host tensors (pinned memory makes the
    copies asynchronous); out: host tensor; staging: CUDA tensor of (p + 1) * n elements."""
    import torch
    tab = inputs if isinstance(inputs, PointerTable) else PointerTable(inputs)
    n = out.numel()
    if tab.is_cuda or tab.n != n or tab.dtype != out.dtype or out.is_cuda:
        raise ValueError("inputs and out must be contiguous host tensors of the same dtype and length")
    if staging.numel() < (tab.p + 1) * n or staging.dtype != out.dtype or not staging.is_cuda:
        raise ValueError("staging must be a CUDA tensor of (p + 1) * n elements")
    s = stream if stream is not None else torch.cuda.current_stream(staging.device)
    with torch.cuda.device(staging.device):
        _check(lib().rd_reduce_host(h, tab.array, out.data_ptr(), staging.data_ptr(), n, _dtype_code(out), int(op),
                                    s.cuda_stream), "rd_reduce_host")


def rd_schedule_set_wait_budget(h, seconds) -> None:
    _check(lib().rd_schedule_set_wait_budget(h, float(seconds)), "rd_schedule_set_wait_budget")


def rd_schedule_set_tree_variant(h, variant) -> None:
    _check(lib().rd_schedule_set_tree_variant(h, int(variant)), "rd_schedule_set_tree_variant")


def rd_schedule_tree_shape(h) -> dict:
    v, b, r, t = C.c_int(), C.c_int(), C.c_int(), C.c_size_t()
    _check(lib().rd_schedule_tree_shape(h, C.byref(v), C.byref(b), C.byref(r), C.byref(t)), "rd_schedule_tree_shape")
    return dict(variant=v.value, blocks_per_sm=b.value, ring_stages=r.value, n_tiles=t.value)


def rd_schedule_trace(h) -> np.ndarray:
    """[n_events, 3] uint64 nanoseconds: receiver ready, data available, combine written."""
    n = rd_schedule_info(h)["n_events"]
    t = np.zeros((n, 3), dtype=np.uint64)
    _check(lib().rd_schedule_trace(h, t.ctypes.data, n), "rd_schedule_trace")
    return t


def rd_schedule_faithful_shape(h) -> dict:
    b, s, sc = C.c_int(), C.c_int(), C.c_size_t()
    _check(lib().rd_schedule_faithful_shape(h, C.byref(b), C.byref(s), C.byref(sc)), "rd_schedule_faithful_shape")
    return dict(blocks_per_process=b.value, slots_per_process=s.value, scratch_bytes=sc.value)


ACTION_FIELDS = ("seg", "peer", "kind", "slot", "peer_slot", "first", "event", "wait_event")


def rd_schedule_actions(h, process):
    """(actions as an [n, 8] int32 array with columns ACTION_FIELDS, scratch slots per process)."""
    n, slots = C.c_size_t(), C.c_int()
    rc = lib().rd_schedule_actions(h, int(process), None, 0, C.byref(n), C.byref(slots))
    if rc not in (RD_OK, RD_ERR_TOO_SMALL):
        raise RdError(rc, "rd_schedule_actions")
    buf = np.zeros((n.value, 8), dtype=np.int32)
    _check(lib().rd_schedule_actions(h, int(process), buf.ctypes.data, n.value, C.byref(n), C.byref(slots)),
           "rd_schedule_actions")
    return buf, slots.value


def rd_search_segmentation(p, msg_bytes, unit_bytes, alpha, beta, gamma, tick=0.0):
    """(segment sizes in bytes, predicted completion ticks) of the local search around the best equi-segmentation."""
    m = _model(alpha, beta, gamma, tick)
    cap = int(msg_bytes) // int(unit_bytes) if unit_bytes else 0
    arr = (C.c_size_t * max(cap, 1))()
    q, ticks = C.c_size_t(), C.c_int64()
    _check(lib().rd_search_segmentation(int(p), int(msg_bytes), int(unit_bytes), C.byref(m), arr, cap, C.byref(q),
                                        C.byref(ticks)), "rd_search_segmentation")
    return [int(arr[j]) for j in range(q.value)], ticks.value


def rd_schedule_status(h) -> int:
    """Waits for the device and returns (and clears) the status word of the schedule's kernels."""
    st = C.c_int(0)
    _check(lib().rd_schedule_status(h, C.byref(st)), "rd_schedule_status")
    return st.value


def rd_destroy(h) -> None:
    lib().rd_destroy(h)
