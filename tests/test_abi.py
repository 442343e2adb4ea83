"""The C ABI: the library loads, exports what include/rd.h declares, and rejects bad arguments
(no GPU needed: nothing here launches a kernel)."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import paper_1310_4645_b200 as rd

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
MODEL = (2e-6, 1e-10, 5e-11)


def declared_functions():
    text = open(os.path.join(ROOT, "include", "rd.h")).read()
    return sorted(set(re.findall(r"RD_API\s+[\w\s\*]*?\b(rd_\w+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_functions()
    assert len(names) >= 12 and set(names) == set(rd.EXPORTS)
    L = C.CDLL(rd.LIB_PATH)
    for n in names:
        assert getattr(L, n) is not None


def test_only_the_abi_is_exported():
    """Internal C++ symbols stay hidden: the dynamic symbol table's rd:: / rd_ definitions are the ABI."""
    out = os.popen("nm -D --defined-only %s" % rd.LIB_PATH).read()
    mine = [ln.split()[-1] for ln in out.splitlines() if " T " in ln and ("rd" in ln.split()[-1])]
    assert sorted(m for m in mine if m.startswith("rd_")) == sorted(rd.EXPORTS)
    assert not [m for m in mine if m.startswith("_ZN2rd")]


def test_strerror():
    assert rd.rd_strerror(0) == "success"
    for code in range(-9, 0):
        assert rd.rd_strerror(code) and rd.rd_strerror(code) != "unknown status"
    assert rd.rd_strerror(-99) == "unknown status"


def status_of(fn, *a):
    with pytest.raises(rd.RdError) as e:
        fn(*a)
    return e.value.status


def test_create_rejects_bad_arguments():
    f = rd.rd_schedule_create
    assert status_of(f, rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, 0, 64, 16, *MODEL) == rd.RD_ERR_INVALID_ARG
    assert status_of(f, rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, 5000, 64, 16, *MODEL) == rd.RD_ERR_INVALID_ARG
    assert status_of(f, rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, 4, 66, 16, *MODEL) == rd.RD_ERR_INVALID_ARG
    assert status_of(f, rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, 4, 64, 18, *MODEL) == rd.RD_ERR_INVALID_ARG
    assert status_of(f, 17, rd.RD_PORT_UNI, 4, 64, 16, *MODEL) == rd.RD_ERR_INVALID_ARG
    assert status_of(f, rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, 4, 64, 16, -1.0, 1e-10, 0) == rd.RD_ERR_INVALID_ARG
    # pairs the method does not define
    assert status_of(f, rd.RD_UNI_GREEDY, rd.RD_PORT_BI, 4, 64, 16, *MODEL) == rd.RD_ERR_UNSUPPORTED
    assert status_of(f, rd.RD_BI_GREEDY, rd.RD_PORT_UNI, 4, 64, 16, *MODEL) == rd.RD_ERR_UNSUPPORTED
    assert status_of(f, rd.RD_BUTTERFLY, rd.RD_PORT_UNI, 4, 64, 16, *MODEL) == rd.RD_ERR_UNSUPPORTED
    assert status_of(rd.rd_schedule_create_segments, rd.RD_BUTTERFLY, rd.RD_PORT_BI, 4, [32, 32], *MODEL) \
        == rd.RD_ERR_UNSUPPORTED
    assert status_of(rd.rd_schedule_create_segments, rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, 4, [32, 0], *MODEL) \
        == rd.RD_ERR_INVALID_ARG
    # null pointers straight through ctypes
    L = rd.lib()
    m = rd.rd_model_t(*MODEL, 0.0)
    assert L.rd_schedule_create(None, 0, 0, 4, 64, 16, C.byref(m)) == rd.RD_ERR_INVALID_ARG
    h = C.c_void_p(0x1234)
    assert L.rd_schedule_create(C.byref(h), 0, 0, 4, 64, 16, None) == rd.RD_ERR_INVALID_ARG
    assert h.value == 0x1234            # untouched on failure
    L.rd_destroy(None)                  # allowed


def test_info_events_segments_program_capacity_checks():
    h = rd.rd_schedule_create(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, 8, 16384, 2048, *MODEL)
    try:
        info = rd.rd_schedule_info(h)
        assert info["p"] == 8 and info["q"] == 8 and info["n_events"] == 56
        L = rd.lib()
        buf = np.zeros(10, dtype=rd.EVENT_DTYPE)
        assert L.rd_schedule_events(h, buf.ctypes.data, 10) == rd.RD_ERR_TOO_SMALL
        off = np.zeros(4, dtype=np.uint64)
        assert L.rd_schedule_segments(h, off.ctypes.data, 4) == rd.RD_ERR_TOO_SMALL
        ops = np.zeros(4, dtype=np.uint32)
        assert L.rd_schedule_program(h, 0, ops.ctypes.data, 4) == rd.RD_ERR_TOO_SMALL
        assert L.rd_schedule_program(h, 8, ops.ctypes.data, 4) == rd.RD_ERR_INVALID_ARG
        assert (rd.rd_schedule_segments(h) == np.arange(9) * 512).all()
        # argument checks of rd_reduce come before any CUDA call
        ptrs = (C.c_void_p * 8)(*([0x1000] * 8))
        assert L.rd_reduce(h, ptrs, 0x2000, 100, rd.RD_INT32, rd.RD_SUM, rd.RD_EXEC_TREE, None, None) \
            == rd.RD_ERR_SIZE_MISMATCH
        assert L.rd_reduce(h, ptrs, 0x2000, 4096, 7, rd.RD_SUM, rd.RD_EXEC_TREE, None, None) == rd.RD_ERR_INVALID_ARG
        assert L.rd_reduce(h, ptrs, None, 4096, rd.RD_INT32, rd.RD_SUM, rd.RD_EXEC_TREE, None, None) \
            == rd.RD_ERR_INVALID_ARG
        ptrs[3] = 0x1002                 # misaligned input
        assert L.rd_reduce(h, ptrs, 0x2000, 4096, rd.RD_INT32, rd.RD_SUM, rd.RD_EXEC_TREE, None, None) \
            == rd.RD_ERR_INVALID_ARG
        # 8-byte element types: half as many elements, buffers aligned to 8 bytes
        ptrs = (C.c_void_p * 8)(*([0x1000] * 8))
        assert L.rd_reduce(h, ptrs, 0x2000, 4096, rd.RD_FP64, rd.RD_SUM, rd.RD_EXEC_TREE, None, None) \
            == rd.RD_ERR_SIZE_MISMATCH
        ptrs[5] = 0x1004
        assert L.rd_reduce(h, ptrs, 0x2000, 2048, rd.RD_INT64, rd.RD_SUM, rd.RD_EXEC_TREE, None, None) \
            == rd.RD_ERR_INVALID_ARG
    finally:
        rd.rd_destroy(h)
    # a segment boundary inside an 8-byte element is refused before any CUDA call
    h = rd.rd_schedule_create(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, 4, 64, 12, *MODEL)
    try:
        ptrs = (C.c_void_p * 4)(*([0x1000] * 4))
        assert rd.lib().rd_reduce(h, ptrs, 0x2000, 8, rd.RD_FP64, rd.RD_SUM, rd.RD_EXEC_TREE, None, None) \
            == rd.RD_ERR_INVALID_ARG
        assert rd.lib().rd_reduce_faithful_static(h, ptrs, 0x2000, 8, rd.RD_INT64, rd.RD_MAX, None, None) \
            == rd.RD_ERR_INVALID_ARG
    finally:
        rd.rd_destroy(h)


def test_missing_library_fails_loudly(monkeypatch):
    import paper_1310_4645_b200.binding as b
    monkeypatch.setattr(b, "_lib", None)
    monkeypatch.setattr(b, "LIB_PATH", "/nonexistent/librd.so")
    with pytest.raises(ImportError):
        b.rd_schedule_create(0, 0, 4, 64, 16, *MODEL)


def test_empty_message_and_single_process():
    h = rd.rd_schedule_create(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, 4, 0, 16, *MODEL)
    assert rd.rd_schedule_info(h)["q"] == 0 and rd.rd_schedule_info(h)["n_events"] == 0
    rd.rd_destroy(h)
    h = rd.rd_schedule_create(rd.RD_PIPELINE, rd.RD_PORT_BI, 1, 64, 16, *MODEL)
    info = rd.rd_schedule_info(h)
    assert info["q"] == 4 and info["n_events"] == 0 and info["predicted_ticks"] == 0
    assert list(rd.rd_schedule_program(h, 2)) == [0]      # LOAD process 0
    rd.rd_destroy(h)


def test_batch_argument_checks_come_before_any_cuda_call():
    L = rd.lib()
    h = rd.rd_schedule_create(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, 4, 4096, 1024, *MODEL)
    try:
        vp = C.c_void_p
        def call(in_addrs, out_addrs, n=1024):
            k = len(out_addrs)
            tabs = [(vp * 4)(*a) for a in in_addrs]
            return L.rd_reduce_batch(k, (vp * k)(*[h] * k), (vp * k)(*[C.cast(t, vp).value for t in tabs]),
                                     (vp * k)(*out_addrs), (C.c_size_t * k)(*[n] * k), rd.RD_FP32, rd.RD_SUM, None)
        rows = lambda base: [base + i * 4096 for i in range(4)]
        assert L.rd_reduce_batch(0, None, None, None, None, rd.RD_FP32, rd.RD_SUM, None) == rd.RD_OK
        assert L.rd_reduce_batch(1, None, None, None, None, rd.RD_FP32, rd.RD_SUM, None) == rd.RD_ERR_INVALID_ARG
        # job 1 writes into job 0's second input
        assert call([rows(0x100000), rows(0x200000)], [0x300000, 0x101000]) == rd.RD_ERR_INVALID_ARG
        # the two outputs overlap
        assert call([rows(0x100000), rows(0x200000)], [0x300000, 0x300800]) == rd.RD_ERR_INVALID_ARG
        # wrong length
        assert call([rows(0x100000)], [0x300000], n=1000) == rd.RD_ERR_SIZE_MISMATCH
    finally:
        rd.rd_destroy(h)


def test_tree_variant_is_checked_on_the_host():
    """Choosing the tree-mode kernel is host work: the direct kernel exists for at most 8 processes."""
    for p, direct_ok in ((1, True), (2, True), (8, True), (9, False), (64, False)):
        h = rd.rd_schedule_create(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, p, 4096, 1024, *MODEL)
        try:
            rd.rd_schedule_set_tree_variant(h, rd.RD_TREE_STREAM)
            rd.rd_schedule_set_tree_variant(h, rd.RD_TREE_AUTO)
            if direct_ok:
                rd.rd_schedule_set_tree_variant(h, rd.RD_TREE_DIRECT)
            else:
                assert status_of(rd.rd_schedule_set_tree_variant, h, rd.RD_TREE_DIRECT) == rd.RD_ERR_UNSUPPORTED
            assert status_of(rd.rd_schedule_set_tree_variant, h, 4) == rd.RD_ERR_INVALID_ARG
            assert status_of(rd.rd_schedule_set_tree_variant, h, -1) == rd.RD_ERR_INVALID_ARG
        finally:
            rd.rd_destroy(h)
    assert rd.lib().rd_schedule_set_tree_variant(None, rd.RD_TREE_AUTO) == rd.RD_ERR_INVALID_ARG
    assert rd.lib().rd_schedule_tree_shape(None, None, None, None, None) == rd.RD_ERR_INVALID_ARG


def test_binding_constants_match_the_header():
    """Every enumerator of include/rd.h has the same value in the binding."""
    text = open(os.path.join(ROOT, "include", "rd.h")).read()
    seen = 0
    for body in re.findall(r"typedef enum\s*\{(.*?)\}", text, flags=re.S):
        body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
        value = -1
        for item in body.split(","):
            item = item.strip()
            if not item:
                continue
            if "=" in item:
                name, v = [t.strip() for t in item.split("=")]
                value = int(v, 0)
            else:
                name, value = item, value + 1
            assert hasattr(rd, name), name
            assert getattr(rd, name) == value, name
            seen += 1
    assert seen >= 30


def test_a_model_whose_communications_take_no_time_is_refused():
    """alpha = beta = 0 (in ticks): every send would start and end at time 0, the event order is undefined."""
    for f, args in ((rd.rd_schedule_create, (rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, 8, 4096, 1024)),
                    (rd.rd_schedule_create, (rd.RD_BI_GREEDY, rd.RD_PORT_BI, 8, 4096, 1024)),
                    (rd.rd_schedule_create, (rd.RD_BUTTERFLY, rd.RD_PORT_BI, 8, 4096, 0)),
                    (rd.rd_schedule_create_segments, (rd.RD_PIPELINE, rd.RD_PORT_UNI, 8, [1024, 512])),
                    (rd.rd_optimal_segment, (rd.RD_BINARY, rd.RD_PORT_BI, 8, 4096)),
                    (rd.rd_search_segmentation, (8, 4096, 4))):
        assert status_of(f, *args, 0.0, 0.0, 0.0) == rd.RD_ERR_INVALID_ARG
        assert status_of(f, *args, 0.0, 0.0, 5e-11) == rd.RD_ERR_INVALID_ARG
        assert status_of(f, *args, 1e-17, 1e-17, 5e-11) == rd.RD_ERR_INVALID_ARG      # both round to 0 ticks of 1 fs
    # either of the two alone is enough, and gamma may be zero
    for model in ((2e-6, 0.0, 0.0), (0.0, 1e-10, 0.0), (0.0, 1.0, 1.0, 1.0)):
        h = rd.rd_schedule_create(rd.RD_BI_GREEDY, rd.RD_PORT_BI, 8, 4096, 1024, *model)
        assert rd.rd_schedule_info(h)["n_events"] == 7 * 4
        rd.rd_destroy(h)


def test_distinct_schedules_from_distinct_threads():
    """The header's promise: threads that each own their schedules need no lock around the library."""
    import threading
    from helpers import oracle_schedule
    cases = [(rd.RD_UNI_GREEDY, rd.RD_PORT_UNI, 37, 40000, 1000), (rd.RD_BI_GREEDY, rd.RD_PORT_BI, 24, 36000, 1200),
             (rd.RD_BINARY, rd.RD_PORT_BI, 100, 8000, 400), (rd.RD_BUTTERFLY, rd.RD_PORT_BI, 16, 64000, 0)]
    want = [oracle_schedule(a, pt, p, m, s if s else m, *MODEL) for a, pt, p, m, s in cases]
    errors = []

    def work(k):
        try:
            for rep in range(20):
                a, pt, p, m, s = cases[(k + rep) % len(cases)]
                ev, off, comp = want[(k + rep) % len(cases)]
                h = rd.rd_schedule_create(a, pt, p, m, s, *MODEL)
                try:
                    got = rd.rd_schedule_events(h)
                    assert rd.rd_schedule_info(h)["predicted_ticks"] == comp
                    for f in ("seg", "src", "dst", "t_start"):
                        assert (got[f] == ev[f]).all()
                    assert (rd.rd_schedule_segments(h) == off).all()
                finally:
                    rd.rd_destroy(h)
        except BaseException as e:      # noqa: BLE001 - reported by the main thread
            errors.append(repr(e))

    threads = [threading.Thread(target=work, args=(k,)) for k in range(4)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
