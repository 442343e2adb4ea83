"""Builds librd.so (CUDA kernels + C ABI) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys
import tempfile
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "librd.so")
SOURCES = ["rd_api.cpp", "rd_sched.cpp", "rd_compile.cpp", "rd_kernels.cu", "rd_faithful.cu", "rd_broadcast.cu"]
HEADERS = ["rd_internal.h", "rd_kernels.h"]
# rd_kernels.cu is compiled once per element type (-DRD_DT=k: that type's kernels; the 16-bit types count
# twice, once for sum and product and once for max and min) and once without (launch shapes and dispatch),
# side by side
KERNEL_DTYPES = 8
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC,-Wall,-Wextra,-fvisibility=hidden",
]
LINK_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-cudart", "static"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def stale() -> bool:
    if not os.path.exists(LIB):
        return True
    built = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS] + [os.path.join(ROOT, "include", "rd.h")]
    return any(os.path.getmtime(d) > built for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile when sources are newer than the library.  Returns the library path."""
    if not force and not stale():
        return LIB
    nvcc = _nvcc()
    common = [nvcc, *NVCC_FLAGS, "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    if verbose:
        common += ["-Xptxas", "-v"]
    work = tempfile.mkdtemp(prefix="librd_build_")
    try:
        units = []                                   # (object file, source, extra flags)
        for f in SOURCES:
            stem = os.path.splitext(f)[0]
            units.append((os.path.join(work, stem + ".o"), f, []))
            if f == "rd_kernels.cu":
                # (a unit that serves one element type leaves the other types' helpers unreferenced: diagnostic 177)
                units[-1] = (units[-1][0], f, ["-diag-suppress", "177"])
                for k in range(KERNEL_DTYPES):
                    units.append((os.path.join(work, "%s_dt%d.o" % (stem, k)), f, ["-DRD_DT=%d" % k, "-diag-suppress", "177"]))

        def compile_one(unit):
            obj, src, extra = unit
            subprocess.check_call(common + extra + ["-c", "-o", obj, os.path.join(CSRC, src)])
            return obj

        with ThreadPoolExecutor(max_workers=min(len(units), os.cpu_count() or 4)) as pool:
            objs = list(pool.map(compile_one, units))
        tmp = LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call([nvcc, *LINK_FLAGS, "-o", tmp] + objs)
        os.replace(tmp, LIB)
    finally:
        shutil.rmtree(work, ignore_errors=True)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
