"""Build step: compile the CUDA sources in csrc/ into libmxfp8.so (sm_100a only), in-tree."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libmxfp8.so")
# the same sources with -DMXFP8_TEST_HOOKS: wait limits of milliseconds and switches that leave one load out, so that
# the tests can watch a bounded wait run out without hanging anything.  Never loaded by the binding.
LIB_TEST_HOOKS = os.path.join(HERE, "libmxfp8_testhooks.so")
SOURCES = ["quantize.cu", "quantize_tma.cu", "quantize_tma_fp6_fp4.cu", "dequantize.cu", "gemm.cu", "gemm_deep.cu", "api.cu"]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-shared", "-Xcompiler", "-fPIC",
    # static locals of template functions must stay private to each copy of the library that a process loads (the test
    # build is loaded beside the product): GNU "unique" symbols would be shared across them
    "-Xcompiler", "-fno-gnu-unique",
]


def _stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    deps.append(os.path.join(os.path.dirname(HERE), "include", "mxfp8.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, test_hooks: bool = False) -> str:
    """Compile with nvcc if the library is missing or older than its sources: one object file
    per source (in parallel), then one link.  test_hooks=True builds the test variant instead."""
    LIB = LIB_TEST_HOOKS if test_hooks else globals()["LIB"]
    if not (force or _stale(LIB)):
        return LIB
    from concurrent.futures import ThreadPoolExecutor
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    objdir = os.path.join(HERE, ".obj.%d" % os.getpid())
    os.makedirs(objdir, exist_ok=True)
    compile_flags = [f for f in NVCC_FLAGS if f != "-shared"] + (["-Xptxas", "-v"] if verbose else [])
    if test_hooks:
        compile_flags.append("-DMXFP8_TEST_HOOKS")

    def compile_one(src):
        obj = os.path.join(objdir, src + ".o")
        subprocess.check_call([nvcc] + compile_flags + ["-c", os.path.join(CSRC, src), "-o", obj])
        return obj

    try:
        with ThreadPoolExecutor(max_workers=len(SOURCES)) as pool:
            objs = list(pool.map(compile_one, SOURCES))
        tmp = LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call([nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", tmp] + objs)
        os.replace(tmp, LIB)
    finally:
        for f in os.listdir(objdir):
            os.remove(os.path.join(objdir, f))
        os.rmdir(objdir)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, test_hooks="--test-hooks" in sys.argv))
