"""Builds libbitdelta.so in-tree with nvcc for sm_100a (cross-compiles without a GPU).

Every source is compiled to an object file on its own (in parallel), then linked; objects live in
csrc/build/ and are rebuilt only when their source or a header is newer.
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(CSRC, "build")
LIB = os.path.join(HERE, "libbitdelta.so")
SOURCES = ["api.cu", "gemm_tc.cu", "gemm_fp4.cu", "kernels_simple.cu"]
HEADERS = ["ptx.cuh", "plan.h", "gemm_tc.h", "gemm_common.cuh", os.path.join("..", "..", "include", "bitdelta.h")]
ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]


def _nvcc() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def _newest_header() -> float:
    return max(os.path.getmtime(os.path.join(CSRC, h)) for h in HEADERS if os.path.exists(os.path.join(CSRC, h)))


def is_stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS]
    return any(os.path.getmtime(d) > t for d in deps if os.path.exists(d))


def _compile(src: str, force: bool, verbose: bool, trace: bool = False, steps: bool = False) -> str:
    obj = os.path.join(OBJ, os.path.splitext(src)[0] + (".steps.o" if steps else ".trace.o" if trace else ".o"))
    path = os.path.join(CSRC, src)
    if (not force and os.path.exists(obj) and os.path.getmtime(obj) > os.path.getmtime(path)
            and os.path.getmtime(obj) > _newest_header()):
        return obj
    cmd = [_nvcc(), "-std=c++17", "-O3", "-lineinfo", *ARCH, "-Xcompiler", "-fPIC", "-c", path, "-o", obj]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    if trace:
        cmd += ["-DBD_TRACE"]
    if steps:
        cmd += ["-DBD_TRACE_TIMELINE_ONLY", "-DBD_TRACE_STEPS"]
    subprocess.run(cmd, check=True)
    return obj


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not is_stale():
        return LIB
    os.makedirs(OBJ, exist_ok=True)
    with ThreadPoolExecutor(max_workers=len(SOURCES)) as pool:
        objs = list(pool.map(lambda s: _compile(s, force, verbose), SOURCES))
    subprocess.run([_nvcc(), *ARCH, "-shared", "-cudart", "shared", "-o", LIB, *objs], check=True)
    return LIB


def build_trace(steps: bool = False) -> str:
    """The same library with -DBD_TRACE as libbitdelta_trace.so: the 4-bit decode kernel then adds up, per block and
    role, the cycles spent in each kind of wait into a buffer set with bitdelta_debug_set_trace_fp4 (see
    csrc/gemm_fp4.cu).  steps=True (libbitdelta_steps.so): no accumulators, but a time stamp per block, step and event
    behind the first 512 x 32 words of that buffer ([block][step mod 64][16 events]; the buffer must hold them).
    Load either by pointing BITDELTA_LIB at it.  Never the default build: the stamps cost time."""
    os.makedirs(OBJ, exist_ok=True)
    with ThreadPoolExecutor(max_workers=len(SOURCES)) as pool:
        objs = list(pool.map(lambda s: _compile(s, True, False, trace=True, steps=steps), SOURCES))
    lib = os.path.join(HERE, "libbitdelta_steps.so" if steps else "libbitdelta_trace.so")
    subprocess.run([_nvcc(), *ARCH, "-shared", "-cudart", "shared", "-o", lib, *objs], check=True)
    return lib


if __name__ == "__main__":
    if "--trace-steps" in sys.argv:
        print(build_trace(steps=True))
    elif "--trace" in sys.argv:
        print(build_trace())
    else:
        print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
