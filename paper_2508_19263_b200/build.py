"""Builds libzc.so (host logic + sm_100a kernels) in-tree with nvcc.

Every source is compiled to an object file of its own (the decoder's to one per element format; in parallel, and
only when it or a header is newer than its object), then the objects are linked into the shared library.
"""
from __future__ import annotations

import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
LIB = os.path.join(HERE, "libzc.so")
OBJDIR = os.path.join(HERE, "build")
SOURCES = ["zc_host.cpp", "zc_hist.cu", "zc_encode.cu", "zc_decode.cu"]
# (source, extra flags, object name): the decoder's kernels are compiled one element format per object (ZC_DEC_PART),
# so that the longest compile of the build runs four ways in parallel
UNITS = [("zc_host.cpp", [], "zc_host.cpp.o"), ("zc_hist.cu", [], "zc_hist.cu.o"), ("zc_encode.cu", [], "zc_encode.cu.o")] + \
        [("zc_decode.cu", [f"-DZC_DEC_PART={k}"], f"zc_decode.part{k}.o") for k in (1, 2, 3, 4)]
HEADERS = ["zc_internal.h", "zc_bits.cuh", "zc_device.cuh", "zc_encode_rows.cuh"]
ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def _header_time() -> float:
    deps = [os.path.join(CSRC, f) for f in HEADERS]
    deps += [os.path.join(INCLUDE, f) for f in os.listdir(INCLUDE)]
    return max(os.path.getmtime(d) for d in deps)


def is_stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return _header_time() > t or any(os.path.getmtime(os.path.join(CSRC, f)) > t for f in SOURCES)


def extra_flags() -> list:
    """Extra compiler flags from the environment (ZC_NVCC_FLAGS, space separated), e.g. -DZC_DEBUG_CHECKS=1."""
    return os.environ.get("ZC_NVCC_FLAGS", "").split()


def build_library(force: bool = False, verbose: bool = False, lib: str = LIB, flags=None, objdir: str = OBJDIR) -> str:
    """Compile for sm_100a only.  Returns the path of the shared object."""
    flags = extra_flags() if flags is None else list(flags)
    if lib == LIB and not flags and not force and not is_stale():
        return lib
    os.makedirs(objdir, exist_ok=True)
    stamp = os.path.join(objdir, "flags.txt")
    old_flags = open(stamp).read() if os.path.exists(stamp) else None
    if old_flags != " ".join(flags):
        force = True
    hdr_t = _header_time()
    common = [_nvcc(), *ARCH, "-lineinfo", "-O3", "-std=c++17", "-I", INCLUDE, "-Xcompiler", "-fPIC,-pthread", *flags]
    if verbose:
        common += ["-Xptxas", "-v"]

    def compile_one(unit) -> str:
        src, unit_flags, name = unit
        path = os.path.join(CSRC, src)
        obj = os.path.join(objdir, name)
        if force or not os.path.exists(obj) or os.path.getmtime(obj) < max(os.path.getmtime(path), hdr_t):
            tmp = obj + f".tmp{os.getpid()}"
            subprocess.check_call(common + unit_flags + ["-c", path, "-o", tmp])
            os.replace(tmp, obj)
        return obj

    with ThreadPoolExecutor(max_workers=len(UNITS)) as pool:
        objs = list(pool.map(compile_one, UNITS))
    with open(stamp, "w") as f:
        f.write(" ".join(flags))
    tmp = lib + f".tmp{os.getpid()}"
    subprocess.check_call([_nvcc(), *ARCH, "-shared", "-Xcompiler", "-fPIC,-pthread", "-o", tmp] + objs)
    os.replace(tmp, lib)
    return lib


DEBUG_LIB = os.path.join(HERE, "libzc_debug.so")


def build_debug_library(force: bool = False) -> str:
    """The development build: the same sources with -DZC_DEBUG_CHECKS=1 (in-kernel checks of every access the
    kernels' load/store helpers make), as libzc_debug.so with objects of its own; ptxas at -O1, so that it builds
    in a fraction of the library's time (its speed does not matter).  Tests only."""
    if not force and os.path.exists(DEBUG_LIB):
        t = os.path.getmtime(DEBUG_LIB)
        if _header_time() <= t and all(os.path.getmtime(os.path.join(CSRC, f)) <= t for f in SOURCES):
            return DEBUG_LIB
    return build_library(force=force, lib=DEBUG_LIB, flags=["-DZC_DEBUG_CHECKS=1", "-Xptxas", "-O1"], objdir=OBJDIR + "_debug")


if __name__ == "__main__":
    print(build_library(force=True, verbose=True))
