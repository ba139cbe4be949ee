"""Builds libgaconv.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

Each .cu file is compiled to an object on its own (in parallel) and the objects are linked into the
shared library; objects newer than their sources and headers are reused.  Setting GACONV_TUNING=1 in
the environment builds the tuning variant (planner overrides from the environment, phase time stamps)."""
from __future__ import annotations

import glob
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libgaconv.so")
OBJ = os.path.join(PKG, "build")


def sources() -> list[str]:
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def headers() -> list[str]:
    return glob.glob(os.path.join(CSRC, "*.h")) + glob.glob(os.path.join(CSRC, "*.cuh")) \
        + glob.glob(os.path.join(ROOT, "include", "*.h"))


def _flags(verbose: bool = False) -> list[str]:
    flags = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo", "-Xcompiler", "-fPIC",
             "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    if os.environ.get("GACONV_TUNING", "") not in ("", "0"):
        flags.append("-DGACONV_TUNING")
    if verbose:
        flags.append("-Xptxas=-v")
    return flags


def _flags_tag() -> str:
    return os.path.join(OBJ, "flags.txt")


def stale() -> bool:
    """True when the library is missing or older than a source or header.  (Which variant the existing library is
    -- default or tuning -- is not checked here: a library shipped to a machine is used as it is.)"""
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(d) > t for d in sources() + headers())


def build(force: bool = False, verbose: bool = False) -> str:
    flags = _flags(verbose)
    tag = _flags_tag()
    same_flags = os.path.exists(tag) and open(tag).read() == " ".join(flags)
    explicit_variant = "GACONV_TUNING" in os.environ          # the caller asked for a variant: rebuild if it differs
    if not force and not stale() and (same_flags or not explicit_variant):
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    os.makedirs(OBJ, exist_ok=True)
    hdr_time = max(os.path.getmtime(h) for h in headers())

    def compile_one(src: str) -> str:
        obj = os.path.join(OBJ, os.path.basename(src)[:-3] + ".o")
        fresh = same_flags and not force and os.path.exists(obj) and os.path.getmtime(obj) > max(os.path.getmtime(src), hdr_time)
        if not fresh:
            subprocess.check_call([nvcc] + flags + ["-c", "-o", obj, src])
        return obj

    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as pool:
        objs = list(pool.map(compile_one, sources()))
    open(tag, "w").write(" ".join(flags))
    tmp = LIB + ".tmp.%d" % os.getpid()
    subprocess.check_call([nvcc, "-shared", "-o", tmp] + objs)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
