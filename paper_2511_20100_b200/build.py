"""Builds libmtmcfused.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import shutil
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "libmtmcfused.so")
SOURCES = ["api.cu"]
HEADERS = ["ptx.cuh", "gemm_tiled.cuh", "gemm_pair.cuh", "gemm_ksplit.cuh", "gemm_big.cuh", "skinny.cuh", "gemm_mx.cuh", "gemm_mx_pair.cuh"]


def _nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found: libmtmcfused cannot be built")
    return exe


# Build variants: "" the product; "trace" adds device-side time stamps and stall counters (-DMTMC_TRACE) and
# "checks" index checks that report through the status word instead of faulting (-DMTMC_CHECKS).  Each variant
# is a library of its own beside the product (libmtmcfused_<variant>.so), selected with MTMC_LIB_VARIANT.
VARIANT_FLAGS = {"": [], "trace": ["-DMTMC_TRACE"], "checks": ["-DMTMC_CHECKS"]}


def lib_path(variant: str = "") -> str:
    return os.path.join(_HERE, "libmtmcfused%s.so" % ("_" + variant if variant else ""))


def needs_build(variant: str = "") -> bool:
    lib = lib_path(variant)
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS]
    deps.append(os.path.join(os.path.dirname(_HERE), "include", "mtmc_fused.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, variant: str = "") -> str:
    lib = lib_path(variant)
    if not force and not needs_build(variant):
        return lib
    tmp = lib + ".tmp.%d" % os.getpid()
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-o", tmp]
    cmd += VARIANT_FLAGS[variant]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, f) for f in SOURCES]
    subprocess.check_call(cmd)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    import sys
    variants = [a for a in sys.argv[1:] if a in VARIANT_FLAGS] or [""]
    for v in variants:
        print(build(force=True, verbose="-v" in sys.argv, variant=v))
