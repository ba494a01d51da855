"""Build the CUDA library in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "libwisv.so")
SOURCES = [os.path.join(CSRC, "wisv_api.cu"), os.path.join(CSRC, "wisv_static.cu"),
           os.path.join(CSRC, "wisv_link.cu")]
DEPS = SOURCES + [os.path.join(CSRC, n) for n in ("wisv_gemm.cuh", "wisv_gemm2.cuh", "wisv_aux.cuh", "wisv_ptx.cuh")] + \
    [os.path.join(os.path.dirname(_HERE), "include", "wisv.h")]


def nvcc_command(out: str, verbose: bool = False):
    cmd = ["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-o", out] + SOURCES
    if verbose:
        cmd[1:1] = ["-Xptxas", "-v"]
    return cmd


def up_to_date() -> bool:
    if not os.path.exists(LIB):
        return False
    t = os.path.getmtime(LIB)
    return all(os.path.getmtime(d) <= t for d in DEPS)


def build(force: bool = False, verbose: bool = False) -> str:
    if force or verbose or not up_to_date():
        tmp = LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(nvcc_command(tmp, verbose))
        os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
