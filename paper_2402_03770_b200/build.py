"""Builds libcvlc.so (sm_100a only) in-tree with nvcc.

    python -m paper_2402_03770_b200.build [--force] [--verbose]
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
OUT = os.path.join(HERE, "libcvlc.so")
SOURCES = ["cvlc_api.cu", "cvlc_plan.cu", "cvlc_encode.cu", "cvlc_decode.cu", "cvlc_unframed.cu", "cvlc_profile.cu"]
HEADERS = [os.path.join(CSRC, h) for h in ("cvlc_common.cuh", "cvlc_lookback.cuh", "cvlc_quant.cuh")] + [os.path.join(INCLUDE, "cvlc.h")]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found")


def up_to_date() -> bool:
    if not os.path.exists(OUT):
        return False
    t = os.path.getmtime(OUT)
    deps = [os.path.join(CSRC, s) for s in SOURCES] + HEADERS
    return all(os.path.getmtime(d) <= t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and up_to_date():
        return OUT
    cmd = [
        _nvcc(), "-std=c++17", "-O3", "-lineinfo",
        "-gencode", "arch=compute_100a,code=sm_100a",
        "--fmad=false",                      # planner and quantizer arithmetic is rounded per operation
        "-Xcompiler", "-fPIC,-ffp-contract=off,-Wall",
        "-shared", "-o", OUT,
    ]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, s) for s in SOURCES]
    subprocess.run(cmd, check=True)
    return OUT


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
