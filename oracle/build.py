"""Builds the CPU oracle (test infrastructure) into oracle/libcvlc_oracle.so.

Flags matter: -ffp-contract=off keeps every multiply and add separately rounded,
which the oracle's bit-exact planner arithmetic relies on.
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "cvlc_oracle.c")
HDR = os.path.join(HERE, "cvlc_oracle.h")
OUT = os.path.join(HERE, "libcvlc_oracle.so")


def build(force: bool = False) -> str:
    if not force and os.path.exists(OUT):
        newest = max(os.path.getmtime(SRC), os.path.getmtime(HDR))
        if os.path.getmtime(OUT) >= newest:
            return OUT
    cmd = ["gcc", "-std=c11", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
           "-Wall", "-Wextra", "-o", OUT, SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return OUT


if __name__ == "__main__":
    print(build(force="--force" in sys.argv))
