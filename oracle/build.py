"""Compile the C oracle into oracle/libha_oracle.so (test infrastructure, not the product).

Flags: -O2 with hardware FMA enabled so that fmaf() is one instruction, and with floating-point
contraction switched off so that the compiler fuses nothing on its own; the arithmetic is then
exactly the sequence of operations written in ha_oracle.c.
"""
from __future__ import annotations

import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "ha_oracle.c")
LIB = os.path.join(HERE, "libha_oracle.so")


def build(force: bool = False) -> str:
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= os.path.getmtime(SRC):
        return LIB
    cmd = ["gcc", "-std=c11", "-O2", "-mavx2", "-mfma", "-ffp-contract=off", "-fno-fast-math",
           "-fopenmp", "-shared", "-fPIC", "-o", LIB, SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
