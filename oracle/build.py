"""Compile the C oracle into oracle/liblpmm_oracle.so (test infrastructure, not the product).

Flags matter for the arithmetic contract: -ffp-contract=off keeps every binary32 operation
separately rounded (no fused multiply-add), and no fast-math option is given, so divisions and
square roots are IEEE and denormals are kept.
"""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "lpmm_oracle.c")
HDR = os.path.join(HERE, "lpmm_oracle.h")
LIB = os.path.join(HERE, "liblpmm_oracle.so")

CFLAGS = ["-O2", "-std=c99", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
          "-shared", "-fPIC", "-Wall", "-Wextra"]


def build(force: bool = False) -> str:
    newest_src = max(os.path.getmtime(SRC), os.path.getmtime(HDR))
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= newest_src:
        return LIB
    cmd = ["gcc", *CFLAGS, "-o", LIB, SRC, "-lm"]
    subprocess.run(cmd, check=True, cwd=HERE)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv))
