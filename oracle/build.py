"""Compile the C oracle into oracle/libufp4_oracle.so (test infrastructure; gcc only, no CUDA)."""
import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(_HERE, "ufp4_oracle.c")
LIB = os.path.join(_HERE, "libufp4_oracle.so")

# -ffp-contract=off: no fused multiply-add may replace the separately rounded FP32 operations the quantizer's
# definition fixes.  No -ffast-math, no -march: plain IEEE single/double arithmetic.
FLAGS = ["-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC", "-Wall", "-Wextra"]


def build(force: bool = False) -> str:
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= os.path.getmtime(SRC):
        return LIB
    tmp = LIB + ".tmp.%d" % os.getpid()
    subprocess.check_call(["gcc", *FLAGS, "-o", tmp, SRC, "-lm"])
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
