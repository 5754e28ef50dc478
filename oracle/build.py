"""Compile the C part of the CPU oracle (test infrastructure) with gcc.

`python -m oracle.build` writes `oracle/libnsd_oracle.so` next to the source.
Floating-point contraction is switched off so that the only fused operation is the
explicit `fmaf` the quantizer's definition asks for.
"""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "nsd_oracle.c")
LIB = os.path.join(HERE, "libnsd_oracle.so")


def build(force: bool = False) -> str:
    if (not force and os.path.exists(LIB)
            and os.path.getmtime(LIB) >= os.path.getmtime(SRC)):
        return LIB
    cmd = ["gcc", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
           "-o", LIB, SRC, "-lm"]
    subprocess.check_call(cmd)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv))
