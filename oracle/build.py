"""Compile the C oracle into a shared library next to its source.

Test infrastructure only (see pvq_oracle.c).  `python -m oracle.build` or
`build()`; gcc, no CUDA.  -ffp-contract=off keeps every fp32 operation a
single rounding so the oracle's arithmetic is the one its header states.
"""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "pvq_oracle.c")
LIB = os.path.join(HERE, "libpvq_oracle.so")


def build(force: bool = False) -> str:
    if (not force and os.path.exists(LIB)
            and os.path.getmtime(LIB) >= os.path.getmtime(SRC)):
        return LIB
    cmd = ["gcc", "-std=c99", "-O2", "-fPIC", "-shared", "-fopenmp",
           "-ffp-contract=off", "-fno-fast-math", "-Wall", "-Wextra",
           SRC, "-o", LIB, "-lm"]
    subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
