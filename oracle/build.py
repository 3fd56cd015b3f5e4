"""Compile the oracle's C loops into oracle/liboracle_conv.so with gcc (test infrastructure only)."""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "conv_loops.c")
LIB = os.path.join(HERE, "liboracle_conv.so")


def build(force: bool = False) -> str:
    if (not force and os.path.exists(LIB)
            and os.path.getmtime(LIB) >= os.path.getmtime(SRC)):
        return LIB
    # No -ffast-math (keeps IEEE semantics) and no -march=native (the library may be
    # built on one machine and run on another).
    cmd = ["gcc", "-O3", "-fopenmp", "-shared", "-fPIC", "-std=c11", SRC, "-o", LIB, "-lm"]
    subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
