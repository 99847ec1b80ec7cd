"""Compile the oracle's C primitives into oracle/libckks_oracle.so.

TEST INFRASTRUCTURE ONLY: the library built here is the CPU reference the CUDA path is checked
against.  -ffp-contract=off keeps gcc from fusing the encoder's multiplies and adds, which the
encoder's bit-exactness contract forbids.
"""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "ckks_prims.c")
LIB = os.path.join(HERE, "libckks_oracle.so")


def build(force: bool = False) -> str:
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= os.path.getmtime(SRC):
        return LIB
    cmd = ["gcc", "-O2", "-std=gnu11", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
           "-shared", "-fPIC", "-o", LIB, SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
