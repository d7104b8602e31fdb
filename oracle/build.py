"""Build the CPU oracle (test infrastructure) into ``oracle/libsop_oracle.so``.

Plain g++, -O2, no contraction of multiply-add pairs, no fast-math: every float operation in the
source is one IEEE-754 operation.  Nothing here touches the CUDA library.
"""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "sop_oracle.cpp")
LIB = os.path.join(HERE, "libsop_oracle.so")


def build(force: bool = False) -> str:
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= os.path.getmtime(SRC):
        return LIB
    cmd = ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fno-fast-math", "-Wall", "-Wextra",
           "-shared", "-fPIC", SRC, "-o", LIB]
    subprocess.check_call(cmd)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
