"""Compile the CPU oracle (plain C++17, no CUDA) into oracle/libccl_oracle.so.

Test infrastructure: building the checker is not using it.  Run as
``python -m oracle.build`` or call :func:`build`.
"""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "ccl_oracle.cpp")
LIB = os.path.join(HERE, "libccl_oracle.so")


def build(force: bool = False) -> str:
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= os.path.getmtime(SRC):
        return LIB
    # Baseline x86-64 code only: the library is built on one machine and may run on another.
    cmd = ["g++", "-O2", "-std=c++17", "-shared", "-fPIC", "-pthread", "-Wall", "-Wextra",
           "-ffp-contract=off", "-o", LIB, SRC]
    subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
