"""Compile the C oracle into ``oracle/libkvbfp_oracle.so`` with gcc.

Building the checker is not using it: the CUDA library neither links nor loads
this file.
"""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "kvbfp_oracle.c")
HDR = os.path.join(HERE, "kvbfp_oracle.h")
LIB = os.path.join(HERE, "libkvbfp_oracle.so")


def build(force: bool = False) -> str:
    newest_src = max(os.path.getmtime(SRC), os.path.getmtime(HDR))
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= newest_src:
        return LIB
    cmd = ["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-fno-fast-math", "-ffp-contract=off",
           "-Wall", "-Wextra", "-o", LIB, SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
