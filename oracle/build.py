"""Compile the C++ oracle into oracle/libqgx_oracle.so with the host compiler.

Test infrastructure only.  Flags: IEEE arithmetic as written (no FMA contraction, no
fast-math), so that every fp32 operation in the source is one rounding.
"""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "qgx_oracle.cpp")
LIB = os.path.join(HERE, "libqgx_oracle.so")


def build(force: bool = False) -> str:
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= os.path.getmtime(SRC):
        return LIB
    tmp = "%s.%d.tmp" % (LIB, os.getpid())
    cmd = ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
           "-Wall", "-Wextra", "-o", tmp, SRC]
    subprocess.run(cmd, check=True)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
