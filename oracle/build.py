"""Compile the CPU oracle (test infrastructure) into oracle/libnvfp4_oracle.so.

Plain g++; -ffp-contract=off keeps every fp32 operation a single IEEE rounding,
which the bit-exact parity tests rely on.
"""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "nvfp4_oracle.cpp")
OUT = os.path.join(HERE, "libnvfp4_oracle.so")


def build(force: bool = False) -> str:
    deps = [SRC, os.path.join(HERE, "nvfp4_oracle.h")]
    if (not force and os.path.exists(OUT)
            and all(os.path.getmtime(OUT) >= os.path.getmtime(d) for d in deps)):
        return OUT
    cmd = ["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
           "-pthread", "-Wall", "-Wextra", "-o", OUT, SRC]
    subprocess.check_call(cmd)
    return OUT


if __name__ == "__main__":
    print(build(force="--force" in sys.argv))
