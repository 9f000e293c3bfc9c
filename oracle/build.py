"""Compile the CPU oracle (plain C) into oracle/libqesgd_ref.so.

Test infrastructure: only the tests, the smoke check and the benchmark's CPU
leg load the result.  Flags keep IEEE semantics: no FMA contraction, no
fast-math, so every operation rounds once in the precision written.
"""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "qesgd_oracle.c")
LIB = os.path.join(HERE, "libqesgd_ref.so")


def build(force: bool = False) -> str:
    if (not force and os.path.exists(LIB)
            and os.path.getmtime(LIB) >= os.path.getmtime(SRC)):
        return LIB
    cmd = ["gcc", "-std=c11", "-O2", "-ffp-contract=off", "-fno-fast-math",
           "-fPIC", "-shared", "-Wall", "-Wextra", "-o", LIB, SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
