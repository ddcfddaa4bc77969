"""Builds the CPU oracle (test infrastructure) into oracle/libdblp_oracle.so with gcc.

Flags: -O2 for a fair timed baseline, -ffp-contract=off so that no fused multiply-add can
replace the plain fp32 additions the definition asks for, -fopenmp for the one pragma in the reduce.
"""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "dblp_oracle.c")
OUT = os.path.join(HERE, "libdblp_oracle.so")


def build(force: bool = False) -> str:
    if not force and os.path.exists(OUT) and os.path.getmtime(OUT) >= os.path.getmtime(SRC):
        return OUT
    cmd = ["gcc", "-std=c99", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-fPIC", "-shared",
           "-Wall", "-Wextra", "-o", OUT, SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return OUT


if __name__ == "__main__":
    print(build(force=True))
