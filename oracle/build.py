"""Compile the CPU oracle (plain C + OpenMP) into oracle/libmarlaas_oracle.so.  Test infrastructure only."""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
LIB = os.path.join(HERE, "libmarlaas_oracle.so")
SRCS = [os.path.join(HERE, "marlaas_oracle.c"), os.path.join(HERE, "marlaas_oracle_impl.inc")]


def build(force: bool = False) -> str:
    if not force and os.path.exists(LIB) and all(os.path.getmtime(LIB) >= os.path.getmtime(s) for s in SRCS):
        return LIB
    cmd = ["gcc", "-O3", "-fopenmp", "-ffp-contract=off", "-fPIC", "-shared", "-std=c11",
           "-o", LIB + ".tmp", SRCS[0], "-lm"]
    subprocess.run(cmd, check=True, cwd=HERE)
    os.replace(LIB + ".tmp", LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
