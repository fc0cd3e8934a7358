"""Compile the C part of the oracle (test infrastructure only) with gcc.

Usage: ``python -m oracle.build``.  Produces ``oracle/libssm_oracle.so`` beside
the source.  Plain ``-O2``: no fast-math, so the summation order is the one the
source states.
"""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "ssm_recurrence.c")
OUT = os.path.join(HERE, "libssm_oracle.so")


def build(force: bool = False) -> str:
    if (not force and os.path.exists(OUT)
            and os.path.getmtime(OUT) >= os.path.getmtime(SRC)):
        return OUT
    cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-o", OUT, SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return OUT


if __name__ == "__main__":
    print(build(force=True))
