"""Build the fp64 CPU oracle (plain C, OpenMP) into oracle/libssd_oracle.so.

TEST INFRASTRUCTURE: building the checker is allowed anywhere; calling it is reserved to
tests, the smoke check and the bench's CPU-baseline leg.
"""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "ssd_oracle.c")
OUT = os.path.join(HERE, "libssd_oracle.so")


def build(force: bool = False) -> str:
    if (not force and os.path.exists(OUT)
            and os.path.getmtime(OUT) >= os.path.getmtime(SRC)):
        return OUT
    tmp = OUT + ".tmp.%d" % os.getpid()
    # no -ffast-math: the oracle must keep IEEE fp64 semantics and the written order;
    # no -march=native: the built library may be carried to a host with a different CPU
    cmd = ["gcc", "-O3", "-fopenmp", "-fPIC", "-shared",
           "-std=c11", "-Wall", "-o", tmp, SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, OUT)
    return OUT


if __name__ == "__main__":
    print(build(force=True))
