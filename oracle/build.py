"""Compile the CPU oracle (plain C, gcc) into oracle/libslowmo_oracle.so.

TEST INFRASTRUCTURE: the oracle checks the CUDA library; nothing in the CUDA path uses it.
slowmo_oracle.c is compiled twice (binary32 and binary64 arithmetic) and linked with the
noise generator into one shared object. Floating-point contraction is switched off so that
the only fused operations are the fma calls the source spells out.
"""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
LIB = os.path.join(HERE, "libslowmo_oracle.so")
SOURCES = ["slowmo_oracle.c", "slowmo_noise.c", "slowmo_oracle.h"]
CFLAGS = ["-O2", "-std=c11", "-fPIC", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
          "-Wall", "-Wextra", "-D_GNU_SOURCE"]


def needs_build():
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(os.path.join(HERE, s)) > t for s in SOURCES + ["build.py"])


def build(force=False):
    if not force and not needs_build():
        return LIB
    objs = []
    for name, defs in (("slowmo_noise", []), ("slowmo_oracle_f32", ["-DORACLE_F64=0"]),
                       ("slowmo_oracle_f64", ["-DORACLE_F64=1"])):
        src = "slowmo_noise.c" if name == "slowmo_noise" else "slowmo_oracle.c"
        obj = os.path.join(HERE, name + ".o")
        subprocess.check_call(["gcc", *CFLAGS, *defs, "-c", os.path.join(HERE, src), "-o", obj])
        objs.append(obj)
    subprocess.check_call(["gcc", "-shared", "-fopenmp", "-o", LIB, *objs, "-lm"])
    for o in objs:
        os.remove(o)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv))
