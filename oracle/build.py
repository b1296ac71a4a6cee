"""Compile the oracle (test infrastructure) with gcc: one shared object per arithmetic type.

    python oracle/build.py        -> oracle/libkvo_f32.so, oracle/libkvo_f64.so
"""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "kvo.c")
TARGETS = {"f32": "float", "f64": "double"}


def lib_path(kind: str) -> str:
    return os.path.join(HERE, f"libkvo_{kind}.so")


def build(force: bool = False) -> None:
    for kind, ctype in TARGETS.items():
        out = lib_path(kind)
        if not force and os.path.exists(out) and os.path.getmtime(out) >= os.path.getmtime(SRC):
            continue
        # -O2, no fast-math, no FMA contraction: sums are taken exactly in the order written
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               f"-DKVO_REAL={ctype}", "-o", out, SRC, "-lm"]
        subprocess.run(cmd, check=True)


if __name__ == "__main__":
    build(force="--force" in sys.argv)
    print("built", [lib_path(k) for k in TARGETS])
