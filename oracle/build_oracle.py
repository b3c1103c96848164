"""Compile the CPU oracle (test infrastructure) into oracle/liboracle_adams.so.

The same C source is compiled twice, once per working precision, and the two
objects are linked into one shared library with two entry points.  Building the
checker is not using it: nothing in the CUDA library links against this.
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "adams_oracle.c")
STATS_SRC = os.path.join(HERE, "mask_stats_oracle.c")
ADAM_SRC = os.path.join(HERE, "plain_adam_oracle.c")
PRUNE_SRC = os.path.join(HERE, "prune_fold_oracle.c")
KD_SRC = os.path.join(HERE, "kd_loss_oracle.c")
LIB = os.path.join(HERE, "liboracle_adams.so")

# No fast-math, no contraction: the fp32 build must perform exactly the
# operations written in the source, in that order.
CFLAGS = ["-O2", "-fPIC", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-Wall", "-Wextra"]


def build(force: bool = False) -> str:
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= max(os.path.getmtime(SRC), os.path.getmtime(STATS_SRC), os.path.getmtime(ADAM_SRC), os.path.getmtime(PRUNE_SRC), os.path.getmtime(KD_SRC)):
        return LIB
    objs = []
    for real, entry in (("double", "oracle_adams_step_f64"), ("float", "oracle_adams_step_f32")):
        obj = os.path.join(HERE, f"adams_oracle_{real}.o")
        subprocess.check_call(["gcc", *CFLAGS, f"-DREAL={real}", f"-DENTRY={entry}", "-c", SRC, "-o", obj])
        objs.append(obj)
    for src in (STATS_SRC, ADAM_SRC, PRUNE_SRC, KD_SRC):
        obj = src[:-2] + ".o"
        subprocess.check_call(["gcc", *CFLAGS, "-c", src, "-o", obj])
        objs.append(obj)
    subprocess.check_call(["gcc", "-shared", "-o", LIB, *objs, "-lm"])
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv))
