"""Compile the CUDA library in-tree: paper_2509_25996_b200/libcast_adams.so (sm_100a only).

nvcc cross-compiles without a GPU.  The CUDA runtime is linked statically, so the
library loads on a machine without a driver (calls then return CAST_ERR_CUDA).

Every .cu file becomes one object; csrc/step_inst.cu, which instantiates the step kernels,
is compiled once per slice (group size M, 2:4 or general N:M, with or without the statistics
epilogue, literal or alternate reading of Eq. 8) so that the few hundred instantiations compile in parallel.  Objects live in
paper_2509_25996_b200/_build/ and are rebuilt only when a source or header is newer.
"""
from __future__ import annotations

import glob
import os
import shutil
import subprocess
import sys
import time
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ_DIR = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libcast_adams.so")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")

NVCC_FLAGS = [
    "-O3", "-std=c++17",
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-lineinfo",
    "-Xcompiler", "-fPIC,-fvisibility=hidden",
]
LINK_FLAGS = ["--cudart", "static", "-shared", "-gencode", "arch=compute_100a,code=sm_100a"]

# slices of the step kernels: (M, two_four, statistics, alternate reading of Eq. 8); 2:4 exists for M = 4 only
STEP_SLICES = [(m, tf, s, v) for m in (2, 4, 8, 16, 32) for tf in ((0, 1) if m == 4 else (0,)) for s in (0, 1) for v in (0, 1)]


def _nvcc() -> str:
    for cand in (shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: the CUDA library cannot be built")


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _headers():
    return glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(CSRC, "*.h")) + \
        glob.glob(os.path.join(INCLUDE, "*.h")) + [os.path.abspath(__file__)]


def _jobs():
    """(object path, source, extra defines) of every object of the library."""
    jobs = []
    for src in sources():
        base = os.path.splitext(os.path.basename(src))[0]
        if base == "step_inst":
            for m, tf, s, v in STEP_SLICES:
                jobs.append((os.path.join(OBJ_DIR, f"step_inst_m{m}_tf{tf}_s{s}_v{v}.o"), src,
                             [f"-DCAST_INST_M={m}", f"-DCAST_INST_TF={tf}", f"-DCAST_INST_STATS={s}", f"-DCAST_INST_V={v}"]))
        else:
            jobs.append((os.path.join(OBJ_DIR, base + ".o"), src, []))
    return jobs


def build(force: bool = False, verbose: bool = False) -> str:
    jobs = _jobs()
    newest_header = max(os.path.getmtime(p) for p in _headers())
    stale = [j for j in jobs if force or not os.path.exists(j[0]) or
             os.path.getmtime(j[0]) < max(newest_header, os.path.getmtime(j[1]))]
    if not stale and os.path.exists(LIB) and os.path.getmtime(LIB) >= max(os.path.getmtime(j[0]) for j in jobs):
        return LIB
    os.makedirs(OBJ_DIR, exist_ok=True)
    nvcc = _nvcc()

    def compile_one(job):
        obj, src, defines = job
        cmd = [nvcc, *NVCC_FLAGS, *defines, "-I", INCLUDE, "-c", src, "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas=-v")
        res = subprocess.run(cmd, capture_output=True, text=True)
        return job, res

    t0 = time.time()
    workers = max(1, min(len(stale), os.cpu_count() or 1))
    # the largest slices first, so that the pool drains evenly
    stale.sort(key=lambda j: ("_tf1_" not in j[0], "step_inst" not in j[0]))
    with ThreadPoolExecutor(max_workers=workers) as ex:
        for (obj, src, defines), res in ex.map(compile_one, stale):
            if verbose:
                print(f"== {os.path.basename(obj)}\n{res.stderr}")
            if res.returncode != 0:
                raise RuntimeError(f"nvcc failed on {src} {' '.join(defines)}:\n" + res.stdout + res.stderr)
    res = subprocess.run([nvcc, *LINK_FLAGS, "-o", LIB, *[j[0] for j in jobs]], capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("link failed:\n" + res.stdout + res.stderr)
    if verbose:
        print(f"built {len(stale)} objects in {time.time() - t0:.1f} s; {os.path.getsize(LIB) / 1e6:.1f} MB")
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
