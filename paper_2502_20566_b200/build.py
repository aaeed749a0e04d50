"""Compile the CUDA sources into ``libsradamw.so`` (in-tree, next to this file) for sm_100a.

    python -m paper_2502_20566_b200.build [--force] [--verbose]

nvcc cross-compiles without a GPU.  Flags: IEEE arithmetic throughout (no fast-math, denormals
kept, correctly rounded division and square root); the kernels use explicit rounding intrinsics, so
-fmad has nothing to contract in the update itself.
"""

from __future__ import annotations

import os
import shutil
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libsradamw.so")
SOURCES = ["api.cu", "adamw_kernels.cu", "adamw_flat_bf16.cu", "adamw_flat_f32.cu", "adamw_mt_bf16.cu",
           "adamw_mt_f32.cu", "master_kernels.cu", "fp8_kernels.cu", "accum_kernels.cu", "reduce_kernels.cu", "selftest_kernels.cu"]
HEADERS = ["device_math.cuh", "launch.h", "adamw_body.cuh", "adamw_flat.cuh", "adamw_mt.cuh", os.path.join("..", "..", "include", "sradamw.h")]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-ftz=false", "-prec-div=true", "-prec-sqrt=true",
]


def _nvcc() -> str:
    path = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(path):
        raise RuntimeError("nvcc not found")
    return path


def _stale(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    os.makedirs(OBJ, exist_ok=True)
    headers = [os.path.normpath(os.path.join(CSRC, h)) for h in HEADERS] + [os.path.abspath(__file__)]
    nvcc = _nvcc()
    jobs = []
    objects = []
    for src in SOURCES:
        s = os.path.join(CSRC, src)
        o = os.path.join(OBJ, src.replace(".cu", ".o"))
        objects.append(o)
        if force or _stale(o, [s] + headers):
            cmd = [nvcc, *NVCC_FLAGS, "-c", s, "-o", o]
            if verbose:
                cmd.insert(1, "-Xptxas=-v")
            jobs.append(cmd)

    def run(cmd):
        r = subprocess.run(cmd, capture_output=True, text=True)
        return cmd, r

    with ThreadPoolExecutor(max_workers=max(1, len(jobs))) as pool:
        for cmd, r in pool.map(run, jobs):
            if verbose or r.returncode != 0:
                sys.stderr.write(" ".join(cmd) + "\n" + r.stdout + r.stderr)
            if r.returncode != 0:
                raise RuntimeError("nvcc failed: " + os.path.basename(cmd[-3]))
    if jobs or force or _stale(LIB, objects):
        cmd = [nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", *objects, "-o", LIB]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            sys.stderr.write(r.stdout + r.stderr)
            raise RuntimeError("link failed")
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
