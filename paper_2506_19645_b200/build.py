"""Builds libcaat.so (the C-ABI library) in-tree with nvcc for sm_100a.

Run as ``python -m paper_2506_19645_b200.build``; cross-compiles without a GPU.  Every
translation unit is compiled to an object file of its own (in parallel, and only when it or a
header changed), then the objects are linked into the shared library.
"""
from __future__ import annotations

import os
import shlex
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
OBJ = os.path.join(PKG, "build")
LIB = os.path.join(PKG, "libcaat.so")
SOURCES = ["caat_api.cu", "caat_rows.cu", "caat_rows_staged.cu", "caat_rows_lean.cu", "caat_rows_warp.cu", "caat_gemm_simt.cu",
           "caat_gemm_tc.cu", "caat_static.cu", "caat_colpar.cu", "caat_tp_push.cu"]
ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]


def _headers_mtime() -> float:
    files = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))]
    files.append(os.path.join(ROOT, "include", "caat.h"))
    files.append(os.path.abspath(__file__))
    return max(os.path.getmtime(f) for f in files)


def _compile(nvcc: str, src: str, obj: str, verbose: bool) -> str:
    # CAAT_NVCC_EXTRA: extra compiler flags, e.g. -DCAAT_MEASUREMENT_AIDS for a build with the ablation switches
    cmd = [nvcc, *ARCH, "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC", "-rdc=false",
           *shlex.split(os.environ.get("CAAT_NVCC_EXTRA", "")),
           "-I", os.path.join(ROOT, "include"), "-I", CSRC, "-c", src, "-o", obj]
    if verbose:
        cmd[1:1] = ["-Xptxas", "-v"]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError(f"nvcc failed on {os.path.basename(src)}:\n{r.stdout}{r.stderr}")
    return r.stderr


def build(force: bool = False, verbose: bool = False) -> str:
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    os.makedirs(OBJ, exist_ok=True)
    hdr = _headers_mtime()
    jobs, objs = [], []
    for s in SOURCES:
        src, obj = os.path.join(CSRC, s), os.path.join(OBJ, s[:-3] + ".o")
        objs.append(obj)
        if force or verbose or not os.path.exists(obj) or os.path.getmtime(obj) < max(hdr, os.path.getmtime(src)):
            jobs.append((src, obj))
    if jobs:
        with ThreadPoolExecutor(max_workers=min(len(jobs), os.cpu_count() or 4)) as ex:
            logs = list(ex.map(lambda j: _compile(nvcc, j[0], j[1], verbose), jobs))
        if verbose:
            sys.stderr.write("".join(logs))
    if jobs or not os.path.exists(LIB) or os.path.getmtime(LIB) < max(os.path.getmtime(o) for o in objs):
        r = subprocess.run([nvcc, *ARCH, "-shared", "-o", LIB, *objs], capture_output=True, text=True)
        if r.returncode != 0:
            sys.stderr.write(r.stdout + r.stderr)
            raise RuntimeError("nvcc failed linking libcaat.so")
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
