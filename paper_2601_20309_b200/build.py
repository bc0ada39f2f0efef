"""Compile the CUDA library for sm_100a with nvcc, in-tree.

``build()`` produces ``paper_2601_20309_b200/libduplexkv.so`` from ``csrc/duplexkv.cu``
(kernels in ``csrc/kv_kernels.cuh``) and ``csrc/kv_table.cu`` (block table, host code) and ``libkvtestutil.so`` from ``csrc/kv_testutil.cu``
(pool fill / checksum helpers used by tests and the bench to make and check inputs; not
part of the rotation path).  nvcc cross-compiles without a GPU.
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libduplexkv.so")
TESTUTIL_LIB = os.path.join(HERE, "libkvtestutil.so")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-shared"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def _stale(target: str, sources) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(s) > t for s in sources)


def build(force: bool = False, verbose: bool = False) -> str:
    # (target, files to compile, further files the target depends on)
    main_src = [os.path.join(CSRC, "duplexkv.cu"), os.path.join(CSRC, "kv_table.cu")]
    main_dep = [os.path.join(CSRC, "kv_kernels.cuh"), os.path.join(os.path.dirname(HERE), "include", "duplexkv.h")]
    jobs = [(LIB, main_src, main_dep)]
    util_src = os.path.join(CSRC, "kv_testutil.cu")
    if os.path.exists(util_src):
        jobs.append((TESTUTIL_LIB, [util_src], [os.path.join(CSRC, "kv_kernels.cuh")]))
    for target, sources, deps in jobs:
        if not force and not _stale(target, sources + deps):
            continue
        cmd = [_nvcc()] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-o", target] + sources
        res = subprocess.run(cmd, capture_output=True, text=True)
        if verbose:
            sys.stderr.write(res.stderr)
        if res.returncode != 0:
            raise RuntimeError("nvcc failed:\n" + " ".join(cmd) + "\n" + res.stdout + res.stderr)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
