"""Builds libecmoe.so (the C-ABI library) from csrc/ with nvcc for sm_100a, in-tree.

Usage: python -m paper_2202_09368_b200.build [--force] [--verbose] [--debug]
Objects go to paper_2202_09368_b200/_build/, the library next to this file.  --debug builds libecmoe_debug.so as well:
the same sources with -DEC_DEBUG, in which every index a kernel reads from I, row_ptr or slots is range-checked.
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OUT = os.path.join(HERE, "libecmoe.so")
OBJ = os.path.join(HERE, "_build")
SOURCES = ["api.cu", "routing.cu", "capped.cu", "gemm_simt.cu", "gemm_tc.cu"]
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
         "-Xcompiler", "-fPIC", "-DECMOE_BUILD"]


def _newer(src_list, target):
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(s) > t for s in src_list)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    out = build_one(force, verbose, OUT, OBJ, [])
    if debug:
        build_one(force, verbose, OUT.replace("libecmoe.so", "libecmoe_debug.so"), os.path.join(OBJ, "debug"), ["-DEC_DEBUG"])
    return out


def build_one(force, verbose, OUT, OBJ, extra) -> str:
    os.makedirs(OBJ, exist_ok=True)
    headers = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))]
    headers.append(os.path.join(os.path.dirname(HERE), "include", "ecmoe.h"))
    objs, procs = [], []
    for s in SOURCES:
        src = os.path.join(CSRC, s)
        obj = os.path.join(OBJ, s.replace(".cu", ".o"))
        objs.append(obj)
        if force or _newer([src] + headers, obj):
            cmd = [NVCC] + FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + ["-c", src, "-o", obj]
            procs.append((s, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    failed = False
    for s, p in procs:
        out, _ = p.communicate()
        if p.returncode != 0 or verbose:
            sys.stderr.write(f"--- {s}\n{out}\n")
        failed |= p.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed")
    if force or procs or _newer(objs, OUT):
        cmd = [NVCC, "-shared", "-o", OUT] + objs + ["-lcudart"]
        subprocess.check_call(cmd)
    return OUT


if __name__ == "__main__":
    print(build("--force" in sys.argv, "--verbose" in sys.argv, "--debug" in sys.argv))
