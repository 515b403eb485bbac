"""Builds the C-ABI library ``libmnnllm_b200.so`` in-tree with nvcc for sm_100a.

    python -m paper_2506_10443_b200.build [--force] [--verbose]

nvcc cross-compiles without a GPU.  The shared object sits next to this file so that it travels
with the source tree; it is not installed anywhere else.
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libmnnllm_b200.so")

SOURCES = [
    "pack_host.cpp",
    "api_w4a16.cu",
    "gemv_w4a16.cu",
    "gemv_w8a16.cu",
    "stack_w4a16.cu",
    "api_stack.cu",
    "act_quant.cu",
    "gemm_w4a8.cu",
    "gemm_w8a8.cu",
    "attn_decode.cu",
    "api_attn.cu",
    "api_w8a8.cu",
    "gemm_small_w4a8.cu",
    "gemm_limb_w4a8.cu",
    "api_w4a8.cu",
    "bench_mma_i8.cu",
]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC,-fopenmp,-ffp-contract=off",
    "--expt-relaxed-constexpr",
]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [
        os.path.join(os.path.dirname(HERE), "include", "mnnllm.h"), os.path.abspath(__file__)]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not _stale():
        return LIB
    objdir = os.path.join(HERE, "_build")
    os.makedirs(objdir, exist_ok=True)
    objs = []
    procs = []
    for src in SOURCES:
        path = os.path.join(CSRC, src)
        if not os.path.exists(path):
            raise FileNotFoundError(path)
        obj = os.path.join(objdir, os.path.splitext(src)[0] + ".o")
        cmd = ["nvcc", *NVCC_FLAGS, "-x", "cu", "-c", path, "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas=-v")
            print(" ".join(cmd), flush=True)
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
        objs.append(obj)
    failed = False
    for src, p in procs:
        out, _ = p.communicate()
        if p.returncode != 0 or verbose:
            sys.stderr.write("---- %s ----\n%s\n" % (src, out))
        failed |= p.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed")
    tmp = LIB + ".tmp%d" % os.getpid()
    subprocess.check_call(["nvcc", "-arch=sm_100a", "-shared", "-o", tmp, *objs, "-Xcompiler", "-fopenmp", "-lgomp"])
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
