"""Builds ``libfedhe.so`` (the C-ABI CUDA library) in-tree for sm_100a.

Run as ``python paper_2303_10837_b200/build.py`` (a plain script: importing the package
needs the library this script produces).  nvcc cross-compiles without a
GPU; the host-only table code is compiled by g++ because it uses libquadmath.
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OUT = os.path.join(HERE, "libfedhe.so")
BUILD = os.path.join(HERE, "_build")

CUDA_SOURCES = ["fedhe_transform.cu", "fedhe_slots.cu", "fedhe_encrypt.cu", "fedhe_server.cu", "fedhe_decrypt.cu",
                "fedhe_mask.cu", "fedhe_api.cu", "fedhe_noalloc.cu"]
HOST_SOURCES = ["fedhe_host.cpp"]
HEADERS = ["fedhe_device.cuh", "fedhe_ntt.cuh", "fedhe_internal.cuh", "fedhe_launch.h", "fedhe_host.h",
           "fedhe_kernels.cuh", "fedhe_slots.cuh",
           os.path.join("..", "..", "include", "fedhe.h")]

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-Xptxas", "-v", "--expt-relaxed-constexpr"]


def _nvcc() -> str:
    for cand in (shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found")


def _stale(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    os.makedirs(BUILD, exist_ok=True)
    headers = [os.path.join(CSRC, h) for h in HEADERS] + [os.path.abspath(__file__)]
    objs = []

    def compile_cuda(src):
        s = os.path.join(CSRC, src)
        o = os.path.join(BUILD, src + ".o")
        if force or _stale(o, [s] + headers):
            cmd = [_nvcc()] + NVCC_FLAGS + ["-c", s, "-o", o]
            r = subprocess.run(cmd, capture_output=True, text=True)
            with open(os.path.join(BUILD, src + ".log"), "w") as f:
                f.write(r.stdout + r.stderr)
            if verbose or r.returncode:
                sys.stderr.write(r.stdout + r.stderr)
            if r.returncode:
                raise RuntimeError("nvcc failed on " + src)
        return o

    # the translation units are independent: compile them side by side
    with ThreadPoolExecutor(max_workers=min(len(CUDA_SOURCES), os.cpu_count() or 1)) as pool:
        objs.extend(pool.map(compile_cuda, CUDA_SOURCES))
    for src in HOST_SOURCES:
        s = os.path.join(CSRC, src)
        o = os.path.join(BUILD, src + ".o")
        if force or _stale(o, [s] + headers):
            subprocess.run(["g++", "-O2", "-std=c++17", "-fPIC", "-c", s, "-o", o], check=True)
        objs.append(o)
    if force or _stale(OUT, objs):
        tmp = OUT + ".tmp.%d" % os.getpid()
        subprocess.run([_nvcc(), "-shared", "-o", tmp] + objs + ["-lquadmath"], check=True)
        os.replace(tmp, OUT)
    tool_src = os.path.join(CSRC, "int_pipe_bench.cu")
    tool = os.path.join(HERE, "int_pipe_bench")
    if force or _stale(tool, [tool_src]):
        subprocess.run([_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-o", tool, tool_src],
                       check=True, capture_output=True)
    return OUT


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose=True))
