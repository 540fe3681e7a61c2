"""Build the CUDA library in-tree: csrc/*.cu, csrc/*.cpp -> libspmm_b200.so (sm_100a only).

Usage: ``python -m paper_2604_17834_b200.build [--force] [--verbose]``
nvcc cross-compiles without a GPU.  Objects are cached under csrc/build/ and
rebuilt when a source or header is newer.
"""
from __future__ import annotations

import concurrent.futures
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
OUT = os.path.join(HERE, "libspmm_b200.so")
OBJDIR = os.path.join(CSRC, "build")
SOURCES = ["api.cu", "bcsr_kernel.cu", "wcsr_kernel.cu", "format_gpu.cu", "format.cpp"]
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-I", INCLUDE, "-I", CSRC,
]


def _newest_header():
    t = 0.0
    for d in (CSRC, INCLUDE):
        for f in os.listdir(d):
            if f.endswith((".h", ".cuh")):
                t = max(t, os.path.getmtime(os.path.join(d, f)))
    return t


def _compile(src, force, verbose):
    obj = os.path.join(OBJDIR, os.path.splitext(src)[0] + ".o")
    path = os.path.join(CSRC, src)
    if (not force and os.path.exists(obj)
            and os.path.getmtime(obj) >= max(os.path.getmtime(path), _newest_header())):
        return obj, ""
    cmd = [NVCC] + FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-c", path, "-o", obj]
    if src.endswith(".cpp"):
        cmd = [NVCC] + FLAGS + ["-x", "cu", "-c", path, "-o", obj]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError("nvcc failed for %s:\n%s\n%s" % (src, r.stdout, r.stderr))
    return obj, r.stderr


def build(force: bool = False, verbose: bool = False) -> str:
    os.makedirs(OBJDIR, exist_ok=True)
    with concurrent.futures.ThreadPoolExecutor(max_workers=len(SOURCES)) as ex:
        results = list(ex.map(lambda s: _compile(s, force, verbose), SOURCES))
    objs = [o for o, _ in results]
    if verbose:
        for _, log in results:
            if log:
                print(log)
    if force or not os.path.exists(OUT) or any(os.path.getmtime(o) > os.path.getmtime(OUT) for o in objs):
        tmp = OUT + ".tmp%d" % os.getpid()
        cmd = [NVCC, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", tmp] + objs
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError("link failed:\n%s\n%s" % (r.stdout, r.stderr))
        os.replace(tmp, OUT)
    return OUT


UBENCH_OUT = os.path.join(HERE, "spmm_ubench")


def build_ubench(force: bool = False) -> str:
    """The machine-constant microbenchmarks (csrc/ubench.cu), a stand-alone program."""
    src = os.path.join(CSRC, "ubench.cu")
    if (force or not os.path.exists(UBENCH_OUT)
            or os.path.getmtime(UBENCH_OUT) < max(os.path.getmtime(src), _newest_header())):
        tmp = UBENCH_OUT + ".tmp%d" % os.getpid()
        r = subprocess.run([NVCC] + FLAGS + [src, "-o", tmp], capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError("nvcc failed for ubench.cu:\n%s\n%s" % (r.stdout, r.stderr))
        os.replace(tmp, UBENCH_OUT)
    return UBENCH_OUT


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
    print(build_ubench(force="--force" in sys.argv))
