"""Builds ``libapproxifer.so`` (sm_100a) in-tree with nvcc.

    python -m paper_2109_09868_b200.build [--force] [--verbose]

Objects go to ``paper_2109_09868_b200/_build/``; the shared library is written
next to this file.  nvcc cross-compiles, so no GPU is needed to build.
"""
from __future__ import annotations

import argparse
import concurrent.futures
import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
OBJDIR = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libapproxifer.so")

SOURCES = ["api.cu", "tables.cpp", "encode.cu", "decode.cu", "decode_small.cu", "decode_pack.cu", "decode_staged.cu", "locate.cu", "locate_rows.cu", "locate_rows_n8.cu", "locate_rows_n16.cu", "locate_rows_n24.cu", "locate_rows_n32.cu", "host_api.cu", "no_alloc.cu"]
ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]
CFLAGS = ["-O3", "-std=c++17", "-lineinfo", "-Xcompiler", "-fPIC", "-Xcompiler", "-Wall", "--expt-relaxed-constexpr"]


def nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found; the library cannot be built")
    return exe


MIN_CUDA = (12, 8)  # sm_100a needs CUDA 12.8; kernel parameter blocks above 4 KB (the weight tables) need 12.1


def check_toolkit() -> None:
    """Fails with a clear message when nvcc is older than the kernels need."""
    import re

    out = subprocess.run([nvcc(), "--version"], capture_output=True, text=True).stdout
    m = re.search(r"release (\d+)\.(\d+)", out)
    if m and (int(m.group(1)), int(m.group(2))) < MIN_CUDA:
        raise RuntimeError("nvcc %s.%s is too old: the library needs CUDA %d.%d or later (sm_100a target, kernel "
                           "parameter blocks of up to 32 KB)" % (m.group(1), m.group(2), *MIN_CUDA))


def _deps_mtime() -> float:
    paths = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(INCLUDE, "approxifer.h"), __file__]
    return max(os.path.getmtime(p) for p in paths)


def is_stale() -> bool:
    return (not os.path.exists(LIB)) or os.path.getmtime(LIB) < _deps_mtime()


def _compile(src: str, verbose: bool) -> str:
    obj = os.path.join(OBJDIR, os.path.splitext(src)[0] + ".o")
    cmd = [nvcc(), *ARCH, *CFLAGS, "-I", INCLUDE, "-c", os.path.join(CSRC, src), "-o", obj]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
        print(" ".join(cmd), flush=True)
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError("nvcc failed on %s:\n%s\n%s" % (src, r.stdout, r.stderr))
    if verbose:
        print(r.stderr, flush=True)
    return obj


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not is_stale():
        return LIB
    check_toolkit()
    os.makedirs(OBJDIR, exist_ok=True)
    with concurrent.futures.ThreadPoolExecutor(max_workers=len(SOURCES)) as ex:
        objs = list(ex.map(lambda s: _compile(s, verbose), SOURCES))
    tmp = LIB + ".tmp.%d" % os.getpid()
    cmd = [nvcc(), *ARCH, "-shared", "-o", tmp, *objs]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError("link failed:\n%s\n%s" % (r.stdout, r.stderr))
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    ap = argparse.ArgumentParser()
    ap.add_argument("--force", action="store_true")
    ap.add_argument("--verbose", action="store_true")
    args = ap.parse_args()
    print(build(args.force, args.verbose))
    sys.exit(0)
