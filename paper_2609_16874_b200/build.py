"""Builds ``libcpe.so`` (the CUDA decoder behind the C ABI of ``include/cpe.h``) in-tree with nvcc for sm_100a.

Every ``csrc/*.cu`` is one translation unit; the units are compiled side by side (one nvcc process each) into
``csrc/build/*.o`` and linked into the shared library.  An object is rebuilt when its source or any header is newer.
"""
from __future__ import annotations

import concurrent.futures
import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
OBJ = os.path.join(CSRC, "build")
INCLUDE = os.path.join(ROOT, "include")
LIB = os.path.join(PKG, "libcpe.so")

NVCC_FLAGS = [
    "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
    "-Xcompiler", "-fPIC",
    # the per-pixel estimate decides integers: no fast-math, no flush-to-zero, IEEE division and sqrt
    "-ftz=false", "-prec-div=true", "-prec-sqrt=true", "-fmad=true",
]


def sources():
    return sorted(os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith(".cu"))


def _headers():
    out = [os.path.join(INCLUDE, f) for f in os.listdir(INCLUDE)]
    out += [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cuh", ".h"))]
    return out


def _obj(src: str) -> str:
    return os.path.join(OBJ, os.path.basename(src)[:-3] + ".o")


def is_stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(p) > t for p in _headers() + sources())


def _nvcc() -> str:
    nvcc = os.environ.get("NVCC") or "/usr/local/cuda/bin/nvcc"
    return nvcc if os.path.exists(nvcc) else "nvcc"


def build_library(force: bool = False, verbose: bool = False, extra=()) -> str:
    """Compile every ``csrc/*.cu`` and link ``libcpe.so``; returns its path.  Needs nvcc, not a GPU."""
    if not force and not is_stale():
        return LIB
    os.makedirs(OBJ, exist_ok=True)
    nvcc = _nvcc()
    newest_header = max(os.path.getmtime(p) for p in _headers())
    jobs = []
    for src in sources():
        obj = _obj(src)
        if (not force and not extra and os.path.exists(obj)
                and os.path.getmtime(obj) >= max(newest_header, os.path.getmtime(src))):
            continue
        cmd = [nvcc] + NVCC_FLAGS + list(extra) + ["-I", INCLUDE, "-I", CSRC, "-c", "-o", obj, src]
        if verbose:
            cmd.insert(1, "-Xptxas=-v")
        jobs.append(cmd)

    def run(cmd):
        r = subprocess.run(cmd, capture_output=True, text=True)
        return cmd, r

    with concurrent.futures.ThreadPoolExecutor(max_workers=max(1, min(len(jobs), os.cpu_count() or 4))) as pool:
        for cmd, r in pool.map(run, jobs):
            if verbose or r.returncode:
                print(" ".join(cmd), file=sys.stderr)
                sys.stderr.write(r.stdout + r.stderr)
            if r.returncode:
                raise subprocess.CalledProcessError(r.returncode, cmd)
    tmp = LIB + f".{os.getpid()}.tmp"
    subprocess.run([nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", tmp] +
                   [_obj(s) for s in sources()], check=True)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    build_library(force="-f" in sys.argv, verbose="-v" in sys.argv)
    print(LIB)
