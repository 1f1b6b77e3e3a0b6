"""Builds the CUDA library in-tree: csrc/*.cu -> libdl_sparse.so (sm_100a only), and its checked twin
libdl_sparse_checked.so (-DDL_BOUNDS=1: stores through computed indices are compared with their buffers first).

Usage:  python -m paper_2412_00876_b200.build [--force] [--verbose]
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libdl_sparse.so")
LIB_CHECKED = os.path.join(HERE, "libdl_sparse_checked.so")
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC"]


def _sources():
    return sorted(os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith(".cu"))


def source_hash(extra_flags=()) -> str:
    """SHA-256 over every file the library is built from (sources, headers, the C header) and the flags."""
    import hashlib
    h = hashlib.sha256(" ".join([*FLAGS, *extra_flags]).encode())
    paths = sorted(os.path.join(CSRC, f) for f in os.listdir(CSRC))
    paths.append(os.path.join(os.path.dirname(HERE), "include", "dl.h"))
    for p in paths:
        h.update(os.path.basename(p).encode())
        h.update(open(p, "rb").read())
    return h.hexdigest()


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    """Builds the library (or its checked twin) unless the one in place was built from exactly these sources: the
    decision is taken on a hash of the sources stored beside the library, not on file times (a snapshot copied
    elsewhere keeps neither)."""
    variant = ["-DDL_BOUNDS=1"] if checked else []
    LIB = LIB_CHECKED if checked else globals()["LIB"]
    OBJ = globals()["OBJ"] + ("_checked" if checked else "")
    STAMP = LIB + ".src_hash"
    want = source_hash(variant)
    if not force and os.path.exists(LIB) and os.path.exists(STAMP) and open(STAMP).read().strip() == want:
        return LIB
    os.makedirs(OBJ, exist_ok=True)
    extra = variant + (["-Xptxas", "-v"] if verbose else [])

    def compile_one(src):
        obj = os.path.join(OBJ, os.path.basename(src)[:-3] + ".o")
        cmd = [NVCC, *FLAGS, *extra, "-c", src, "-o", obj]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError(f"nvcc failed for {src}:\n{r.stdout}\n{r.stderr}")
        if verbose:
            sys.stderr.write(r.stderr)
        return obj

    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as ex:
        objs = list(ex.map(compile_one, _sources()))
    cmd = [NVCC, "-shared", "-o", LIB, *objs, "-gencode", "arch=compute_100a,code=sm_100a"]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError(f"link failed:\n{r.stdout}\n{r.stderr}")
    with open(STAMP, "w") as f:
        f.write(want + "\n")
    return LIB


def build_all(force: bool = False, verbose: bool = False):
    return build(force, verbose), build(force, verbose, checked=True)


if __name__ == "__main__":
    print(*build_all(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
