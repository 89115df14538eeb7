"""Builds libtucker_attn.so (sm_100a only) next to this file with nvcc, and libtucker_attn_checked.so, the
same sources compiled with -DTA_BOUNDS_CHECK (every global index the kernels form is range-checked on the
device and reported through the device error word; load it with TUCKER_ATTN_LIB=checked).

    python -m paper_2603_30033_b200.build [--force] [--verbose] [--no-checked]

Object files go to _build/ at the repository root (ignored by git); the shared library is
written in-tree so that it travels with the source tree.  nvcc cross-compiles without a GPU.
"""
from __future__ import annotations

import argparse
import concurrent.futures as cf
import hashlib
import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(ROOT, "include")
BUILD = os.path.join(ROOT, "_build")
LIB = os.path.join(HERE, "libtucker_attn.so")
LIB_CHECKED = os.path.join(HERE, "libtucker_attn_checked.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "--expt-relaxed-constexpr", "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden",
    "-I", INCLUDE, "-I", CSRC,
]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found")


def _sources():
    return sorted(os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith(".cu"))


def _digest(paths) -> str:
    h = hashlib.sha256()
    for p in sorted(paths):
        h.update(p.encode())
        with open(p, "rb") as f:
            h.update(f.read())
    h.update(" ".join(NVCC_FLAGS).encode())
    return h.hexdigest()


def build(force: bool = False, verbose: bool = False, checked: bool = True) -> str:
    """Builds the library (and, with checked=True, its bounds-checking twin); returns the library's path."""
    lib = _build_one(LIB, BUILD, [], force, verbose)
    if checked:
        _build_one(LIB_CHECKED, os.path.join(BUILD, "checked"), ["-DTA_BOUNDS_CHECK"], force, verbose)
    return lib


def _build_one(LIB: str, BUILD: str, defines, force: bool, verbose: bool) -> str:
    os.makedirs(BUILD, exist_ok=True)
    srcs = _sources()
    deps = srcs + [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cuh", ".h"))] \
        + [os.path.join(INCLUDE, f) for f in os.listdir(INCLUDE)]
    stamp = os.path.join(BUILD, "stamp.txt")
    dig = _digest(deps) + " ".join(defines)
    if not force and os.path.exists(LIB) and os.path.exists(stamp) and open(stamp).read() == dig:
        return LIB
    nvcc = _nvcc()
    extra = ["-Xptxas", "-v"] if verbose else []

    def compile_one(src):
        obj = os.path.join(BUILD, os.path.basename(src)[:-3] + ".o")
        cmd = [nvcc, *NVCC_FLAGS, *defines, *extra, "-c", src, "-o", obj]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError(f"nvcc failed for {src}:\n{r.stdout}\n{r.stderr}")
        if verbose:
            sys.stderr.write(r.stderr)
        return obj

    with cf.ThreadPoolExecutor(max_workers=min(8, len(srcs))) as ex:
        objs = list(ex.map(compile_one, srcs))
    cmd = [nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", LIB, *objs]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError(f"link failed:\n{r.stdout}\n{r.stderr}")
    with open(stamp, "w") as f:
        f.write(dig)
    return LIB


if __name__ == "__main__":
    ap = argparse.ArgumentParser()
    ap.add_argument("--force", action="store_true")
    ap.add_argument("--verbose", action="store_true")
    ap.add_argument("--no-checked", action="store_true", help="skip the bounds-checking build")
    a = ap.parse_args()
    print(build(force=a.force, verbose=a.verbose, checked=not a.no_checked))
