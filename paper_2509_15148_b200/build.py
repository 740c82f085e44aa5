"""Builds libatts.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import hashlib
import os
import shutil
import subprocess
import sys

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG_DIR)
CSRC = os.path.join(PKG_DIR, "csrc")
LIB_PATH = os.path.join(PKG_DIR, "libatts.so")
SOURCES = [os.path.join(CSRC, "atts.cu")]
HEADERS = [os.path.join(CSRC, "conformal.cuh"), os.path.join(CSRC, "lmhead_lse.cuh"),
           os.path.join(ROOT, "include", "atts.h")]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: libatts cannot be built")


STAMP_PATH = LIB_PATH + ".src"   # digest of the sources the library was built from


def source_digest() -> str:
    h = hashlib.sha256()
    for f in SOURCES + HEADERS:
        with open(f, "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def is_stale() -> bool:
    """True unless libatts.so was built from exactly the present sources (compared by content, not by file time:
    a copy of the tree need not keep modification times)."""
    if not os.path.exists(LIB_PATH) or not os.path.exists(STAMP_PATH):
        return True
    with open(STAMP_PATH) as fh:
        return fh.read().strip() != source_digest()


def build_library(force: bool = False, verbose: bool = False) -> str:
    """Compile csrc/atts.cu into libatts.so next to this file; returns the library path."""
    if not force and not is_stale():
        return LIB_PATH
    digest = source_digest()   # taken before compiling, so an edit during the build leaves the library stale
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC,
           "-o", LIB_PATH] + SOURCES
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed building libatts.so")
    with open(STAMP_PATH, "w") as fh:
        fh.write(digest + "\n")
    return LIB_PATH


if __name__ == "__main__":
    print(build_library(force=True, verbose="-v" in sys.argv))
