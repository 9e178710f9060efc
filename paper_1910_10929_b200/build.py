"""Builds libdgs.so (the C ABI of include/dgs.h) with nvcc for sm_100a, in-tree."""
from __future__ import annotations

import hashlib
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libdgs.so")
SOURCES = [os.path.join(CSRC, "dgs.cu")]
DEPENDS = SOURCES + [os.path.join(CSRC, "dgs_kernels.cuh"), os.path.join(ROOT, "include", "dgs.h")]

NVCC_FLAGS = [
    "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
    # every float operation is a single rounded IEEE operation: no contraction, no flush-to-zero
    "-fmad=false", "-ftz=false", "-prec-div=true", "-prec-sqrt=true",
    "-shared", "-Xcompiler", "-fPIC", "-diag-suppress", "177",
]


STAMP = LIB + ".hash"


def source_hash() -> str:
    """Hash of everything the library is made from: the sources, the header, the compiler flags."""
    h = hashlib.sha256()
    h.update("\0".join(NVCC_FLAGS).encode())
    for p in DEPENDS:
        h.update(b"\0" + os.path.basename(p).encode() + b"\0")
        with open(p, "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def stale() -> bool:
    """True unless the library was built from exactly the sources that are here now (decided by content:
    the hash stored beside the library at build time, not by file times)."""
    if not os.path.exists(LIB) or not os.path.exists(STAMP):
        return True
    with open(STAMP) as f:
        return f.read().strip() != source_hash()


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not stale():
        return LIB
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = LIB + f".{os.getpid()}.tmp"
    cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + [
        "-I", os.path.join(ROOT, "include"), "-o", tmp] + SOURCES
    digest = source_hash()
    subprocess.check_call(cmd)
    os.replace(tmp, LIB)
    with open(STAMP, "w") as f:
        f.write(digest + "\n")
    return LIB


if __name__ == "__main__":
    import sys
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
