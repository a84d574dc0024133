"""Builds libsmtm.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import glob
import hashlib
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libsmtm.so")
STAMP = LIB + ".sources"     # digest of the sources the library was built from
INCLUDE = os.path.join(os.path.dirname(HERE), "include")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "--use_fast_math=false", "-Xcompiler", "-fPIC", "-shared", "-cudart", "static"]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def source_hash() -> str:
    """Digest of everything the library is compiled from (contents, not time stamps)."""
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(CSRC, "*.h")) + \
        glob.glob(os.path.join(INCLUDE, "*.h"))
    h = hashlib.sha256(" ".join(NVCC_FLAGS).encode())
    for d in sorted(deps):
        h.update(os.path.basename(d).encode())
        h.update(open(d, "rb").read())
    return h.hexdigest()


def stale() -> bool:
    """True when the library is missing or was built from other sources than the ones present."""
    if not (os.path.exists(LIB) and os.path.exists(STAMP)):
        return True
    return open(STAMP).read().strip() != source_hash()


def build(force: bool = False, verbose: bool = False) -> str:
    if force or stale():
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        tmp = f"{LIB}.{os.getpid()}.tmp"
        cmd = [nvcc] + [f for f in NVCC_FLAGS if f != "--use_fast_math=false"] + \
            (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp] + sources()
        subprocess.run(cmd, check=True)
        os.replace(tmp, LIB)            # atomic: a process that loads meanwhile sees the old or the new file
        with open(tmp + ".sources", "w") as f:
            f.write(source_hash() + "\n")
        os.replace(tmp + ".sources", STAMP)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
