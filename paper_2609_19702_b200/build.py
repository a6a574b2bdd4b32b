"""Build the CUDA library in-tree: ``python -m paper_2609_19702_b200.build``.

Compiles ``csrc/dsa_api.cu`` (which includes the kernel headers) for sm_100a with nvcc into
``libdsa.so`` beside this file.  nvcc cross-compiles, so no GPU is needed to build.
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libdsa.so")
SOURCES = ["dsa_api.cu"]
HEADERS = ["dsa_attn.cuh", "dsa_attn_mma.cuh", "dsa_tile.cuh", "dsa_common.cuh", "dsa_mask.cuh",
           os.path.join("..", "..", "include", "dsa.h")]


def _newest_source_mtime() -> float:
    paths = [os.path.join(CSRC, s) for s in SOURCES + HEADERS]
    return max(os.path.getmtime(p) for p in paths if os.path.exists(p))


def build(force: bool = False, verbose: bool = False, out: str = LIB) -> str:
    if not force and os.path.exists(out) and os.path.getmtime(out) >= _newest_source_mtime():
        return out
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = out + ".tmp.%d" % os.getpid()
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "--extended-lambda", "-shared", "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden",
           "-o", tmp] + [os.path.join(CSRC, s) for s in SOURCES]
    cmd[1:1] = os.environ.get("DSA_NVCC_FLAGS", "").split()      # e.g. tuning -D overrides
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    subprocess.run(cmd, check=True)
    os.replace(tmp, out)
    return out


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
