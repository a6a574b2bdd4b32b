"""Build the CUDA library in-tree: ``python -m paper_2609_19702_b200.build``.

Compiles the translation units under ``csrc/`` for sm_100a with nvcc -- ``dsa_api.cu`` (entry
points, planner, small kernels) and one unit per (element type, head_dim) with the attention
kernels, in parallel -- and links them into ``libdsa.so`` beside this file.  nvcc cross-compiles,
so no GPU is needed to build.
"""
from __future__ import annotations

import concurrent.futures
import os
import shutil
import subprocess
import sys
import tempfile

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libdsa.so")
SOURCES = ["dsa_api.cu", "dsa_kernels_bf16_d128.cu", "dsa_kernels_bf16_d64.cu", "dsa_kernels_f32_d128.cu",
           "dsa_kernels_f32_d64.cu"]


def _newest_source_mtime() -> float:
    """Newest of the translation units, every header under csrc/ and the public header."""
    paths = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cu", ".cuh", ".h"))]
    paths.append(os.path.join(HERE, "..", "include", "dsa.h"))
    return max(os.path.getmtime(p) for p in paths if os.path.exists(p))


def build(force: bool = False, verbose: bool = False, out: str = LIB) -> str:
    if not force and os.path.exists(out) and os.path.getmtime(out) >= _newest_source_mtime():
        return out
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    flags = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "--extended-lambda",
             "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden"]
    if verbose:
        flags += ["-Xptxas", "-v"]
    work = tempfile.mkdtemp(prefix="dsa_build_")
    try:
        def compile_one(src: str) -> str:
            obj = os.path.join(work, os.path.splitext(src)[0] + ".o")
            subprocess.run([nvcc] + flags + ["-c", os.path.join(CSRC, src), "-o", obj], check=True)
            return obj

        with concurrent.futures.ThreadPoolExecutor(max_workers=min(len(SOURCES), os.cpu_count() or 1)) as pool:
            objs = list(pool.map(compile_one, SOURCES))
        tmp = out + ".tmp.%d" % os.getpid()
        subprocess.run([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-o", tmp] + objs, check=True)
        os.replace(tmp, out)
    finally:
        shutil.rmtree(work, ignore_errors=True)
    return out


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
