"""Build the CUDA library in-tree with nvcc for sm_100a.

Each source is compiled to an object of its own (in parallel, and only when it or a header is newer than
the object), then the objects are linked into libmpgemmfi.so next to this file.
"""
from __future__ import annotations

import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ_DIR = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libmpgemmfi.so")
SOURCES = ["api.cu", "gemm_sm100.cu", "campaign.cu", "operands.cu"]
ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]


def _headers_mtime() -> float:
    paths = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cuh", ".h"))]
    paths.append(os.path.join(os.path.dirname(HERE), "include", "mpgemmfi.h"))
    return max(os.path.getmtime(p) for p in paths)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile csrc/*.cu into libmpgemmfi.so (objects and library are rebuilt only when older than their sources)."""
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    os.makedirs(OBJ_DIR, exist_ok=True)
    hdr_time = _headers_mtime()
    jobs = []
    for src in SOURCES:
        path = os.path.join(CSRC, src)
        obj = os.path.join(OBJ_DIR, src[:-3] + ".o")
        stale = force or not os.path.exists(obj) or os.path.getmtime(obj) < max(os.path.getmtime(path), hdr_time)
        if stale:
            cmd = [nvcc, *ARCH, "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC", "-c", path, "-o", obj]
            if verbose:
                cmd[1:1] = ["-Xptxas", "-v"]
            jobs.append(cmd)
    if jobs:
        with ThreadPoolExecutor(max_workers=len(jobs)) as pool:
            for r in pool.map(lambda c: subprocess.run(c, check=False), jobs):
                if r.returncode != 0:
                    raise subprocess.CalledProcessError(r.returncode, r.args)
    objs = [os.path.join(OBJ_DIR, s[:-3] + ".o") for s in SOURCES]
    if jobs or not os.path.exists(LIB) or os.path.getmtime(LIB) < max(os.path.getmtime(o) for o in objs):
        subprocess.run([nvcc, *ARCH, "-shared", "-Xcompiler", "-fPIC", "-o", LIB, *objs, "-ldl"], check=True)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose=True))
