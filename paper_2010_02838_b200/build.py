"""Builds the C-ABI library ``libcodistill.so`` in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
OBJ_DIR = os.path.join(_HERE, "_build")
LIB = os.path.join(_HERE, "libcodistill.so")
SOURCES = ["api.cu", "rows_generic.cu", "rows_tma.cu", "rows_stream.cu", "rows_stream_kl.cu", "rows_all.cu", "rows_cluster.cu", "schedule.cu", "predictions.cu", "rows_short.cu"]
HEADERS = ["common.cuh", "seg_math.cuh", "stream_common.cuh", "bulk_copy.cuh", "cluster_args.cuh", os.path.join("..", "..", "include", "codistill.h"),
           os.path.join("..", "..", "include", "codistill_schedule.h")]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-Xptxas", "-v"]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS] + [os.path.abspath(__file__)]
    return any(os.path.getmtime(d) > t for d in deps)


def _compile(nvcc: str, src: str, force: bool):
    """One object per source; an object newer than its source, every header and this script is kept."""
    obj = os.path.join(OBJ_DIR, os.path.splitext(src)[0] + ".o")
    log = obj + ".log"
    deps = [os.path.join(CSRC, src)] + [os.path.join(CSRC, h) for h in HEADERS] + [os.path.abspath(__file__)]
    if not force and os.path.exists(obj) and os.path.exists(log) and all(os.path.getmtime(d) <= os.path.getmtime(obj) for d in deps):
        return obj, subprocess.CompletedProcess([], 0, open(log).read(), "")
    res = subprocess.run([nvcc, *NVCC_FLAGS, "-c", "-o", obj, os.path.join(CSRC, src)], capture_output=True, text=True)
    if res.returncode == 0:
        with open(log, "w") as f:
            f.write(res.stdout + res.stderr)
    return obj, res


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every CUDA source (in parallel, one object per file) and link them into one shared
    library (cross-compiles without a GPU)."""
    if force or _stale():
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        os.makedirs(OBJ_DIR, exist_ok=True)
        with ThreadPoolExecutor(max_workers=min(len(SOURCES), os.cpu_count() or 1)) as pool:
            results = list(pool.map(lambda s: _compile(nvcc, s, force), SOURCES))
        log = "".join(r.stdout + r.stderr for _, r in results)
        failed = [r for _, r in results if r.returncode != 0]
        if verbose or failed:
            sys.stderr.write(log)
        if failed:
            raise RuntimeError("nvcc failed building libcodistill.so")
        link = subprocess.run([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "--shared", "-o", LIB,
                               *[o for o, _ in results]], capture_output=True, text=True)
        if link.returncode != 0:
            sys.stderr.write(link.stdout + link.stderr)
            raise RuntimeError("nvcc failed linking libcodistill.so")
        with open(os.path.join(_HERE, "build_ptxas.log"), "w") as f:
            f.write(log + link.stdout + link.stderr)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose=True))
