"""Builds the C-ABI shared library (libsparsed.so) in-tree with nvcc for sm_100a.

Each .cu file is compiled to an object of its own (in parallel, skipped when the object is newer
than the source and every header), then the objects are linked into the shared library.
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(PKG_DIR, "csrc")
OBJ_DIR = os.path.join(PKG_DIR, "build")
LIB_PATH = os.path.join(PKG_DIR, "libsparsed.so")
SOURCES = ["api.cu", "attention.cu", "attention_dense_pair.cu", "scoring.cu", "topk.cu", "pool_select.cu", "patterns.cu",
           "pooled_qk.cu"]
HEADERS = ["internal.h", "sm100_primitives.cuh", "sm100_pair_primitives.cuh", "softmax_pipeline.cuh", "topk_device.cuh",
           os.path.join("..", "..", "include", "sparsed.h")]
ARCH_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a"]
COMMON_FLAGS = ["-O3", "-std=c++17", "-lineinfo", "-Xcompiler", "-fPIC"]
# Flags of single files. The CTA-pair dense kernel is built with denormals flushed to zero: its softmax handles
# probabilities, for which a flushed 1e-38 is as good as the number, and the kernel measured 2-4 % faster that way
# (8k-64k); the other kernels measured the same or slower with it and keep IEEE denormals.
PER_FILE_FLAGS = {"attention_dense_pair.cu": ["-ftz=true"]}


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found; the SparseD library needs the CUDA 12.9 toolkit to build")


def _deps():
    return [os.path.join(CSRC, s) for s in SOURCES + HEADERS if os.path.exists(os.path.join(CSRC, s))]


def is_stale() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    return any(os.path.getmtime(d) > t for d in _deps())


def _compile_one(nvcc: str, src: str, obj: str, verbose: bool, extra):
    own = PER_FILE_FLAGS.get(os.path.basename(src), [])
    cmd = [nvcc] + ARCH_FLAGS + COMMON_FLAGS + own + list(extra) + (["-Xptxas", "-v"] if verbose else []) + ["-c", src, "-o", obj]
    res = subprocess.run(cmd, capture_output=True, text=True)
    return src, res


def build_library(force: bool = False, verbose: bool = False, extra_flags=()) -> str:
    if not force and not is_stale() and not extra_flags:
        return LIB_PATH
    nvcc = _nvcc()
    os.makedirs(OBJ_DIR, exist_ok=True)
    header_time = max(os.path.getmtime(os.path.join(CSRC, h)) for h in HEADERS if os.path.exists(os.path.join(CSRC, h)))
    jobs, objs = [], []
    for s in SOURCES:
        src = os.path.join(CSRC, s)
        obj = os.path.join(OBJ_DIR, s.replace(".cu", ".o"))
        objs.append(obj)
        fresh = (os.path.exists(obj) and os.path.getmtime(obj) > max(os.path.getmtime(src), header_time))
        if force or verbose or extra_flags or not fresh:
            jobs.append((src, obj))
    with ThreadPoolExecutor(max_workers=min(8, max(1, len(jobs)))) as pool:
        results = list(pool.map(lambda j: _compile_one(nvcc, j[0], j[1], verbose, extra_flags), jobs))
    for src, res in results:
        if verbose:
            sys.stderr.write(res.stderr)
        if res.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}:\n" + res.stdout + res.stderr)
    tmp_path = f"{LIB_PATH}.tmp{os.getpid()}.so"
    res = subprocess.run([nvcc] + ARCH_FLAGS + ["-shared", "-o", tmp_path] + objs, capture_output=True, text=True)
    if res.returncode != 0:
        if os.path.exists(tmp_path):
            os.remove(tmp_path)
        raise RuntimeError("link failed:\n" + res.stdout + res.stderr)
    os.replace(tmp_path, LIB_PATH)   # atomic: a concurrent loader never sees a half-written library
    return LIB_PATH


if __name__ == "__main__":
    print(build_library(force=True, verbose="-v" in sys.argv))
