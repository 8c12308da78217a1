"""Builds the CUDA library in-tree with nvcc for sm_100a (no JIT cache, no torch extension machinery)."""
from __future__ import annotations

import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(PKG, "csrc")
# FICACHE_LIB names another build of the library to load instead of the in-tree one (it is then never rebuilt here)
LIB = os.environ.get("FICACHE_LIB") or os.path.join(PKG, "libficache.so")
SOURCES = ["fi_api.cu", "fi_stream.cu", "fi_finalize.cu", "fi_gemm.cu", "fi_noalloc.cu", "fi_kmeans.cu"]
HEADERS = [os.path.join(CSRC, "fi_internal.cuh"), os.path.join(os.path.dirname(PKG), "include", "fi.h")]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC"]
OBJ_DIR = os.path.join(PKG, "_build")


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    return "nvcc"


def stale() -> bool:
    if not os.path.exists(LIB):
        return True
    built = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, s) for s in SOURCES] + HEADERS
    return any(os.path.getmtime(d) > built for d in deps)


def build_library(force: bool = False, verbose: bool = False) -> str:
    """Compile csrc/*.cu into libficache.so next to this file; returns its path.  The sources are compiled side by
    side into objects under _build/ (only those older than their source or a header) and then linked."""
    if os.environ.get("FICACHE_LIB"):
        return LIB
    if not force and not stale():
        return LIB
    from concurrent.futures import ThreadPoolExecutor
    os.makedirs(OBJ_DIR, exist_ok=True)
    newest_header = max(os.path.getmtime(h) for h in HEADERS)

    def compile_one(src: str):
        path = os.path.join(CSRC, src)
        obj = os.path.join(OBJ_DIR, src[:-3] + ".o")
        if not force and os.path.exists(obj) and os.path.getmtime(obj) > max(os.path.getmtime(path), newest_header):
            return obj, 0, ""
        tmp = obj + f".{os.getpid()}.tmp"
        cmd = [_nvcc()] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-c", "-o", tmp, path]
        proc = subprocess.run(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
        if proc.returncode == 0:
            os.replace(tmp, obj)
        return obj, proc.returncode, proc.stdout

    with ThreadPoolExecutor(len(SOURCES)) as ex:
        results = list(ex.map(compile_one, SOURCES))
    for _, rc, out in results:
        if verbose or rc != 0:
            sys.stderr.write(out)
    if any(rc != 0 for _, rc, _ in results):
        raise RuntimeError("nvcc failed building libficache.so")
    tmp = LIB + f".{os.getpid()}.tmp"
    proc = subprocess.run([_nvcc(), "-shared", "-o", tmp] + [o for o, _, _ in results], stdout=subprocess.PIPE,
                          stderr=subprocess.STDOUT, text=True)
    if proc.returncode != 0:
        sys.stderr.write(proc.stdout)
        raise RuntimeError("linking libficache.so failed")
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv))
