"""Builds the CUDA library in-tree: ``paper_2503_09387_b200/lib/libvideoscan.so``.

Every translation unit is compiled for sm_100a only (``-gencode
arch=compute_100a,code=sm_100a``); the CUDA runtime is linked statically and the driver
entry point needed for TMA descriptors is resolved at run time, so the library loads on
a machine without a GPU (e.g. to check its exported symbols).
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB_DIR = os.path.join(HERE, "lib")
LIB_PATH = os.path.join(LIB_DIR, "libvideoscan.so")
SOURCES = ["vs_host.cu", "vs_kernels_misc.cu", "vs_gemm_tcgen05.cu", "vs_gemv.cu", "vs_attention.cu", "vs_attention_tc.cu", "vs_noalloc.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC"]


def _nvcc() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def _stale(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


CHECKED_LIB_PATH = os.path.join(LIB_DIR, "libvideoscan_checked.so")


def build_library(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    """checked=True builds the same sources with -DVS_DEBUG_BOUNDS into libvideoscan_checked.so: every kernel store into
    the workspace is checked against the region it names, and guard bytes lie behind every region."""
    os.makedirs(LIB_DIR, exist_ok=True)
    obj_dir = os.path.join(LIB_DIR, "obj_checked" if checked else "obj")
    lib_path = CHECKED_LIB_PATH if checked else LIB_PATH
    extra = ["-DVS_DEBUG_BOUNDS"] if checked else []
    os.makedirs(obj_dir, exist_ok=True)
    headers = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cuh", ".h"))]
    headers.append(os.path.join(os.path.dirname(HERE), "include", "videoscan.h"))
    jobs = []
    for src in SOURCES:
        s = os.path.join(CSRC, src)
        o = os.path.join(obj_dir, src.replace(".cu", ".o"))
        if force or _stale(o, [s] + headers):
            cmd = [_nvcc()] + NVCC_FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + ["-c", s, "-o", o]
            jobs.append(cmd)
    def run(cmd):
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError("nvcc failed: %s\n%s\n%s" % (" ".join(cmd), r.stdout, r.stderr))
        if verbose:
            sys.stderr.write(r.stderr)
    with ThreadPoolExecutor(max_workers=4) as ex:
        list(ex.map(run, jobs))
    objs = [os.path.join(obj_dir, s.replace(".cu", ".o")) for s in SOURCES]
    if force or jobs or _stale(lib_path, objs):
        cmd = [_nvcc(), "-shared", "-cudart", "static", "-o", lib_path] + objs + ["-lpthread", "-ldl", "-lrt"]
        run(cmd)
    return lib_path


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv, checked="--checked" in sys.argv))
