"""Builds libpqhsa.so (sm_100a) in-tree with nvcc.  `python -m paper_2609_33746_b200.build`."""
from __future__ import annotations

import concurrent.futures
import os
import shutil
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libpqhsa.so")
SOURCES = ["api.cu", "lut.cu", "scan.cu", "scan4.cu", "select.cu", "attend.cu", "select_static.cu", "dense.cu",
           "update.cu", "build.cu", "rescore.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"),
              "-I", CSRC]


def _nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found: the CUDA library cannot be built")
    return exe


def _stale(sources, lib=None) -> bool:
    lib = lib or LIB
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + \
           [os.path.join(ROOT, "include", "pqhsa.h"), os.path.abspath(__file__)]
    return any(os.path.getmtime(d) > t for d in deps)


DEBUG_LIB = os.path.join(PKG, "libpqhsa_debug.so")


def build_library(force: bool = False, verbose: bool = False, extra_flags=(), debug: bool = False) -> str:
    """Compile every .cu under csrc/ for sm_100a and link libpqhsa.so next to this file.

    debug=True builds libpqhsa_debug.so with -DPQHSA_DEBUG instead: the same kernels, which also
    record (in the status word) every index that the release build silently clamps or skips.
    Select it at run time with the environment variable PQHSA_LIBRARY."""
    sources = [s for s in SOURCES if os.path.exists(os.path.join(CSRC, s))]
    lib = DEBUG_LIB if debug else LIB
    if debug:
        extra_flags = tuple(extra_flags) + ("-DPQHSA_DEBUG",)
    if not force and not _stale(sources, lib):
        return lib
    nvcc = _nvcc()
    objdir = os.path.join(PKG, "build", "debug" if debug else "release")
    os.makedirs(objdir, exist_ok=True)

    def compile_one(src):
        obj = os.path.join(objdir, src.replace(".cu", ".o"))
        cmd = [nvcc, *NVCC_FLAGS, *extra_flags, "-c", os.path.join(CSRC, src), "-o", obj]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError(f"nvcc failed for {src}:\n{r.stdout}\n{r.stderr}")
        if verbose and (r.stdout or r.stderr):
            print(r.stdout, r.stderr, file=sys.stderr)
        return obj

    with concurrent.futures.ThreadPoolExecutor(max_workers=len(sources)) as ex:
        objs = list(ex.map(compile_one, sources))
    cmd = [nvcc, "-shared", "-o", lib, *objs, "-lcudart"]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError(f"link failed:\n{r.stdout}\n{r.stderr}")
    return lib


if __name__ == "__main__":
    flags = ["-Xptxas", "-v"] if "-v" in sys.argv else []
    print(build_library(force=True, verbose=True, extra_flags=flags, debug="--debug" in sys.argv))
