"""Builds libpsd_b200.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libpsd_b200.so")
LIB_DEBUG = os.path.join(PKG, "libpsd_b200_debug.so")   # the same sources compiled with -DPSD_DEBUG
SOURCES = ["psd_api.cu", "confidence_tc.cu", "confidence_tc2.cu", "confidence_simt.cu", "combine.cu", "policy.cu",
           "confidence_static.cu", "decode_loop.cu", "dag.cu", "compact.cu"]
EXTRA_SOURCES: list[str] = []
NVCC_FLAGS = [*os.environ.get("PSD_NVCC_EXTRA", "").split(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-Xptxas", "-v"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def _newest_source_mtime() -> float:
    paths = [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    paths.append(os.path.join(ROOT, "include", "psd.h"))
    return max(os.path.getmtime(p) for p in paths)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Compile every .cu of the package into one shared library; returns its path.  debug=True builds
    the variant with device-side bounds and ring-order checks (PSD_DEBUG) next to it."""
    lib = LIB_DEBUG if debug else LIB
    if not force and os.path.exists(lib) and os.path.getmtime(lib) >= _newest_source_mtime():
        return lib
    srcs = [os.path.join(CSRC, s) for s in SOURCES + EXTRA_SOURCES]
    tmp = lib + ".tmp.%d" % os.getpid()
    cmd = [_nvcc(), *NVCC_FLAGS, *(["-DPSD_DEBUG"] if debug else []), "-I", os.path.join(ROOT, "include"), "-I", CSRC,
           "-shared", "-o", tmp, *srcs, "-lcudart"]
    res = subprocess.run(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
    if verbose or res.returncode != 0:
        sys.stderr.write(res.stdout)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed building " + os.path.basename(lib))
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose=True, debug="--debug" in sys.argv))
