"""Builds libgnnpre.so in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
SOURCES = ["plan.cu", "propagate.cu", "stream.cu", "noalloc.cu", "normalize.cu", "lc_layer.cu", "api.cu"]
LIB = os.path.join(HERE, "lib", "libgnnpre.so")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-shared"]


def _inputs():
    src = [os.path.join(HERE, "csrc", s) for s in SOURCES]
    hdr = [os.path.join(HERE, "csrc", "gnnpre_internal.cuh"), os.path.join(HERE, "csrc", "segments_tma.cuh"),
           os.path.join(HERE, "csrc", "segments.cuh"), os.path.join(HERE, "csrc", "segments_common.cuh"), os.path.join(HERE, "csrc", "fixups.cuh"), os.path.join(HERE, "csrc", "ceiling.cuh"),
           os.path.join(ROOT, "include", "gnnpre.h")]
    return src, hdr


def is_stale() -> bool:
    if not os.path.exists(LIB):
        return True
    src, hdr = _inputs()
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(f) > t for f in src + hdr)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile the library if a source is newer than it; returns its path."""
    if not force and not is_stale():
        return LIB
    src, _ = _inputs()
    os.makedirs(os.path.dirname(LIB), exist_ok=True)
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = LIB + f".tmp{os.getpid()}"
    extra = os.environ.get("GNNPRE_NVCC_FLAGS", "").split()
    cmd = [nvcc, *NVCC_FLAGS, *extra, "-I", os.path.join(ROOT, "include"), "-o", tmp, *src]
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    subprocess.run(cmd, check=True)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose=True))
