"""Builds libciera.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import shutil
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libciera.so")
SOURCES = ["ciera_host.cu", "ciera_encode.cu", "ciera_encode_hashed.cu", "ciera_decode.cu", "ciera_entropy.cu", "ciera_kernels.cu"]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden",
    "-Xptxas", "-v",
]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found")


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(ROOT, "include", "ciera.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build_library(force: bool = False, verbose: bool = False) -> str:
    if not force and not needs_build():
        return LIB
    tmp = f"{LIB}.{os.getpid()}.tmp"  # built beside its place and moved there whole: nobody loads half a library
    cmd = [_nvcc(), "-shared", "-o", tmp, "-I", os.path.join(ROOT, "include"), "-I", CSRC] + NVCC_FLAGS
    cmd += [os.path.join(CSRC, s) for s in SOURCES]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or res.returncode != 0:
        print(res.stdout)
        print(res.stderr)
    if res.returncode != 0:
        if os.path.exists(tmp):
            os.remove(tmp)
        raise RuntimeError("nvcc failed building libciera.so")
    os.replace(tmp, LIB)
    return LIB


def ensure_library(wait_s: float = 600.0) -> str:
    """Builds the library if it is not there at all (a fresh checkout); a library that is there is used as it
    is.  Of several processes started together (one per GPU) the one with LOCAL_RANK 0 builds, the others wait."""
    import time

    if os.path.exists(LIB):
        return LIB
    if int(os.environ.get("LOCAL_RANK", "0")) == 0:
        return build_library(force=True)
    t0 = time.time()
    while not os.path.exists(LIB):
        if time.time() - t0 > wait_s:
            raise RuntimeError("libciera.so did not appear: build it with python -m paper_2609_04609_b200.build")
        time.sleep(1.0)
    return LIB


if __name__ == "__main__":
    build_library(force=True, verbose=True)
