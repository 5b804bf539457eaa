"""Builds libpasta.so (CUDA kernels + C ABI) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import hashlib
import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libpasta.so")
SOURCES = ["pool.cpp", "plan.cpp", "kernels.cu", "attn_tensor.cu", "api.cu", "noalloc.cu", "dense_mask.cu"]
HEADERS = ["pool.hpp", "plan.hpp", "pasta_plan.h", "device_common.cuh", "kernels.hpp",
           os.path.join("..", "..", "include", "pasta.h")]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found")


FLAGS = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
         "-Xcompiler", "-fPIC,-Wall", "-shared", "-cudart", "shared", "-Xlinker", "-rpath,/usr/local/cuda/lib64"]
STAMP = LIB + ".sha256"


def source_hash() -> str:
    """Hash of everything the library is built from: sources, headers and compiler flags."""
    h = hashlib.sha256(" ".join(FLAGS).encode())
    for f in SOURCES + HEADERS:
        with open(os.path.join(CSRC, f), "rb") as fh:
            h.update(f.encode() + b"\0" + fh.read() + b"\0")
    return h.hexdigest()


def is_stale() -> bool:
    """True unless the library on disk was built from exactly the sources on disk (file times say nothing after a
    checkout or a copy): the hash of the sources it was built from is kept beside it."""
    if not os.path.exists(LIB) or not os.path.exists(STAMP):
        return True
    with open(STAMP) as fh:
        return fh.read().strip() != source_hash()


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not is_stale():
        return LIB
    stamp = source_hash()
    cmd = [_nvcc()] + FLAGS + ["-o", LIB] + [os.path.join(CSRC, f) for f in SOURCES]
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    if os.path.exists(STAMP):
        os.unlink(STAMP)
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + " ".join(cmd) + "\n" + res.stdout + res.stderr)
    with open(STAMP, "w") as fh:
        fh.write(stamp + "\n")
    if verbose:
        print(res.stdout + res.stderr)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
