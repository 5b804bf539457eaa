"""Decode attention for interpreter-driven asynchronous decoding on NVIDIA B200 (sm_100a).

`binding` is a thin ctypes layer over the C ABI declared in include/pasta.h; every step of the
path runs in the CUDA library `libpasta.so`, which `build.build()` compiles in-tree.  Nothing
here falls back to the CPU: importing `binding` without the library raises.
"""
from .build import build  # noqa: F401
