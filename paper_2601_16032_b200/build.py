"""Builds libsawtooth_attn.so (the C-ABI library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess

PKG = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(PKG, "csrc")
ROOT = os.path.dirname(PKG)
LIB = os.path.join(PKG, "libsawtooth_attn.so")
SOURCES = [os.path.join(CSRC, "api.cu")]
DEPS = SOURCES + [os.path.join(CSRC, f) for f in ("attn_fwd_sm100.cuh", "ptx.cuh", "schedule.h")] + \
    [os.path.join(ROOT, "include", "sawtooth_attn.h")]

NVCC_FLAGS = [
    "-std=c++17", "-O3", "-lineinfo",
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-Xcompiler", "-fPIC", "-shared",
    "-cudart", "static",
]


def is_stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(f) > t for f in DEPS)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not is_stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-o", LIB] + SOURCES
    subprocess.run(cmd, check=True)
    return LIB


HOST_CALL_SRC = os.path.join(ROOT, "profile_host_call.cu")
HOST_CALL_BIN = os.path.join(PKG, "profile_host_call")


def build_host_call_probe(force: bool = False) -> str:
    """Builds the C program that times one attn_fwd call from C (a measuring aid of bench.py) against the in-tree library."""
    build()
    if not force and os.path.exists(HOST_CALL_BIN) and os.path.getmtime(HOST_CALL_BIN) >= max(os.path.getmtime(HOST_CALL_SRC), os.path.getmtime(LIB)):
        return HOST_CALL_BIN
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-O2", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-o", HOST_CALL_BIN, HOST_CALL_SRC,
           "-L" + PKG, "-lsawtooth_attn", "-Xlinker", "-rpath", "-Xlinker", "$ORIGIN"]
    subprocess.run(cmd, check=True, cwd=ROOT)
    return HOST_CALL_BIN


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv))
    print(build_host_call_probe(force=True))
