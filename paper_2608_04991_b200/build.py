"""Builds ``librac.so`` (the C-ABI library of CUDA kernels) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "librac.so")
SOURCES = ["rac_codec.cu", "rac_codec_dyn.cu", "rac_match.cu"]
HEADERS = ["rac_common.cuh", "rac_codec_dev.cuh", os.path.join("..", "..", "include", "rac.h")]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-shared", "--threads", "0", "-Xptxas", "-v",
]


def _newest_source() -> float:
    files = [os.path.join(CSRC, s) for s in SOURCES + HEADERS]
    return max(os.path.getmtime(f) for f in files)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile when the library is missing or older than its sources.  Returns the library path."""
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= _newest_source():
        return LIB
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = LIB + f".tmp{os.getpid()}"
    cmd = [nvcc, *NVCC_FLAGS, "-o", tmp, *[os.path.join(CSRC, s) for s in SOURCES]]
    try:
        res = subprocess.run(cmd, capture_output=True, text=True)
        if verbose or res.returncode != 0:
            sys.stderr.write(res.stdout + res.stderr)
        if res.returncode != 0:
            raise RuntimeError("nvcc failed: " + " ".join(cmd))
        os.replace(tmp, LIB)
    finally:
        if os.path.exists(tmp):     # a failed or interrupted build leaves nothing behind
            os.remove(tmp)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose=True))
