"""Builds libzccl.so (the C-ABI library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent
CSRC = PKG / "csrc"
LIB = PKG / "libzccl.so"
SOURCES = [CSRC / "zccl_kernels.cu", CSRC / "zccl_codec.cu", CSRC / "zccl_api.cu", CSRC / "zccl_noalloc.cu", CSRC / "zccl_generic.cu"]
HEADERS = [CSRC / "zccl_internal.h", CSRC / "zccl_device.cuh", CSRC / "zccl_codec_f64.cuh", CSRC / "zccl_codec_tiled.cuh", PKG.parent / "include" / "zccl.h"]

NVCC_FLAGS = [
    "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
    "--fmad=false",                       # no contraction anywhere: streams must be reproducible bit for bit
    "-Xcompiler", "-fPIC,-ffp-contract=off,-fno-fast-math",
    "-shared", "-cudart", "shared",
]


def nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (cand == "nvcc" or Path(cand).exists()):
            return cand
    raise RuntimeError("nvcc not found")


def needs_build() -> bool:
    if not LIB.exists():
        return True
    t = LIB.stat().st_mtime
    return any(p.stat().st_mtime > t for p in SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False, extra: list[str] | None = None) -> Path:
    if not force and not needs_build():
        return LIB
    tmp = LIB.with_suffix(f".tmp{os.getpid()}.so")
    extra = list(extra or []) + os.environ.get("ZCCL_NVCC_EXTRA", "").split()
    cmd = [nvcc(), *NVCC_FLAGS, *extra, "-o", str(tmp), *map(str, SOURCES)]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
        print(" ".join(cmd), file=sys.stderr)
    subprocess.check_call(cmd)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    build(force=True, verbose="-v" in sys.argv)
    print(LIB)
