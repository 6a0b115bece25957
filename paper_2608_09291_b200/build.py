"""Builds the C-ABI shared library (in-tree) with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent
CSRC = PKG / "csrc"
LIB = PKG / "libunionsparse.so"
SOURCES = [CSRC / "us_api.cu", CSRC / "us_encode.cpp"]
HEADERS = [CSRC / "us_host.h", CSRC / "us_spmm_kernel.cuh", CSRC / "us_quant_kernels.cuh", PKG.parent / "include" / "unionsparse.h"]


def nvcc_command(out: Path, verbose: bool = False) -> list[str]:
    cmd = ["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-Xcompiler", "-fPIC,-O3,-Wall", "-shared", "-cudart", "shared"]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += os.environ.get("US_NVCC_FLAGS", "").split()
    return cmd + [str(s) for s in SOURCES] + ["-o", str(out)]


def is_stale() -> bool:
    if not LIB.exists():
        return True
    t = LIB.stat().st_mtime
    return any(p.stat().st_mtime > t for p in SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False) -> Path:
    if force or verbose or is_stale():
        tmp = LIB.with_suffix(f".tmp{os.getpid()}.so")
        r = subprocess.run(nvcc_command(tmp, verbose), capture_output=True, text=True)
        if verbose:
            sys.stderr.write(r.stderr)
        if r.returncode != 0:
            raise RuntimeError("nvcc failed:\n" + r.stdout + r.stderr)
        os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    build(force=True, verbose="-v" in sys.argv)
    print(LIB)
