"""Builds ``libghd.so`` (the CUDA kernels and the C-ABI) in-tree for sm_100a."""
from __future__ import annotations

import os
import subprocess
from pathlib import Path

_PKG = Path(__file__).resolve().parent
_CSRC = _PKG / "csrc"
_INC = _PKG.parent / "include"
LIB = _PKG / "libghd.so"

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-shared"]


def sources():
    return sorted(_CSRC.glob("*.cu"))


def is_stale() -> bool:
    if not LIB.exists():
        return True
    deps = list(_CSRC.glob("*")) + list(_INC.glob("*.h"))
    return any(p.stat().st_mtime > LIB.stat().st_mtime for p in deps)


def build(force: bool = False, verbose: bool = False) -> Path:
    """Compile every .cu under csrc/ into libghd.so; no-op when up to date."""
    if not force and not is_stale():
        return LIB
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = LIB.with_suffix(f".tmp{os.getpid()}.so")
    cmd = [nvcc] + NVCC_FLAGS + [f"-I{_INC}", f"-I{_CSRC}"] + (["-Xptxas", "-v"] if verbose else []) + \
          ["-o", str(tmp)] + [str(s) for s in sources()]
    subprocess.check_call(cmd)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose=True))
