"""Builds the C-ABI CUDA library in-tree: ``paper_2604_24273_b200/libbitrl.so`` (sm_100a only)."""
from __future__ import annotations

import os
import subprocess
import sys
from pathlib import Path

HERE = Path(__file__).resolve().parent
CSRC = HERE / "csrc"
LIB = HERE / "libbitrl.so"
SOURCES = [CSRC / "bitrl.cu"]
DEPS = sorted(CSRC.glob("*.cu*")) + [HERE.parent / "include" / "bitrl.h"]


def nvcc_path() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    return "nvcc"


def build(force: bool = False, verbose: bool = False) -> Path:
    if not force and LIB.exists() and all(LIB.stat().st_mtime >= d.stat().st_mtime for d in DEPS):
        return LIB
    tmp = LIB.with_suffix(f".{os.getpid()}.tmp")
    cmd = [nvcc_path(), "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
           "-shared", "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "--fmad=false",
           "-cudart", "static", "-Xlinker", "--exclude-libs,ALL", "-Xlinker", "-Bsymbolic"]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += os.environ.get("BITRL_NVCC_FLAGS", "").split()  # tuning builds, e.g. -DGM_MAXREG=128
    cmd += [str(s) for s in SOURCES] + ["-o", str(tmp)]
    subprocess.check_call(cmd)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
