"""Builds libpulseinfer_b200.so (sm_100a only) in-tree with nvcc.

    python -m paper_2609_34555_b200.build [--force] [--verbose]
"""
from __future__ import annotations

import os
import subprocess
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent
CSRC = PKG / "csrc"
INCLUDE = PKG.parent / "include"
LIB = PKG / "libpulseinfer_b200.so"

SOURCES = ["pi_api.cu", "pi_score_select.cu", "pi_select_diff.cu", "pi_diff_misses.cu", "pi_recall.cu", "pi_attn.cu", "pi_attn_headmajor.cu",
           "pi_helpers.cu", "pi_append.cu"]


def sources() -> list[Path]:
    return [CSRC / s for s in SOURCES if (CSRC / s).exists()]


def _stale() -> bool:
    if not LIB.exists():
        return True
    t = LIB.stat().st_mtime
    deps = sources() + list(CSRC.glob("*.cuh")) + list(INCLUDE.glob("*.h"))
    return any(d.stat().st_mtime > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> Path:
    if not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = LIB.with_suffix(f".tmp{os.getpid()}.so")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-Xcompiler", "-fPIC", "-shared", f"-I{INCLUDE}", f"-I{CSRC}",
           "-o", str(tmp)] + [str(s) for s in sources()]
    cmd[1:1] = os.environ.get("PI_NVCC_FLAGS", "").split()       # extra flags for experiments (-D..., -Xptxas=-v)
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    subprocess.check_call(cmd)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
