"""Builds libquoka.so (the C-ABI shared library) in-tree with nvcc for sm_100a.

    python -m paper_2602_08722_b200.build [--force] [--verbose] [--debug]
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libquoka.so")
LIB_DEBUG = os.path.join(PKG, "libquoka_debug.so")
SOURCES = ["quoka_api.cu", "select_queries.cu", "score_keys_simt.cu", "score_keys_tc.cu", "select_keys.cu",
           "attn_simt.cu", "attn_tc.cu", "attn_tc_pair.cu", "no_alloc.cu", "cache_ops.cu", "diagnostics.cu", "decode.cu"]


def _sources():
    return [os.path.join(CSRC, s) for s in SOURCES if os.path.exists(os.path.join(CSRC, s))]


def _stale(LIB: str) -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = _sources() + [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith(".cuh")]
    deps.append(os.path.join(ROOT, "include", "quoka.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Builds libquoka.so, or with debug=True libquoka_debug.so (-DQUOKA_DEBUG: the attention kernel range-checks
    every selected row and page id before it uses them)."""
    if debug:
        return _build(LIB_DEBUG, force, verbose, ["-DQUOKA_DEBUG"])
    return _build(LIB, force, verbose, [])


def _build(LIB: str, force: bool, verbose: bool, extra) -> str:
    if not force and not _stale(LIB):
        return LIB
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(nvcc):
        raise RuntimeError("nvcc not found: cannot build libquoka.so")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
           "-Xcompiler", "-fPIC", "-shared", "--threads", "0",
           "-I", os.path.join(ROOT, "include"), "-I", CSRC, "-o", LIB] + list(extra) + _sources()
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed building libquoka.so")
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, debug="--debug" in sys.argv))
