"""Builds the CUDA library (libmlora.so) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG_DIR)
LIB_PATH = os.path.join(PKG_DIR, "libmlora.so")
SOURCES = [os.path.join(PKG_DIR, "csrc", "mlora_api.cu"), os.path.join(PKG_DIR, "csrc", "sched.cpp")]
HEADERS = [os.path.join(PKG_DIR, "csrc", f) for f in
           ("plan.h", "ptx.cuh", "dropout.cuh", "gemm_tcgen05.cuh", "gemm2_tcgen05.cuh", "skinny.cuh", "grad_tc.cuh", "shrink_tc.cuh", "simt.cuh", "glue.cuh", "attention.cuh", "attention_tc.cuh")] + \
          [os.path.join(ROOT, "include", f) for f in ("mlora.h", "mlora_sched.h", "mlora_layer_ops.h")]


def nvcc_path() -> str:
    for cand in (shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: the CUDA library cannot be built")


def is_stale() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    return any(os.path.getmtime(p) > t for p in SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile csrc/ into libmlora.so (skipped when the library is newer than its sources)."""
    if not force and not is_stale():
        return LIB_PATH
    cmd = [nvcc_path(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"),
           "-I", os.path.join(PKG_DIR, "csrc")]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += SOURCES + ["-o", LIB_PATH]
    proc = subprocess.run(cmd, capture_output=True, text=True)
    if verbose:
        sys.stderr.write(proc.stderr)
    if proc.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + proc.stdout + proc.stderr)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
