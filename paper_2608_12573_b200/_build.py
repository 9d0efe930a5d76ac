"""In-tree build of the CUDA library: nvcc -> paper_2608_12573_b200/libprofk.so (sm_100a only)."""
from __future__ import annotations

import os
import subprocess
import sys

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG_DIR)
CSRC = os.path.join(PKG_DIR, "csrc")
LIB_PATH = os.path.join(PKG_DIR, "libprofk.so")
SOURCES = ["profk_api.cu", "plan.cpp"]


def _newest_source_mtime() -> float:
    paths = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(ROOT, "include", "profk.h")]
    return max(os.path.getmtime(p) for p in paths)


def nvcc_command(extra: list[str] | None = None) -> list[str]:
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
           "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(ROOT, "include"), "-I", CSRC,
           "-o", LIB_PATH] + [os.path.join(CSRC, s) for s in SOURCES]
    return cmd + (extra or []) + os.environ.get("PROFK_NVCC_FLAGS", "").split()


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile the library unless an up-to-date one is already in the tree; returns its path."""
    if not force and os.path.exists(LIB_PATH) and os.path.getmtime(LIB_PATH) >= _newest_source_mtime():
        return LIB_PATH
    cmd = nvcc_command(["-Xptxas", "-v"] if verbose else None)
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError("nvcc failed building libprofk.so")
    if verbose:
        sys.stderr.write(res.stdout + res.stderr)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
