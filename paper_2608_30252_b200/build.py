"""Builds the CUDA library in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import shutil
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB_PATH = os.path.join(HERE, "libmasw.so")
TRACE_LIB_PATH = os.path.join(HERE, "libmasw_trace.so")
SOURCES = ["api.cu", "attend.cu", "prefill.cu", "mem.cu", "accept.cu"]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "--expt-relaxed-constexpr", "-Xcompiler", "-fPIC", "-shared",
]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: the MASW library cannot be built")


def needs_build(lib_path: str = None) -> bool:
    lib_path = lib_path or LIB_PATH
    if not os.path.exists(lib_path):
        return True
    lib_mtime = os.path.getmtime(lib_path)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(HERE, "..", "include", "masw.h")]
    return any(os.path.getmtime(d) > lib_mtime for d in deps)


def build_trace(force: bool = False) -> str:
    """Compile the developer build (-DMASW_TRACE: phase stamps, settable wait limit, droppable tile copy) into
    paper_2608_30252_b200/libmasw_trace.so.  Only `bench.py --timeline` and the give-up test load it."""
    if not force and not needs_build(TRACE_LIB_PATH):
        return TRACE_LIB_PATH
    cmd = [_nvcc(), *NVCC_FLAGS, "-DMASW_TRACE", "-o", TRACE_LIB_PATH] + [os.path.join(CSRC, s) for s in SOURCES]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    return TRACE_LIB_PATH


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile csrc/*.cu into paper_2608_30252_b200/libmasw.so; returns the library path."""
    if not force and not needs_build():
        return LIB_PATH
    cmd = [_nvcc(), *NVCC_FLAGS, "-o", LIB_PATH] + [os.path.join(CSRC, s) for s in SOURCES]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    if verbose:
        print(res.stderr)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force=True, verbose=True))
