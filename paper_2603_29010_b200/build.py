"""Builds libsolgemm.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
_CSRC = os.path.join(_PKG, "csrc")
LIB_PATH = os.path.join(_PKG, "libsolgemm.so")
_SOURCES = ["sg_api.cu"]
_DEPS = ["sg_api.cu", "sg_kernel.cuh", "sg_ptx.cuh", "sg_transpose.cuh", os.path.join(_ROOT, "include", "solgemm.h")]


def _nvcc() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def is_stale() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    built = os.path.getmtime(LIB_PATH)
    return any(os.path.getmtime(os.path.join(_CSRC, d)) > built for d in _DEPS)


def build(force: bool = False, verbose: bool = False, extra_flags=(), out_path: str = LIB_PATH) -> str:
    """Compile the CUDA sources into ``libsolgemm.so`` next to this file and return its path.

    ``extra_flags`` / ``out_path`` build an experimental variant (e.g. ``-DSG_MAX_STAGES=4``) beside the
    product library; ``SOLGEMM_LIB`` makes the binding load it.
    """
    if out_path == LIB_PATH and not extra_flags and not force and not is_stale():
        return LIB_PATH
    tmp = out_path + ".tmp%d" % os.getpid()
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
           "--shared", "-Xcompiler", "-fPIC", "-Xptxas", "-v",
           "-I", os.path.join(_ROOT, "include"), "-I", _CSRC]
    cmd += list(extra_flags) + [os.path.join(_CSRC, s) for s in _SOURCES] + ["-o", tmp]
    proc = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or proc.returncode != 0:
        sys.stderr.write(proc.stdout + proc.stderr)
    if proc.returncode != 0:
        raise RuntimeError("nvcc failed building libsolgemm.so")
    with open(os.path.join(_PKG, "ptxas.log"), "w") as f:
        f.write(proc.stderr)
    os.replace(tmp, out_path)
    return out_path


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
