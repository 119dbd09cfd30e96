"""Builds libsolgemm.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
_CSRC = os.path.join(_PKG, "csrc")
LIB_PATH = os.path.join(_PKG, "libsolgemm.so")
_SOURCES = ["sg_api.cu"] + [f"sg_variant_{v}.cu" for v in range(10)]
_DEPS = _SOURCES + ["sg_kernel.cuh", "sg_ptx.cuh", "sg_transpose.cuh", "sg_gemv.cuh", "sg_splitk.cuh", "sg_variants.h", "sg_variant.inc",
                    os.path.join(_ROOT, "include", "solgemm.h")]


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

    The translation units (the host API and one file per kernel variant) are compiled in parallel and linked.
    ``extra_flags`` / ``out_path`` build an experimental variant (e.g. ``-DSG_MAX_STAGES=4``) beside the
    product library; ``SOLGEMM_LIB`` makes the binding load it.
    """
    if out_path == LIB_PATH and not extra_flags and not force and not is_stale():
        return LIB_PATH
    import shutil
    import tempfile
    from concurrent.futures import ThreadPoolExecutor
    base = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
            "-Xcompiler", "-fPIC", "-Xptxas", "-v", "-I", os.path.join(_ROOT, "include"), "-I", _CSRC] + list(extra_flags)
    work = tempfile.mkdtemp(prefix="solgemm_build_")
    try:
        def compile_one(src):
            obj = os.path.join(work, src.replace(".cu", ".o"))
            return src, obj, subprocess.run(base + ["-c", os.path.join(_CSRC, src), "-o", obj], capture_output=True, text=True)
        with ThreadPoolExecutor(max_workers=len(_SOURCES)) as pool:
            results = list(pool.map(compile_one, _SOURCES))
        log = "".join(f"==== {src}\n{r.stdout}{r.stderr}" for src, _, r in results)
        if verbose or any(r.returncode != 0 for _, _, r in results):
            sys.stderr.write(log)
        if any(r.returncode != 0 for _, _, r in results):
            raise RuntimeError("nvcc failed building libsolgemm.so")
        tmp = out_path + ".tmp%d" % os.getpid()
        link = subprocess.run([_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "--shared", "-Xcompiler", "-fPIC"] +
                              [obj for _, obj, _ in results] + ["-o", tmp], capture_output=True, text=True)
        if link.returncode != 0:
            sys.stderr.write(link.stdout + link.stderr)
            raise RuntimeError("nvcc failed linking libsolgemm.so")
        with open(os.path.join(_PKG, "ptxas.log"), "w") as f:
            f.write(log)
        os.replace(tmp, out_path)
    finally:
        shutil.rmtree(work, ignore_errors=True)
    return out_path


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
