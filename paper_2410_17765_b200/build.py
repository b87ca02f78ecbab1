"""In-tree build of libcpmtp.so for sm_100a with nvcc (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(PKG_DIR, "csrc")
LIB_PATH = os.path.join(PKG_DIR, "libcpmtp.so")
DEBUG_LIB_PATH = os.path.join(PKG_DIR, "libcpmtp_debug.so")   # the same sources with -DCPMTP_DEBUG (index checks)
SOURCES = ["cpmtp_api.cu"]
HEADERS = ["ptx.cuh", "tmap.cuh", "tc_gemm.cuh", "epilogues.cuh", "small_kernels.cuh", "sampler_kernels.cuh",
           "distill_epilogues.cuh", "distill_kernels.cuh"]


def _nvcc() -> str:
    for cand in (shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found")


def is_stale(lib_path: str = LIB_PATH) -> bool:
    if not os.path.exists(lib_path):
        return True
    built = os.path.getmtime(lib_path)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS]
    deps.append(os.path.join(os.path.dirname(PKG_DIR), "include", "cpmtp.h"))
    return any(os.path.getmtime(p) > built for p in deps)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Compile the library if it is missing or older than its sources; return its path.  `debug` builds the
    checked variant (every epilogue store and gather compares its index with the buffer extent first)."""
    lib_path = DEBUG_LIB_PATH if debug else LIB_PATH
    if not force and not is_stale(lib_path):
        return lib_path
    cmd = [
        _nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
        "-shared", "-Xcompiler", "-fPIC",
    ]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    if debug:
        cmd += ["-DCPMTP_DEBUG"]
    cmd += [os.path.join(CSRC, s) for s in SOURCES] + ["-o", lib_path]
    proc = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or proc.returncode != 0:
        sys.stderr.write(proc.stdout + proc.stderr)
    if proc.returncode != 0:
        raise RuntimeError(f"nvcc failed building {os.path.basename(lib_path)}")
    return lib_path


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
