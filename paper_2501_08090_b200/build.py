"""Compile the CUDA library in-tree for sm_100a with nvcc (no JIT cache, no other arch)."""
from __future__ import annotations

import os
import shutil
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_HERE)
CSRC = os.path.join(_HERE, "csrc")
SOURCES = [os.path.join(CSRC, "ckv_api.cu"), os.path.join(CSRC, "ckv_autoscaler.cc"),
           os.path.join(CSRC, "ckv_global_sim.cc")]
HEADERS = [os.path.join(CSRC, "ckv_device.cuh"), os.path.join(_ROOT, "include", "chiron_kv.h"),
           os.path.join(_ROOT, "include", "chiron_autoscaler.h")]
LIBRARY = os.path.join(_HERE, "libchiron_kv.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-O3", "-std=c++17", "-lineinfo",
    "-Xcompiler", "-fPIC", "-shared", "-cudart", "static",
    "-I", os.path.join(_ROOT, "include"), "-I", CSRC,
]


def _nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found; the CUDA library cannot be built")
    return exe


def is_stale() -> bool:
    if not os.path.exists(LIBRARY):
        return True
    built = os.path.getmtime(LIBRARY)
    return any(os.path.getmtime(p) > built for p in SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False) -> str:
    """Build libchiron_kv.so if missing or older than its sources; return its path."""
    if force or is_stale():
        tmp = LIBRARY + ".tmp.%d" % os.getpid()
        cmd = [_nvcc()] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp] + SOURCES
        res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode != 0:
            raise RuntimeError("nvcc failed:\n%s\n%s" % (res.stdout, res.stderr))
        if verbose:
            print(res.stderr)
        os.replace(tmp, LIBRARY)
    return LIBRARY


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv))
