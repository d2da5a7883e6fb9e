"""Compile the 3D-DSA CUDA library for sm_100a into libdsa3d.so next to this file."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libdsa3d.so")
LIB_DEBUG = os.path.join(HERE, "libdsa3d_debug.so")     # the checked build (-DDSA3D_DEBUG)
SOURCES = ["dsa3d_api.cu", "dsa3d_forward.cu", "dsa3d_backward.cu", "dsa3d_backward_blocks.cu", "dsa3d_noalloc.cu", "dsa3d_probes.cu",
           "dsa3d_producer.cu", "dsa3d_fixed_window.cu", "dsa3d_fixed_window_planes.cu", "dsa3d_fixed_window_tables.cu",
           "dsa3d_fixed_window_backward.cu", "dsa3d_fixed_window_tile_grad.cu",
           "dsa3d_fixed_window_planes_grad.cu", "dsa3d_bounded_offsets_backward.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
              "-Xcompiler", "-fPIC"]


def _nvcc() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def _stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    built = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + \
           [os.path.join(os.path.dirname(HERE), "include", "dsa3d.h")]
    return any(os.path.getmtime(p) > built for p in deps)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Build libdsa3d.so (or, with debug=True, the bounds-checked libdsa3d_debug.so) if it is missing
    or older than its sources; return its path."""
    lib = LIB_DEBUG if debug else LIB
    if not force and not _stale(lib):
        return lib
    flags = list(NVCC_FLAGS) + os.environ.get("DSA3D_NVCC_EXTRA", "").split() + (["-DDSA3D_DEBUG"] if debug else [])
    if verbose:
        flags += ["-Xptxas", "-v"]
    cmd = [_nvcc(), "-shared", "-o", lib] + flags + [os.path.join(CSRC, s) for s in SOURCES]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose:
        sys.stderr.write(res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    return lib


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
