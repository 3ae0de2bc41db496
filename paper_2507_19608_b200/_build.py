"""Builds libdelta_attn.so (sm_100a) in-tree with nvcc.  No JIT cache, no torch extension:
the library has a plain C ABI and is loaded with ctypes."""
from __future__ import annotations

import os
import shutil
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libdelta_attn.so")
LIB_DEBUG = os.path.join(HERE, "libdelta_attn_dbg.so")      # the same sources with -DDELTA_DEBUG_BOUNDS
SOURCES = ["api.cu", "k1_delta_construct.cu", "k2_hybrid_attn_generic.cu", "k2_hybrid_attn_tc.cu", "k2_hybrid_attn_tcq.cu",
           "k3_decode_step.cu", "k3_decode_step_tc.cu", "k3_decode_step_key.cu", "k3_decode_step_keypacked.cu", "decode_noalloc.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "--shared", "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden",
              "-DDELTA_BUILDING_LIB", "-lcuda"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: the delta-attention library cannot be built")


def _stale(lib: str) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    deps.append(os.path.join(os.path.dirname(HERE), "include", "delta_attn.h"))
    deps.append(os.path.abspath(__file__))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, debug_bounds: bool = False) -> str:
    """Compile the library if it is missing or older than its sources; returns its path.
    debug_bounds: the bounds-checking build (libdelta_attn_dbg.so, -DDELTA_DEBUG_BOUNDS)."""
    lib = LIB_DEBUG if debug_bounds else LIB
    if not force and not _stale(lib):
        return lib
    flags = NVCC_FLAGS + (["-DDELTA_DEBUG_BOUNDS"] if debug_bounds else [])
    cmd = [_nvcc(), *flags, "-o", lib + ".tmp", *[os.path.join(CSRC, s) for s in SOURCES]]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + r.stdout + r.stderr)
    os.replace(lib + ".tmp", lib)
    if verbose:
        print(r.stderr)
    return lib


if __name__ == "__main__":
    import sys
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug_bounds="--debug-bounds" in sys.argv))
