"""Build ``libhpsgd.so`` (CUDA, sm_100a only) in-tree with nvcc."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libhpsgd.so")
SOURCES = [os.path.join(CSRC, "hpsgd_api.cu")]
DEPENDS = SOURCES + [os.path.join(CSRC, "hpsgd_kernels.cuh"), os.path.join(CSRC, "hpsgd_state.cuh"),
                     os.path.join(CSRC, "hpsgd_schedule.cuh"), os.path.join(CSRC, "hpsgd_staged.cuh"),
                     os.path.join(os.path.dirname(HERE), "include", "hpsgd.h")]
# --fmad=false: the compiler never contracts a*b+c on its own; fused multiply-adds are
# written explicitly where the update rule has them.
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "--fmad=false", "-Xcompiler", "-fPIC", "-shared", "-cudart", "static"]


def nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    raise RuntimeError("nvcc not found")


def build(force: bool = False, verbose: bool = False, debug: bool = False, out: str | None = None) -> str:
    """Compile the library if it is missing or older than its sources; returns its path.

    ``debug`` builds the checked variant (-DHPSGD_DEBUG: kernel guards that record and skip an
    out-of-range access, host-side validation of sparse row lists) into ``out`` (default
    ``libhpsgd_debug.so`` beside the normal library)."""
    lib = out or (os.path.join(HERE, "libhpsgd_debug.so") if debug else LIB)
    if not force and os.path.exists(lib):
        newest = max(os.path.getmtime(p) for p in DEPENDS)
        if os.path.getmtime(lib) >= newest:
            return lib
    tmp = lib + ".tmp.%d" % os.getpid()
    cmd = [nvcc(), *NVCC_FLAGS, *(["-DHPSGD_DEBUG"] if debug else []), *(["-Xptxas", "-v"] if verbose else []),
           "-o", tmp, *SOURCES]
    proc = subprocess.run(cmd, capture_output=True, text=True)
    if proc.returncode != 0:
        raise RuntimeError("nvcc failed:\n%s\n%s" % (proc.stdout, proc.stderr))
    if verbose:
        sys.stderr.write(proc.stderr)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
