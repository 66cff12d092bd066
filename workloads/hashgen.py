"""ctypes front end of the seeded input generator in ``hashgen.c``.

Inputs only (initial models, gradients, row masks, dtype storage conversion); no HPSGD
arithmetic lives here.  The shared object is compiled with gcc on first use and cached
beside the source.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hashgen.c")
_LIB = os.path.join(_HERE, "libhashgen.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile ``hashgen.c`` into ``libhashgen.so`` (no-op when up to date)."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + ".tmp.%d" % os.getpid()
    cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True, capture_output=True)
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is not None:
            return _lib
        lib = ctypes.CDLL(build())
        u64, i64, f32, f64 = ctypes.c_uint64, ctypes.c_int64, ctypes.c_float, ctypes.c_double
        vp = ctypes.c_void_p
        lib.hg_hash.restype = u64
        lib.hg_hash.argtypes = [u64, u64, u64, u64, u64]
        lib.hg_grad_uniform.restype = None
        lib.hg_grad_uniform.argtypes = [u64, u64, u64, i64, vp, i64, f32, vp]
        lib.hg_grad_gauss.restype = None
        lib.hg_grad_gauss.argtypes = [u64, u64, u64, i64, vp, i64, f64, vp]
        lib.hg_init_global.restype = None
        lib.hg_init_global.argtypes = [u64, i64, vp, i64, vp]
        lib.hg_row_mask.restype = None
        lib.hg_row_mask.argtypes = [u64, u64, u64, i64, vp]
        lib.hg_layout_u.restype = f64
        lib.hg_layout_u.argtypes = [u64, u64]
        lib.hg_f32_to_bf16.restype = None
        lib.hg_f32_to_bf16.argtypes = [vp, i64, vp]
        lib.hg_bf16_to_f32.restype = None
        lib.hg_bf16_to_f32.argtypes = [vp, i64, vp]
        _lib = lib
        return lib


def _idx_args(idx, idx0, n):
    """Return (idx0, pointer-or-None, n, keepalive) for a contiguous range or an index list."""
    if idx is None:
        return int(idx0), None, int(n), None
    a = np.ascontiguousarray(idx, dtype=np.int64)
    if a.size and (a.min() < 0 or a.max() >= 2 ** 32):
        raise ValueError("indices must lie in [0, 2^32)")
    return 0, a.ctypes.data, int(a.size), a


def hash64(seed: int, stream: int, step: int, worker: int, idx: int) -> int:
    """The raw 64-bit hash value h(seed, stream, step, worker, idx)."""
    return int(_load().hg_hash(seed, stream, step, worker, idx))


def grad_uniform(seed, step, worker, *, idx0=0, n=None, idx=None, scale=1e-2) -> np.ndarray:
    """fp32 gradients ``scale * uniform[-1,1)`` over a range ``[idx0, idx0+n)`` or ``idx``."""
    i0, ip, cnt, keep = _idx_args(idx, idx0, n)
    out = np.empty(cnt, dtype=np.float32)
    _load().hg_grad_uniform(seed, step, worker, i0, ip, cnt, scale, out.ctypes.data)
    return out


def grad_gauss(seed, step, worker, *, idx0=0, n=None, idx=None, sigma=1e-3) -> np.ndarray:
    """fp32 gradients N(0, sigma) (sigma is the standard deviation) by Box-Muller."""
    i0, ip, cnt, keep = _idx_args(idx, idx0, n)
    out = np.empty(cnt, dtype=np.float32)
    _load().hg_grad_gauss(seed, step, worker, i0, ip, cnt, sigma, out.ctypes.data)
    return out


def init_global(seed, *, idx0=0, n=None, idx=None) -> np.ndarray:
    """Initial global model, uniform[-0.1, 0.1) in fp32."""
    i0, ip, cnt, keep = _idx_args(idx, idx0, n)
    out = np.empty(cnt, dtype=np.float32)
    _load().hg_init_global(seed, i0, ip, cnt, out.ctypes.data)
    return out


def row_mask(seed, step, worker, rows) -> np.ndarray:
    """Boolean mask of the embedding rows that carry a gradient for (worker, step)."""
    out = np.empty(int(rows), dtype=np.uint8)
    _load().hg_row_mask(seed, step, worker, int(rows), out.ctypes.data)
    return out.astype(bool)


def layout_u(seed, tensor) -> float:
    """53-bit uniform in [0, 1) attached to a tensor number (used to draw tensor sizes)."""
    return float(_load().hg_layout_u(seed, tensor))


def f32_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even storage conversion; returns the bf16 bit patterns (uint16)."""
    a = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty(a.shape, dtype=np.uint16)
    _load().hg_f32_to_bf16(a.ctypes.data, a.size, out.ctypes.data)
    return out


def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to fp32."""
    a = np.ascontiguousarray(bits, dtype=np.uint16)
    out = np.empty(a.shape, dtype=np.float32)
    _load().hg_bf16_to_f32(a.ctypes.data, a.size, out.ctypes.data)
    return out
