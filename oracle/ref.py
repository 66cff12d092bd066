"""ctypes front end of the CPU oracle ``hpsgd_ref.cpp``.

TEST INFRASTRUCTURE ONLY: imported by tests, the smoke check and the CPU-baseline legs
of the benchmark; never by the CUDA package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hpsgd_ref.cpp")
_LIB = os.path.join(_HERE, "libhpsgd_ref.so")
# One IEEE operation per written operation: no contraction, no fast-math; -mfma only
# makes std::fmaf a hardware instruction instead of a (bit-identical) software routine.
CXXFLAGS = ["-O2", "-std=c++17", "-ffp-contract=off", "-fno-fast-math", "-mfma", "-fPIC", "-shared"]
_lib = None


def build(force: bool = False, extra_flags=(), out: str | None = None) -> str:
    """Compile the oracle (no-op when up to date); ``extra_flags``/``out`` serve mutant builds."""
    lib = out or _LIB
    if (not force and os.path.exists(lib)
            and os.path.getmtime(lib) >= os.path.getmtime(_SRC)):
        return lib
    tmp = lib + ".tmp.%d" % os.getpid()
    subprocess.run(["g++", *CXXFLAGS, *extra_flags, "-o", tmp, _SRC], check=True, capture_output=True)
    os.replace(tmp, lib)
    return lib


def _bind(lib):
    i64, f32, vp, ci = ctypes.c_int64, ctypes.c_float, ctypes.c_void_p, ctypes.c_int
    lib.ref_create.restype = vp
    lib.ref_create.argtypes = [i64, ci, f32, f32, f32, ci]
    lib.ref_destroy.restype = None
    lib.ref_destroy.argtypes = [vp]
    lib.ref_set_global.restype = None
    lib.ref_set_global.argtypes = [vp, vp]
    lib.ref_local_step.restype = ci
    lib.ref_local_step.argtypes = [vp, ci, vp]
    lib.ref_local_step_bf16.restype = ci
    lib.ref_local_step_bf16.argtypes = [vp, ci, vp]
    lib.ref_local_step_sparse.restype = ci
    lib.ref_local_step_sparse.argtypes = [vp, ci, vp, ci, i64, i64, i64, vp, ctypes.c_int32, vp]
    lib.ref_sync_merge.restype = None
    lib.ref_sync_merge.argtypes = [vp]
    for name in ("ref_get_global", "ref_get_pending"):
        getattr(lib, name).restype = ctypes.POINTER(ctypes.c_float)
        getattr(lib, name).argtypes = [vp]
    for name in ("ref_get_replica", "ref_get_momentum"):
        getattr(lib, name).restype = ctypes.POINTER(ctypes.c_float)
        getattr(lib, name).argtypes = [vp, ci]
    lib.ref_merges.restype = i64
    lib.ref_merges.argtypes = [vp]
    lib.ref_acc_create.restype = vp
    lib.ref_acc_create.argtypes = [i64, ci, f32]
    lib.ref_acc_destroy.restype = None
    lib.ref_acc_destroy.argtypes = [vp]
    lib.ref_acc_set_global.restype = None
    lib.ref_acc_set_global.argtypes = [vp, vp]
    lib.ref_acc_local_step.restype = ci
    lib.ref_acc_local_step.argtypes = [vp, ci, vp]
    lib.ref_acc_sync.restype = None
    lib.ref_acc_sync.argtypes = [vp]
    for name in ("ref_acc_get_global", "ref_acc_get_synced"):
        getattr(lib, name).restype = ctypes.POINTER(ctypes.c_float)
        getattr(lib, name).argtypes = [vp]
    for name in ("ref_acc_get_replica", "ref_acc_get_accumulated"):
        getattr(lib, name).restype = ctypes.POINTER(ctypes.c_float)
        getattr(lib, name).argtypes = [vp, ci]
    return lib


def load(path: str | None = None):
    global _lib
    if path is not None:
        return _bind(ctypes.CDLL(path))
    if _lib is None:
        _lib = _bind(ctypes.CDLL(build()))
    return _lib


class RefHPSGD:
    """K replicas of a P-element model, stepped and merged by the oracle."""

    def __init__(self, P, K, lr, momentum=0.0, weight_decay=0.0, staleness=1, lib=None):
        self._lib = lib or load()
        self.P, self.K = int(P), int(K)
        self._h = self._lib.ref_create(self.P, self.K, lr, momentum, weight_decay, staleness)
        if not self._h:
            raise ValueError("ref_create rejected the arguments")

    def close(self):
        if self._h:
            self._lib.ref_destroy(self._h)
            self._h = None

    def __del__(self):
        self.close()

    def set_global(self, w0):
        a = np.ascontiguousarray(w0, dtype=np.float32)
        assert a.size == self.P
        self._lib.ref_set_global(self._h, a.ctypes.data)

    def local_step(self, worker, g):
        """Dense gradient: fp32 array, or uint16 array of bf16 bit patterns."""
        a = np.ascontiguousarray(g)
        assert a.size == self.P
        if a.dtype == np.uint16:
            rc = self._lib.ref_local_step_bf16(self._h, worker, a.ctypes.data)
        else:
            a = np.ascontiguousarray(a, dtype=np.float32)
            rc = self._lib.ref_local_step(self._h, worker, a.ctypes.data)
        if rc:
            raise ValueError("bad worker index")

    def local_step_sparse(self, worker, dense, seg_start, rows, cols, row_idx, row_vals):
        d = np.ascontiguousarray(dense)
        is_bf16 = int(d.dtype == np.uint16)
        if not is_bf16:
            d = np.ascontiguousarray(d, dtype=np.float32)
        v = np.ascontiguousarray(row_vals, dtype=d.dtype)
        ri = np.ascontiguousarray(row_idx, dtype=np.int32)
        assert d.size == self.P and v.size == ri.size * cols
        rc = self._lib.ref_local_step_sparse(self._h, worker, d.ctypes.data, is_bf16, seg_start,
                                             rows, cols, ri.ctypes.data, ri.size, v.ctypes.data)
        if rc:
            raise ValueError("bad sparse-step arguments")

    def sync_merge(self):
        self._lib.ref_sync_merge(self._h)

    def _view(self, ptr):
        return np.ctypeslib.as_array(ptr, shape=(self.P,)).copy()

    def get_global(self):
        return self._view(self._lib.ref_get_global(self._h))

    def get_pending(self):
        return self._view(self._lib.ref_get_pending(self._h))

    def get_replica(self, i):
        return self._view(self._lib.ref_get_replica(self._h, i))

    def get_momentum(self, i):
        return self._view(self._lib.ref_get_momentum(self._h, i))

    @property
    def merges(self):
        return int(self._lib.ref_merges(self._h))


class RefHPSGDAccum:
    """Algorithms 2 and 3 as printed (plain SGD): explicit accumulated gradients per worker."""

    def __init__(self, P, K, lr, lib=None):
        self._lib = lib or load()
        self.P, self.K = int(P), int(K)
        self._h = self._lib.ref_acc_create(self.P, self.K, lr)
        if not self._h:
            raise ValueError("ref_acc_create rejected the arguments")

    def close(self):
        if self._h:
            self._lib.ref_acc_destroy(self._h)
            self._h = None

    def __del__(self):
        self.close()

    def set_global(self, w0):
        a = np.ascontiguousarray(w0, dtype=np.float32)
        assert a.size == self.P
        self._lib.ref_acc_set_global(self._h, a.ctypes.data)

    def local_step(self, worker, g):
        a = np.ascontiguousarray(g, dtype=np.float32)
        assert a.size == self.P
        if self._lib.ref_acc_local_step(self._h, worker, a.ctypes.data):
            raise ValueError("bad worker index")

    def sync_merge(self):
        self._lib.ref_acc_sync(self._h)

    def _view(self, ptr):
        return np.ctypeslib.as_array(ptr, shape=(self.P,)).copy()

    def get_global(self):
        return self._view(self._lib.ref_acc_get_global(self._h))

    def get_synced(self):
        return self._view(self._lib.ref_acc_get_synced(self._h))

    def get_replica(self, i):
        return self._view(self._lib.ref_acc_get_replica(self._h, i))

    def get_accumulated(self, i):
        return self._view(self._lib.ref_acc_get_accumulated(self._h, i))
