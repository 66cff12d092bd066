"""Thin ctypes binding of ``libhpsgd.so``: same names as the C ABI, argument marshalling
only.  Every step of the path runs in the library's CUDA kernels; there is no fallback.
See ``include/hpsgd.h`` for the contract of each call.
"""
from __future__ import annotations

import ctypes
import os

HERE = os.path.dirname(os.path.abspath(__file__))
# HPSGD_LIBRARY names another build of the same library (the checked build, a tuning variant)
LIB_PATH = os.environ.get("HPSGD_LIBRARY") or os.path.join(HERE, "libhpsgd.so")

HPSGD_OK = 0
HPSGD_E_BADARG, HPSGD_E_STATE, HPSGD_E_NOMEM = -1, -2, -3
HPSGD_E_CUDA, HPSGD_E_TIMEOUT, HPSGD_E_UNSUPPORTED = -4, -5, -6
HPSGD_OPT_WEIGHT_DECAY, HPSGD_OPT_STALENESS, HPSGD_OPT_GRAD_DTYPE = 1, 2, 3
HPSGD_OPT_OVERLAP, HPSGD_OPT_CHUNKS, HPSGD_OPT_PROFILE, HPSGD_OPT_FUSE = 4, 5, 6, 7
HPSGD_OPT_DEBUG_GROUP_LIMIT = 8
HPSGD_OPT_STAGING = 9
HPSGD_OPT_DEBUG_STAGE_STALL = 10
HPSGD_KERNEL_LOCAL_STEP, HPSGD_KERNEL_MERGE, HPSGD_KERNEL_MERGE_STEP, HPSGD_KERNEL_ROUND = 0, 1, 2, 3
HPSGD_KERNEL_MERGE_STAGED = 4
HPSGD_F32, HPSGD_BF16 = 0, 1
HPSGD_GEN_UNIFORM, HPSGD_GEN_GAUSS = 0, 1
HPSGD_ARENA_MOMENTUM = 1
HPSGD_ARENA_PIPELINE = 2
HPSGD_FORM_REPLICA_CHANGE, HPSGD_FORM_GRADIENT_ACCUMULATION = 0, 1
HPSGD_NOALLOC_MAX_ROWS = 262144


class hpsgd_grad_desc(ctypes.Structure):
    _fields_ = [("dense", ctypes.c_void_p), ("row_idx", ctypes.c_void_p),
                ("n_rows", ctypes.c_int32), ("row_vals", ctypes.c_void_p)]


class HpsgdError(RuntimeError):
    def __init__(self, code, text):
        super().__init__("hpsgd status %d: %s" % (code, text))
        self.code = code


_i64, _u64, _ci, _f32, _f64 = ctypes.c_int64, ctypes.c_uint64, ctypes.c_int, ctypes.c_float, ctypes.c_double
_vp, _sz = ctypes.c_void_p, ctypes.c_size_t
_P = ctypes.POINTER

# name -> (restype, argtypes); must list every symbol declared in include/hpsgd.h
SIGNATURES = {
    "hpsgd_init": (_ci, [_i64, _ci, _f32, _f32, _u64]),
    "hpsgd_local_step": (_ci, [_ci, _vp]),
    "hpsgd_sync_merge": (_ci, []),
    "hpsgd_get_global": (_vp, []),
    "hpsgd_layout_padded": (_i64, [_ci, _P(_i64), _P(_i64)]),
    "hpsgd_set_layout": (_ci, [_ci, _P(_i64)]),
    "hpsgd_set_form": (_ci, [_ci]),
    "hpsgd_set_pipeline": (_ci, [_ci]),
    "hpsgd_arena_bytes": (_sz, [_i64, _ci, _ci, _i64]),
    "hpsgd_bind": (_ci, [_vp, _sz, _vp, _vp]),
    "hpsgd_set_option": (_ci, [_ci, _f64]),
    "hpsgd_set_sparse_segment": (_ci, [_ci, _i64, _i64]),
    "hpsgd_local_step_ex": (_ci, [_ci, _P(hpsgd_grad_desc)]),
    "hpsgd_local_step_all": (_ci, [_vp, _i64]),
    "hpsgd_local_step_all_ex": (_ci, [_P(hpsgd_grad_desc)]),
    "hpsgd_local_step_sparse_noalloc": (_ci, [_vp, _vp, _i64, _P(hpsgd_grad_desc), _ci, _i64, _i64, _i64,
                                              _f32, _f32, _f32, _vp]),
    "hpsgd_local_step_host": (_ci, [_ci, _vp]),
    "hpsgd_set_global_host": (_ci, [_vp, _i64]),
    "hpsgd_fill_global": (_ci, [_u64]),
    "hpsgd_copy_global": (_ci, [_vp, _i64]),
    "hpsgd_copy_global_async": (_ci, [_vp, _i64]),
    "hpsgd_get_replica": (_ci, [_ci, _P(_vp), _P(_vp)]),
    "hpsgd_get_pending": (_ci, [_P(_vp)]),
    "hpsgd_state_bytes": (_sz, []),
    "hpsgd_export_state": (_ci, [_vp, _sz]),
    "hpsgd_import_state": (_ci, [_vp, _sz]),
    "hpsgd_get_sizes": (_ci, [_P(_i64), _P(_i64), _P(_ci), _P(_i64)]),
    "hpsgd_tensor_offset": (_i64, [_ci]),
    "hpsgd_gen_grads": (_ci, [_vp, _ci, _ci, _ci, _f64]),
    "hpsgd_gen_row_vals": (_ci, [_vp, _ci, _ci, _ci, _f64, _vp, ctypes.c_int32]),
    "hpsgd_synchronize": (_ci, []),
    "hpsgd_profile_read": (_ci, [_ci, _P(_f64), _P(_i64)]),
    "hpsgd_probe_hbm": (_ci, [_vp, _sz, _ci, _ci, _i64, _ci, _P(_f64)]),
    "hpsgd_flush": (_ci, []),
    "hpsgd_launch_count": (_i64, []),
    "hpsgd_last_error": (ctypes.c_char_p, []),
    "hpsgd_destroy": (_ci, []),
}

_lib = None


def use_library(path=None):
    """Point the binding at another build of the library (the checked build, say); None = the
    in-tree one.  Call hpsgd_destroy() first: each loaded library has its own state."""
    global _lib, LIB_PATH
    _lib = None
    LIB_PATH = os.path.join(HERE, "libhpsgd.so") if path is None else str(path)


def load():
    """Load the CUDA library; raises if it has not been built (there is no other path)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError("%s is missing: build it with paper_2009_02701_b200.build.build(); "
                              "there is no non-CUDA implementation" % LIB_PATH)
        lib = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


def last_error() -> str:
    return load().hpsgd_last_error().decode()


def _check(rc):
    if rc < 0:
        raise HpsgdError(rc, last_error())
    return rc


def _ptr(x):
    """Device/host address of a torch tensor, numpy array, int, or None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    if hasattr(x, "ctypes"):
        return x.ctypes.data
    raise TypeError("cannot take the address of %r" % type(x))


def _stream(s):
    if s is None:
        return None
    return s.cuda_stream if hasattr(s, "cuda_stream") else int(s)


# ---- the four core calls -------------------------------------------------------------
def hpsgd_init(P, K, lr, momentum, seed):
    return _check(load().hpsgd_init(int(P), int(K), float(lr), float(momentum), int(seed)))


def hpsgd_local_step(worker, grads):
    return _check(load().hpsgd_local_step(int(worker), _ptr(grads)))


def hpsgd_sync_merge():
    return _check(load().hpsgd_sync_merge())


def hpsgd_get_global():
    """Device address of w (int); raises on error."""
    p = load().hpsgd_get_global()
    if not p:
        raise HpsgdError(HPSGD_E_STATE, last_error())
    return p


# ---- layout, memory, options ---------------------------------------------------------
def hpsgd_layout_padded(sizes):
    """Returns (P_pad, offsets)."""
    n = len(sizes)
    arr = (_i64 * n)(*[int(s) for s in sizes])
    off = (_i64 * n)()
    pad = load().hpsgd_layout_padded(n, arr, off)
    _check(pad)
    return int(pad), list(off)


def hpsgd_set_layout(sizes):
    n = len(sizes)
    return _check(load().hpsgd_set_layout(n, (_i64 * n)(*[int(s) for s in sizes])))


def hpsgd_set_form(form):
    return _check(load().hpsgd_set_form(int(form)))


def hpsgd_set_pipeline(enable):
    return _check(load().hpsgd_set_pipeline(int(enable)))


def hpsgd_arena_bytes(P_pad, K, flags=0, sparse_rows=0):
    return int(load().hpsgd_arena_bytes(int(P_pad), int(K), int(flags), int(sparse_rows)))


def hpsgd_bind(arena, nbytes, main_stream, side_stream):
    return _check(load().hpsgd_bind(_ptr(arena), int(nbytes), _stream(main_stream), _stream(side_stream)))


def hpsgd_set_option(key, value):
    return _check(load().hpsgd_set_option(int(key), float(value)))


def hpsgd_set_sparse_segment(tensor_id, rows, cols):
    return _check(load().hpsgd_set_sparse_segment(int(tensor_id), int(rows), int(cols)))


# ---- batched / sparse / host local steps ---------------------------------------------
def make_desc(dense, row_idx=None, n_rows=0, row_vals=None):
    return hpsgd_grad_desc(_ptr(dense), _ptr(row_idx), int(n_rows), _ptr(row_vals))


def hpsgd_local_step_ex(worker, desc):
    return _check(load().hpsgd_local_step_ex(int(worker), ctypes.byref(desc)))


def hpsgd_local_step_all(grads, worker_stride_bytes):
    return _check(load().hpsgd_local_step_all(_ptr(grads), int(worker_stride_bytes)))


def hpsgd_local_step_all_ex(descs):
    arr = (hpsgd_grad_desc * len(descs))(*descs)
    return _check(load().hpsgd_local_step_all_ex(arr))


def hpsgd_local_step_sparse_noalloc(replica, momentum_buf, n_elems, desc, grad_dtype, seg_offset, rows, cols,
                                    lr, momentum, weight_decay, stream=None):
    """Sparse-row local step on caller-owned buffers; allocates nothing (see hpsgd.h)."""
    return _check(load().hpsgd_local_step_sparse_noalloc(
        _ptr(replica), _ptr(momentum_buf), int(n_elems), ctypes.byref(desc), int(grad_dtype),
        int(seg_offset), int(rows), int(cols), float(lr), float(momentum), float(weight_decay),
        _stream(stream)))


def hpsgd_local_step_host(worker, host_grads):
    return _check(load().hpsgd_local_step_host(int(worker), _ptr(host_grads)))


def _count(x):
    """Number of elements of a numpy array or torch tensor."""
    return int(x.numel()) if hasattr(x, "numel") else int(x.size)


def hpsgd_set_global_host(host_w):
    return _check(load().hpsgd_set_global_host(_ptr(host_w), _count(host_w)))


def hpsgd_fill_global(seed):
    return _check(load().hpsgd_fill_global(int(seed)))


def hpsgd_copy_global(host_out):
    return _check(load().hpsgd_copy_global(_ptr(host_out), _count(host_out)))


def hpsgd_copy_global_async(host_out):
    return _check(load().hpsgd_copy_global_async(_ptr(host_out), _count(host_out)))


# ---- inspection ----------------------------------------------------------------------
def hpsgd_get_replica(worker):
    """Returns (address of r_worker, address of m_worker or None)."""
    r, m = _vp(), _vp()
    _check(load().hpsgd_get_replica(int(worker), ctypes.byref(r), ctypes.byref(m)))
    return r.value, m.value


def hpsgd_get_pending():
    d = _vp()
    _check(load().hpsgd_get_pending(ctypes.byref(d)))
    return d.value


def hpsgd_state_bytes():
    return int(load().hpsgd_state_bytes())


def hpsgd_export_state(host_buf):
    """host_buf: a writable host buffer (e.g. numpy uint8 array) of hpsgd_state_bytes() bytes."""
    return _check(load().hpsgd_export_state(_ptr(host_buf), int(host_buf.nbytes)))


def hpsgd_import_state(host_buf):
    return _check(load().hpsgd_import_state(_ptr(host_buf), int(host_buf.nbytes)))


def hpsgd_get_sizes():
    """Returns (P, P_pad, K, merges)."""
    P, Pp, K, s = _i64(), _i64(), _ci(), _i64()
    _check(load().hpsgd_get_sizes(ctypes.byref(P), ctypes.byref(Pp), ctypes.byref(K), ctypes.byref(s)))
    return P.value, Pp.value, K.value, s.value


def hpsgd_tensor_offset(tensor_id):
    return int(_check(load().hpsgd_tensor_offset(int(tensor_id))))


# ---- generators, housekeeping ----------------------------------------------------------
def hpsgd_gen_grads(out, worker, step, kind, scale):
    return _check(load().hpsgd_gen_grads(_ptr(out), int(worker), int(step), int(kind), float(scale)))


def hpsgd_gen_row_vals(out, worker, step, kind, scale, row_idx, n_rows):
    return _check(load().hpsgd_gen_row_vals(_ptr(out), int(worker), int(step), int(kind), float(scale),
                                            _ptr(row_idx), int(n_rows)))


def hpsgd_synchronize():
    return _check(load().hpsgd_synchronize())


def hpsgd_profile_read(kind):
    """Returns (milliseconds, launches) of one kernel kind since its last read."""
    ms, n = _f64(), _i64()
    _check(load().hpsgd_profile_read(int(kind), ctypes.byref(ms), ctypes.byref(n)))
    return ms.value, n.value


def hpsgd_probe_hbm(scratch, scratch_bytes, n_read, n_write, row_bytes, iters):
    """GB/s (1e9 bytes/s) of a kernel that only reads n_read and writes n_write arrays of row_bytes."""
    out = _f64()
    _check(load().hpsgd_probe_hbm(_ptr(scratch), int(scratch_bytes), int(n_read), int(n_write), int(row_bytes),
                                  int(iters), ctypes.byref(out)))
    return out.value


def hpsgd_flush():
    return _check(load().hpsgd_flush())


def hpsgd_launch_count():
    return int(load().hpsgd_launch_count())


def hpsgd_destroy():
    return _check(load().hpsgd_destroy())
