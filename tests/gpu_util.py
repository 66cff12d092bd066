"""Helpers for the GPU parity tests: drive libhpsgd (through its C ABI binding) and the CPU
oracle with the same seeded inputs and compare.  Nothing here computes the update rule."""
from __future__ import annotations

import contextlib

import numpy as np
import torch

import paper_2009_02701_b200 as hp
from oracle.ref import RefHPSGD
from workloads import hashgen

DEV = "cuda:0"


class _RawDeviceArray:
    """Exposes a raw device address through the CUDA array interface."""

    def __init__(self, addr, n, typestr):
        self.__cuda_array_interface__ = {"shape": (n,), "typestr": typestr, "data": (int(addr), False),
                                         "version": 2}


def dev_view(addr: int, n: int, typestr="<f4") -> torch.Tensor:
    """Copy n elements starting at a raw device address into a new torch tensor."""
    return torch.as_tensor(_RawDeviceArray(addr, n, typestr), device=DEV).clone()


def dev_tensor(addr: int, n: int, typestr="<f4") -> torch.Tensor:
    """The n elements at a raw device address as a torch tensor that aliases them (no copy)."""
    return torch.as_tensor(_RawDeviceArray(addr, n, typestr), device=DEV)


def to_device(a: np.ndarray) -> torch.Tensor:
    """Upload a numpy array (fp32, or uint16 bf16 bit patterns, or int32)."""
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).to(DEV)
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


@contextlib.contextmanager
def session(cfg, *, staleness=None, overlap=1, chunks=1, fuse=0, form=0, pipeline=0, lend_arena=False, streams=False,
            canary=False, staging=0):
    """hpsgd_init for a workload (layout, options, optional lent arena/streams); destroys on exit."""
    hp.hpsgd_destroy()
    lay = cfg.layout
    keep = {}
    if len(cfg.sizes) > 1:
        hp.hpsgd_set_layout(list(cfg.sizes))
    hp.hpsgd_set_form(form)
    hp.hpsgd_set_pipeline(pipeline)
    if lend_arena or streams:
        arena, nbytes, main, side = None, 0, None, None
        if lend_arena:
            rows = cfg.sparse[1] if cfg.sparse else 0
            flags = (hp.HPSGD_ARENA_MOMENTUM if (cfg.momentum or form) else 0) | (hp.HPSGD_ARENA_PIPELINE if pipeline else 0)
            nbytes = hp.hpsgd_arena_bytes(lay.P_pad, cfg.K, flags, rows)
            guard = 4096 if canary else 0
            buf = torch.full((nbytes + 2 * guard + 256,), 0xA5, dtype=torch.uint8, device=DEV)
            torch.cuda.synchronize()     # the fill runs on torch's stream; the library works on its own
            base = buf.data_ptr() + guard
            base += (-base) % 256
            keep.update(buf=buf, base=base, nbytes=nbytes, guard=guard)
            arena = base
        if streams:
            main, side = torch.cuda.Stream(device=DEV), torch.cuda.Stream(device=DEV)
            keep.update(main=main, side=side)
        hp.hpsgd_bind(arena, nbytes, main, side)
    try:
        hp.hpsgd_init(cfg.P, cfg.K, cfg.lr, cfg.momentum, cfg.seed)
        if cfg.weight_decay:
            hp.hpsgd_set_option(hp.HPSGD_OPT_WEIGHT_DECAY, cfg.weight_decay)
        hp.hpsgd_set_option(hp.HPSGD_OPT_STALENESS, cfg.staleness if staleness is None else staleness)
        hp.hpsgd_set_option(hp.HPSGD_OPT_GRAD_DTYPE, hp.HPSGD_BF16 if cfg.grad_dtype == "bf16" else hp.HPSGD_F32)
        hp.hpsgd_set_option(hp.HPSGD_OPT_OVERLAP, overlap)
        hp.hpsgd_set_option(hp.HPSGD_OPT_CHUNKS, chunks)
        hp.hpsgd_set_option(hp.HPSGD_OPT_FUSE, fuse)
        if staging:
            hp.hpsgd_set_option(hp.HPSGD_OPT_STAGING, staging)
        if cfg.sparse:
            hp.hpsgd_set_sparse_segment(*cfg.sparse)
        yield keep
        hp.hpsgd_synchronize()
        if canary and lend_arena:
            buf, base, nbytes = keep["buf"], keep["base"], keep["nbytes"]
            off = base - buf.data_ptr()
            assert bool((buf[:off] == 0xA5).all()), "bytes before the arena were overwritten"
            assert bool((buf[off + nbytes:] == 0xA5).all()), "bytes after the arena were overwritten"
    finally:
        hp.hpsgd_destroy()


def gpu_global(cfg) -> np.ndarray:
    out = np.empty(cfg.P, dtype=np.float32)
    hp.hpsgd_copy_global(out)
    return out


def gpu_flat(addr, cfg) -> np.ndarray:
    """A flat padded device buffer as the un-padded numpy concatenation (pads checked zero)."""
    padded = dev_view(addr, cfg.layout.P_pad).cpu().numpy()
    is_pad = np.ones(cfg.layout.P_pad, dtype=bool)
    for size, off in zip(cfg.layout.sizes, cfg.layout.offsets):
        is_pad[off:off + size] = False
    assert not padded[is_pad].any(), "a pad element is non-zero"
    return cfg.layout.unpack(padded)


def gpu_state(cfg):
    """(w, D, [r_i], [m_i]) as un-padded numpy arrays, after synchronising."""
    hp.hpsgd_synchronize()
    w = gpu_flat(hp.hpsgd_get_global(), cfg)
    D = gpu_flat(hp.hpsgd_get_pending(), cfg)
    rs, ms = [], []
    for i in range(cfg.K):
        r, m = hp.hpsgd_get_replica(i)
        rs.append(gpu_flat(r, cfg))
        ms.append(gpu_flat(m, cfg) if m else None)      # momentum, or accumulated gradients
    return w, D, rs, ms


def host_inputs(cfg, worker, step):
    """The stored gradient of (worker, step) in both index spaces, plus the sparse rows.

    Returns dict(flat=un-padded stored gradient (fp32 or bf16 bits) with zero rows,
                 padded=the same in the flat padded layout,
                 rows=int32 active rows or None, vals=[n_rows x cols] stored values or None).
    """
    flat = cfg.stored_gradient(worker, step)
    out = {"flat": flat, "padded": cfg.layout.pack(flat), "rows": None, "vals": None}
    if cfg.sparse:
        tid, rows, cols = cfg.sparse
        start = cfg.layout.starts[tid]
        idx = cfg.sparse_rows(worker, step)
        out["rows"] = idx
        out["vals"] = flat[start:start + rows * cols].reshape(rows, cols)[idx].copy()
    return out


def oracle_for(cfg, staleness=None) -> RefHPSGD:
    o = RefHPSGD(cfg.P, cfg.K, cfg.lr, cfg.momentum, cfg.weight_decay,
                 cfg.staleness if staleness is None else staleness)
    o.set_global(cfg.initial_global())
    return o


def oracle_step(o, cfg, worker, inp, sparse_api=True):
    if cfg.sparse and sparse_api:
        tid, rows, cols = cfg.sparse
        dense = inp["flat"].copy()
        start = cfg.layout.starts[tid]
        dense[start:start + rows * cols] = 0x7FC0 if dense.dtype == np.uint16 else np.nan   # must be ignored
        o.local_step_sparse(worker, dense, start, rows, cols, inp["rows"], inp["vals"])
    else:
        o.local_step(worker, inp["flat"])


def gpu_step(cfg, worker, inp, keep, sparse_api=True):
    """Upload one worker's gradient and enqueue its local step; returns tensors to keep alive."""
    g = to_device(inp["padded"])
    keep.append(g)
    if cfg.sparse and sparse_api:
        idx = to_device(inp["rows"])
        vals = to_device(inp["vals"].reshape(-1))
        keep += [idx, vals]
        hp.hpsgd_local_step_ex(worker, hp.make_desc(g, idx, len(inp["rows"]), vals))
    else:
        hp.hpsgd_local_step(worker, g)


def assert_bitwise(got, want, what):
    got = np.ascontiguousarray(got, dtype=np.float32)
    want = np.ascontiguousarray(want, dtype=np.float32)
    same = got.view(np.uint32) == want.view(np.uint32)
    same |= (got == 0) & (want == 0)            # +0 and -0 are the same parameter value
    if not same.all():
        bad = np.flatnonzero(~same)
        j = bad[0]
        raise AssertionError("%s: %d of %d elements differ; first at %d: got %r want %r"
                             % (what, bad.size, got.size, j, got[j], want[j]))


def max_rel_err(got, want, floor=1e-6):
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    return float(np.max(np.abs(got - want) / np.maximum(np.abs(want), floor)))


def run_both(cfg, T, *, staleness=None, overlap=1, chunks=1, fuse=0, pipeline=0, batched=False, steps_per_round=1,
             skip_worker=None, session_kw=None, check_each_round=False):
    """Run T rounds on the GPU and on the oracle with host-generated inputs; compare bitwise."""
    o = oracle_for(cfg, staleness)
    with session(cfg, staleness=staleness, overlap=overlap, chunks=chunks, fuse=fuse, pipeline=pipeline,
                 **(session_kw or {})):
        assert_bitwise(gpu_global(cfg), o.get_global(), "initial global model")
        step = 0
        alive = []
        for t in range(T):
            keep = []
            for h in range(steps_per_round):
                inputs = [host_inputs(cfg, i, step) for i in range(cfg.K)]
                if batched and not cfg.sparse:
                    stacked = np.stack([inp["padded"] for inp in inputs])
                    g = to_device(stacked.reshape(-1))
                    keep.append(g)
                    hp.hpsgd_local_step_all(g, stacked.shape[1] * stacked.itemsize)
                elif batched:
                    descs = []
                    for inp in inputs:
                        g, idx, vals = to_device(inp["padded"]), to_device(inp["rows"]), to_device(inp["vals"].reshape(-1))
                        keep += [g, idx, vals]
                        descs.append(hp.make_desc(g, idx, len(inp["rows"]), vals))
                    hp.hpsgd_local_step_all_ex(descs)
                else:
                    for i, inp in enumerate(inputs):
                        if i != skip_worker:
                            gpu_step(cfg, i, inp, keep)
                for i, inp in enumerate(inputs):
                    if i != skip_worker or batched:
                        oracle_step(o, cfg, i, inp)
                step += 1
            if check_each_round:
                w, D, rs, ms = gpu_state(cfg)
                for i in range(cfg.K):
                    assert_bitwise(rs[i], o.get_replica(i), "replica %d before merge %d" % (i, t))
            hp.hpsgd_sync_merge()
            o.sync_merge()
            if check_each_round:
                w, D, rs, ms = gpu_state(cfg)
                assert_bitwise(w, o.get_global(), "global after merge %d" % t)
                assert_bitwise(D, o.get_pending(), "pending change after merge %d" % t)
            if fuse or pipeline:
                alive.append(keep)          # no synchronise here: keep the merge and the next steps in flight
            else:
                hp.hpsgd_synchronize()
                del keep
        w, D, rs, ms = gpu_state(cfg)
        assert_bitwise(w, o.get_global(), "global model")
        assert_bitwise(D, o.get_pending(), "pending change")
        for i in range(cfg.K):
            assert_bitwise(rs[i], o.get_replica(i), "replica %d" % i)
            if cfg.momentum:
                assert_bitwise(ms[i], o.get_momentum(i), "momentum %d" % i)
        assert_bitwise(gpu_global(cfg), o.get_global(), "hpsgd_copy_global")
        got = w
    want = o.get_global()
    o.close()
    return got, want


def dev_gather(addr: int, n: int, positions: np.ndarray) -> np.ndarray:
    """Elements at `positions` of the n-float device buffer at a raw address."""
    view = torch.as_tensor(_RawDeviceArray(addr, n, "<f4"), device=DEV)
    return view[torch.from_numpy(np.ascontiguousarray(positions, dtype=np.int64)).to(DEV)].cpu().numpy()


def stratified_sample(cfg, n_random=1 << 18, edge=64, seed=12345) -> np.ndarray:
    """Un-padded indices: the first and last `edge` elements of every tensor plus random ones."""
    picks = []
    for size, start in zip(cfg.layout.sizes, cfg.layout.starts):
        e = min(edge, size)
        picks.append(np.arange(start, start + e))
        picks.append(np.arange(start + size - e, start + size))
    rng = np.random.default_rng(seed)
    picks.append(rng.integers(0, cfg.P, size=n_random))
    return np.unique(np.concatenate(picks)).astype(np.int64)


def run_both_accum(cfg, T, *, staleness=1, overlap=1, chunks=1, batched=False, steps_per_round=1, session_kw=None):
    """Gradient-accumulation form (Algorithms 2/3 as printed) on the GPU and on the oracle."""
    from oracle.ref import RefHPSGDAccum
    assert staleness == 1 and not cfg.momentum and not cfg.weight_decay
    o = RefHPSGDAccum(cfg.P, cfg.K, cfg.lr)
    o.set_global(cfg.initial_global())
    with session(cfg, staleness=staleness, overlap=overlap, chunks=chunks, form=hp.HPSGD_FORM_GRADIENT_ACCUMULATION,
                 **(session_kw or {})):
        step = 0
        for t in range(T):
            keep = []
            for h in range(steps_per_round):
                inputs = [host_inputs(cfg, i, step) for i in range(cfg.K)]
                if batched and not cfg.sparse:
                    stacked = np.stack([inp["padded"] for inp in inputs])
                    g = to_device(stacked.reshape(-1))
                    keep.append(g)
                    hp.hpsgd_local_step_all(g, stacked.shape[1] * stacked.itemsize)
                else:
                    for i, inp in enumerate(inputs):
                        gpu_step(cfg, i, inp, keep)
                for i, inp in enumerate(inputs):
                    flat = inp["flat"]
                    o.local_step(i, hashgen.bf16_to_f32(flat) if flat.dtype == np.uint16 else flat)
                step += 1
            hp.hpsgd_synchronize()
            for i in range(cfg.K):
                r, a = hp.hpsgd_get_replica(i)
                assert_bitwise(gpu_flat(r, cfg), o.get_replica(i), "replica %d before sync %d" % (i, t))
                assert_bitwise(gpu_flat(a, cfg), o.get_accumulated(i), "accumulated gradient %d before sync %d" % (i, t))
            hp.hpsgd_sync_merge()
            o.sync_merge()
            hp.hpsgd_synchronize()
            w, ghat, rs, accs = gpu_state(cfg)
            assert_bitwise(w, o.get_global(), "global after sync %d" % t)
            assert_bitwise(ghat, o.get_synced(), "AllReduce result after sync %d" % t)
            for i in range(cfg.K):
                assert_bitwise(rs[i], o.get_global(), "replica %d after sync %d" % (i, t))
                assert not accs[i].any(), "accumulator %d not reset" % i
        got = gpu_global(cfg)
    want = o.get_global()
    o.close()
    return got, want
