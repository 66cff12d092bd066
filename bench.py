#!/usr/bin/env python
"""Benchmark of the HPSGD replica-update + merge path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg4] [--impl reference]

A "step" is one round of the whole path on one workload: one local step of every one of
the K simulated workers followed by one synchronisation (merge).  The metric is
parameter updates per second, K*P*steps / time.  One JSON line is printed by rank 0.

  * own arm (default): inputs resident in HBM, timed on the device with CUDA events;
    plus `e2e` (host gradient buffers through hpsgd_local_step_host, host copy of the
    global model every step), `roofline` for the kernels and `cpu_baseline`.
  * --impl reference: the CPU oracle, as it stands, on a bounded sample of the workload.

With N > 1 (torchrun) every rank runs an independent replica of the same workload (the
path has no inter-GPU exchange); time is the max over ranks, value the sum of units.
"""
from __future__ import annotations

import argparse
import datetime
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import workloads  # noqa: E402

METRIC = "parameter_updates_per_sec"
UNIT = "K*P elems/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


# ------------------------------------------------------------------------------ helpers
def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (6.65 TB/s, earlier measurement on this pool)"


def local_bytes_per_elem(cfg):
    """Algorithmic HBM bytes per parameter and worker of one local step."""
    g = 2 if cfg.grad_dtype == "bf16" else 4
    return g + 8 + (8 if cfg.momentum else 0)


def fused_bytes_per_index(cfg):
    """Fused merge + local step: the merge without its K replica writes plus the K local steps
    without their replica reads = 16 + K * (local step bytes)."""
    return 16 + cfg.K * local_bytes_per_elem(cfg)


# DRAM bytes per parameter index (dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture divided by
# the indices of that launch), keyed by (kernel, K, gradient dtype), with the SHA-1 of the kernel source the
# capture was taken from.  A changed source voids them.
NCU_TRAFFIC = {
    # profiles/round_kernel_cfg4_cut16M.txt: 2.176072 GB read + 1.103841 GB written over 16,000,000 indices
    ('round_kernel', 16, 'f32'): {"bytes_per_index": 3.279913e9 / 16e6, "source_sha1": "65baeb17746e2dd5628b51694946b71740efbca2"},
    # profiles/merge_step_kernel_cfg4_cut16M.txt: 3.200026 GB read + 2.121919 GB written over 16,000,000 indices
    ('merge_step_kernel', 16, 'f32'): {"bytes_per_index": 5.321945e9 / 16e6, "source_sha1": "65baeb17746e2dd5628b51694946b71740efbca2"},
    # profiles/merge_kernel_cfg4_cut16M.txt: 1.152136 GB read + 1.094072 GB written over 16,000,000 indices
    ('merge_kernel', 16, 'f32'): {"bytes_per_index": 2.246208e9 / 16e6, "source_sha1": "65baeb17746e2dd5628b51694946b71740efbca2"},
    # profiles/local_step_kernel_cfg4_cut16M.txt: 3.072011 GB read + 1.991900 GB written over 16,000,000 indices
    ('local_step_kernel', 16, 'f32'): {"bytes_per_index": 5.063911e9 / 16e6, "source_sha1": "65baeb17746e2dd5628b51694946b71740efbca2"},
    # profiles/round_kernel_cfg3.txt: 1.843402 GB read + 0.974777 GB written over 25,600,000 indices
    ('round_kernel', 8, 'f32'): {"bytes_per_index": 2.818179e9 / 25.6e6, "source_sha1": "65baeb17746e2dd5628b51694946b71740efbca2"},
}


def ncu_traffic(kernel, cfg, fuse):
    """Measured DRAM bytes of one full launch of that kernel on this workload, or None.  The captures
    are of momentum workloads in the default call form; nothing else is extrapolated from them."""
    entry = NCU_TRAFFIC.get((kernel, cfg.K, cfg.grad_dtype))
    if entry is None or not cfg.momentum or cfg.sparse:
        return None
    if kernel == "merge_kernel" and fuse == 2:
        return None                      # the lazy-clone merge writes no replicas: not the captured kernel
    import hashlib
    src = os.path.join(ROOT, "paper_2009_02701_b200", "csrc", "hpsgd_kernels.cuh")
    if hashlib.sha1(open(src, "rb").read()).hexdigest() != entry["source_sha1"]:
        return None
    return entry["bytes_per_index"] * cfg.P


def merge_bytes_per_index(cfg):
    """Algorithmic HBM bytes per parameter index of one merge: (2K + 4) * 4."""
    return (2 * cfg.K + 4) * 4


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples; only those taken inside the timed window
    (host wall clock between mark_begin and mark_end) are summarised."""

    QUERY = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu_index = gpu_index
        self.proc = None
        self.t0 = self.t1 = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_index), "--query-gpu=" + self.QUERY,
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def mark_begin(self):
        self.t0 = datetime.datetime.now()

    def mark_end(self):
        self.t1 = datetime.datetime.now()

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.05)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, smax, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        total = 0
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            total += 1
            try:
                stamp = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f")
                if self.t0 and self.t1 and not (self.t0 <= stamp <= self.t1):
                    continue
                sm.append(float(f[1]))
                smax.append(float(f[2]))
                power.append(float(f[3]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(smax) if smax else None,
                "power_w_max": max(power) if power else None,
                "samples_in_timed_region": len(sm), "samples_total": total, "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------ CPU oracle legs
def oracle_sample_run(cfg, seconds, sample_params=4_000_000, min_rounds=2, max_rounds=None):
    """Time the CPU oracle on the first `sample_params` parameters of the workload.

    Gradient generation is outside the timed part (as on the GPU).  Returns
    (elems_per_s, rounds, seconds_timed, description)."""
    from oracle.ref import RefHPSGD
    P = min(cfg.P, sample_params)
    idx = np.arange(P, dtype=np.int64)
    o = RefHPSGD(P, cfg.K, cfg.lr, cfg.momentum, cfg.weight_decay, cfg.staleness)
    o.set_global(cfg.initial_global(idx))
    grads = [[cfg.stored_gradient(i, t, idx) for i in range(cfg.K)] for t in range(2)]
    rounds, spent = 0, 0.0
    while True:
        g = grads[rounds % 2]
        t0 = time.perf_counter()
        for i in range(cfg.K):
            o.local_step(i, g[i])
        o.sync_merge()
        spent += time.perf_counter() - t0
        rounds += 1
        if max_rounds is not None and rounds >= max_rounds:
            break
        if max_rounds is None and rounds >= min_rounds and spent >= seconds:
            break
    o.close()
    desc = ("first %d of %d parameters of %s, all K=%d workers, %d rounds (local steps + merge; "
            "sparse rows given as dense zeros), single thread" % (P, cfg.P, cfg.name, cfg.K, rounds))
    return cfg.K * P * rounds / spent, rounds, spent, desc, P


def _oracle_range_worker(job):
    """One process of oracle_all_cores: the oracle on parameters [lo, hi) of the workload, `rounds` rounds
    timed after every process has its inputs (the barrier)."""
    name, lo, hi, rounds, barrier = job
    from oracle.ref import RefHPSGD
    cfg = workloads.get(name)
    idx = np.arange(lo, hi, dtype=np.int64)
    o = RefHPSGD(idx.size, cfg.K, cfg.lr, cfg.momentum, cfg.weight_decay, cfg.staleness)
    o.set_global(cfg.initial_global(idx))
    grads = [[cfg.stored_gradient(i, t, idx) for i in range(cfg.K)] for t in range(2)]
    barrier.wait()
    t0 = time.perf_counter()
    for r in range(rounds):
        for i in range(cfg.K):
            o.local_step(i, grads[r % 2][i])
        o.sync_merge()
    spent = time.perf_counter() - t0
    o.close()
    return spent


def oracle_all_cores(cfg, per_core_params=1_000_000, rounds=12):
    """The same oracle, unchanged, as one single-threaded process per host core, each on its own index
    range of the workload (the path is independent per index, so the results are those of one process).
    Processes are spawned, not forked: the parent has already used the GPU."""
    import multiprocessing as mp
    cores = os.cpu_count() or 1
    per = min(per_core_params, cfg.P // cores)
    ctx = mp.get_context("spawn")
    with ctx.Manager() as manager:
        barrier = manager.Barrier(cores)
        jobs = [(cfg.name, j * per, (j + 1) * per, rounds, barrier) for j in range(cores)]
        with ctx.Pool(cores) as pool:
            times = pool.map(_oracle_range_worker, jobs, chunksize=1)
    slowest = max(times)
    return {"value": cfg.K * per * cores * rounds / slowest, "unit": UNIT, "cores": cores,
            "sample": "%d processes x %d parameters each (the first %d of %s), all K=%d workers, %d rounds, "
                      "slowest process" % (cores, per, per * cores, cfg.name, cfg.K, rounds),
            "seconds": slowest}


def run_reference(args, cfg):
    """--impl reference: the CPU oracle as it stands; each step is one round (K local steps + one
    merge) on a bounded sample of the workload, the first `--ref-sample` parameters."""
    from oracle.ref import RefHPSGD
    P = min(cfg.P, args.ref_sample)
    idx = np.arange(P, dtype=np.int64)
    o = RefHPSGD(P, cfg.K, cfg.lr, cfg.momentum, cfg.weight_decay, cfg.staleness)
    o.set_global(cfg.initial_global(idx))
    grads = [[cfg.stored_gradient(i, t, idx) for i in range(cfg.K)] for t in range(2)]   # untimed, as on the GPU

    def one_round(t):
        t0 = time.perf_counter()
        for i in range(cfg.K):
            o.local_step(i, grads[t % 2][i])
        o.sync_merge()
        return time.perf_counter() - t0

    for t in range(max(0, args.warmup)):
        one_round(t)
    t_total = sum(one_round(args.warmup + t) for t in range(args.steps))
    o.close()
    value = cfg.K * P * args.steps / t_total
    desc = ("first %d of %d parameters of %s, all K=%d workers, one round per step (local steps + merge; "
            "sparse rows given as dense zeros), single thread" % (P, cfg.P, cfg.name, cfg.K))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t_total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic (counter-hash gradients)",
        "config": workload_config(cfg, {"sample": "each step = one round on the first %d parameters" % P}),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


def cut_workload(cfg, max_params):
    """The same rule, K and gradients on the leading part of the parameter set: tensors are taken
    in order until `max_params` is reached, the one that crosses it is shortened (a sparse-row
    tensor keeps whole rows).  Used for profiler captures, which must stay small."""
    sizes, total, sparse = [], 0, None
    for t, size in enumerate(cfg.sizes):
        room = max_params - total
        if room < 64:
            break
        if cfg.sparse and t == cfg.sparse[0]:
            cols = cfg.sparse[2]
            rows = max(1, min(cfg.sparse[1], room // cols))
            size = rows * cols
            sparse = (len(sizes), rows, cols)
        else:
            size = min(size, room)
        sizes.append(size)
        total += size
    cut = cfg.subset(cfg.name, sizes, sparse=sparse)
    object.__setattr__(cut, "note", "%s, cut to its first %d parameters" % (cfg.note, total))
    return cut


def workload_config(cfg, extra=None):
    c = {"workload": "%s: %s" % (cfg.name, cfg.note), "K": cfg.K, "P": cfg.P, "tensors": len(cfg.sizes),
         "lr": cfg.lr, "momentum": cfg.momentum, "weight_decay": cfg.weight_decay,
         "grad_dtype": cfg.grad_dtype, "staleness": cfg.staleness, "local_steps_per_merge": 1}
    if extra:
        c.update(extra)
    return c


# ------------------------------------------------------------------------------ distributed plumbing
def dist_setup(n_gpus):
    """Returns (rank, world, local_rank, dist-module-or-None)."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world <= 1:
        return 0, 1, 0, None
    import torch.distributed as dist
    backend = os.environ.get("HPSGD_BENCH_BACKEND", "nccl")
    dist.init_process_group(backend=backend)
    return dist.get_rank(), dist.get_world_size(), int(os.environ.get("LOCAL_RANK", "0")), dist


def aggregate(dist, device, elapsed_ms, units):
    """Whole-job figures: time = max over ranks, units = sum over ranks."""
    if dist is None:
        return elapsed_ms, units
    import torch
    t = torch.tensor([elapsed_ms], dtype=torch.float64, device=device)
    u = torch.tensor([float(units)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


# ------------------------------------------------------------------------------ GPU arm
class _RawDeviceArray:
    """A raw device address as something torch.as_tensor can wrap (CUDA array interface)."""

    def __init__(self, addr, n, typestr="<f4"):
        self.__cuda_array_interface__ = {"shape": (n,), "typestr": typestr, "data": (int(addr), False), "version": 2}


def parity_sample(cfg, n_random=1 << 14, edge=32, seed=2024):
    """Un-padded parameter indices the oracle recomputes: both ends of every tensor plus random ones."""
    picks = []
    for size, start in zip(cfg.layout.sizes, cfg.layout.starts):
        e = min(edge, size)
        picks += [np.arange(start, start + e), np.arange(start + size - e, start + size)]
    picks.append(np.random.default_rng(seed).integers(0, cfg.P, size=n_random))
    return np.unique(np.concatenate(picks)).astype(np.int64)


def ulp_distance(a, b):
    a = np.ascontiguousarray(a, dtype=np.float32).view(np.int32).astype(np.int64)
    b = np.ascontiguousarray(b, dtype=np.float32).view(np.int32).astype(np.int64)
    a = np.where(a < 0, -(a & 0x7FFFFFFF), a)
    b = np.where(b < 0, -(b & 0x7FFFFFFF), b)
    return np.abs(a - b)


PROBE_MIXES = ((16, 0), (16, 4), (12, 4), (13, 7), (12, 8), (8, 8), (4, 16), (0, 16))


def do_nothing_rates(hp, torch, dev, cfg):
    """GB/s of a kernel with the hot kernels' access shape and no arithmetic, for each built mix of
    read and write streams (hpsgd_probe_hbm), on arrays as long as one flat buffer of the workload
    (at most 512 MB each), so that a short launch is compared with an equally short one."""
    row_bytes = min(512 << 20, -(-cfg.layout.P_pad * 4 // 4096) * 4096)
    iters = int(min(500, max(10, 4e9 // (16 * row_bytes))))
    buf = torch.empty(20 * row_bytes + 4096, dtype=torch.uint8, device=dev)
    base = buf.data_ptr() + (-buf.data_ptr()) % 4096
    torch.cuda.synchronize(dev)
    warm = int(min(10000, max(1, 4e10 // (16 * row_bytes))))
    hp.hpsgd_probe_hbm(base, 20 * row_bytes, 8, 8, row_bytes, warm)    # ~60 ms of load first: the clocks drop while the oracle runs
    out = []
    for n_read, n_write in PROBE_MIXES:
        rate = max(hp.hpsgd_probe_hbm(base, 20 * row_bytes, n_read, n_write, row_bytes, iters) for _ in range(2))
        out.append({"reads": n_read, "writes": n_write, "write_share": n_write / (n_read + n_write), "GB/s": rate})
    del buf
    torch.cuda.empty_cache()
    return {"array_bytes": row_bytes, "launches_timed": iters, "rates": out}


def against_do_nothing(rates, share, achieved):
    """The probe rate at the kernel's share of writes (linear between the two nearest built mixes)."""
    pts = sorted((r["write_share"], r["GB/s"]) for r in rates["rates"])
    rate = pts[-1][1]
    for (s0, r0), (s1, r1) in zip(pts, pts[1:]):
        if s0 <= share <= s1:
            rate = r0 + (r1 - r0) * (share - s0) / (s1 - s0)
            break
    return {"write_share": share, "do_nothing_GB/s": rate, "kernel_over_do_nothing": achieved / rate}


class GpuWorkload:
    """One workload resident on one GPU: arena and streams from torch, `nbuf` rounds of
    device-generated gradients, and the schedules of the path timed on them."""

    KERNELS = ("local_step_kernel", "merge_kernel", "merge_step_kernel", "round_kernel", "merge_staged_kernel")

    def __init__(self, hp, torch, dev, cfg, args):
        self.hp, self.torch, self.dev, self.cfg, self.args = hp, torch, dev, cfg, args
        lay = cfg.layout
        K, P_pad = cfg.K, lay.P_pad
        self.bf16 = cfg.grad_dtype == "bf16"
        self.gdt = torch.int16 if self.bf16 else torch.float32
        self.gsz = 2 if self.bf16 else 4
        self.kind = hp.HPSGD_GEN_UNIFORM if cfg.grad_kind == "uniform" else hp.HPSGD_GEN_GAUSS
        # state: arena and streams come from torch, the library only computes.  The arena is sized
        # for the pipelined schedule too, so that every schedule can be timed in one run.
        self.nbytes = hp.hpsgd_arena_bytes(P_pad, K, (hp.HPSGD_ARENA_MOMENTUM if cfg.momentum else 0) | hp.HPSGD_ARENA_PIPELINE,
                                           cfg.sparse[1] if cfg.sparse else 0)
        self.arena = torch.empty(self.nbytes + 256, dtype=torch.uint8, device=dev)
        self.base = self.arena.data_ptr() + (-self.arena.data_ptr()) % 256
        self.main, self.side = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
        self.setup(args.pipeline, args.fuse, args.chunks, args.staging)
        # inputs: `nbuf` rounds of gradients for all K workers, generated on the device
        self.nbuf = nbuf = args.grad_buffers
        self.row = -(-P_pad // 2048) * 2048          # every worker's gradient starts on a 4 KB boundary
        self.grads = torch.empty((nbuf, K, self.row), dtype=self.gdt, device=dev)[:, :, :P_pad]
        self.sparse_in = None
        self.keep = []
        if cfg.sparse:
            cols = cfg.sparse[2]
            self.sparse_in = []
            for b in range(nbuf):
                per_worker = []
                for i in range(K):
                    idx = torch.from_numpy(cfg.sparse_rows(i, b)).to(dev)
                    vals = torch.empty(idx.numel() * cols, dtype=self.gdt, device=dev)
                    hp.hpsgd_gen_row_vals(vals, i, b, self.kind, cfg.grad_scale, idx, idx.numel())
                    per_worker.append((idx, vals))
                self.sparse_in.append(per_worker)
        for b in range(nbuf):
            for i in range(K):
                hp.hpsgd_gen_grads(self.grads[b, i], i, b, self.kind, cfg.grad_scale)
        hp.hpsgd_synchronize()

    def setup(self, pipeline, fuse, chunks, staging=0):
        hp, cfg = self.hp, self.cfg
        hp.hpsgd_destroy()
        if len(cfg.sizes) > 1:
            hp.hpsgd_set_layout(list(cfg.sizes))
        hp.hpsgd_set_pipeline(pipeline)
        hp.hpsgd_bind(self.base, self.nbytes, self.main, self.side)
        hp.hpsgd_init(cfg.P, cfg.K, cfg.lr, cfg.momentum, cfg.seed)
        if cfg.weight_decay:
            hp.hpsgd_set_option(hp.HPSGD_OPT_WEIGHT_DECAY, cfg.weight_decay)
        hp.hpsgd_set_option(hp.HPSGD_OPT_STALENESS, cfg.staleness)
        hp.hpsgd_set_option(hp.HPSGD_OPT_GRAD_DTYPE, hp.HPSGD_BF16 if self.bf16 else hp.HPSGD_F32)
        hp.hpsgd_set_option(hp.HPSGD_OPT_OVERLAP, self.args.overlap)
        hp.hpsgd_set_option(hp.HPSGD_OPT_CHUNKS, 1 if pipeline else chunks)
        hp.hpsgd_set_option(hp.HPSGD_OPT_FUSE, fuse)
        hp.hpsgd_set_option(hp.HPSGD_OPT_STAGING, staging)
        if cfg.sparse:
            hp.hpsgd_set_sparse_segment(*cfg.sparse)
        self.pipeline, self.fuse, self.chunks = pipeline, (0 if pipeline else fuse), (1 if pipeline else chunks)

    def regenerate(self, b, step):
        """Refill gradient buffer `b` with the gradients of round `step` (device generator, main stream)."""
        hp, cfg = self.hp, self.cfg
        if cfg.sparse:
            cols = cfg.sparse[2]
            per_worker = []
            for i in range(cfg.K):
                idx = self.torch.from_numpy(cfg.sparse_rows(i, step)).to(self.dev)
                vals = self.torch.empty(idx.numel() * cols, dtype=self.gdt, device=self.dev)
                self.torch.cuda.current_stream().synchronize()      # the upload ran on torch's stream
                hp.hpsgd_gen_row_vals(vals, i, step, self.kind, cfg.grad_scale, idx, idx.numel())
                per_worker.append((idx, vals))
            self.keep.append(self.sparse_in[b])                     # earlier rows may still be in use by queued work
            self.sparse_in[b] = per_worker
        for i in range(cfg.K):
            hp.hpsgd_gen_grads(self.grads[b, i], i, step, self.kind, cfg.grad_scale)

    def one_round(self, t):
        hp, cfg, args = self.hp, self.cfg, self.args
        b = t % self.nbuf
        if cfg.sparse:
            descs = [hp.make_desc(self.grads[b, i], self.sparse_in[b][i][0], self.sparse_in[b][i][0].numel(),
                                  self.sparse_in[b][i][1]) for i in range(cfg.K)]
            if args.per_worker:
                for i in range(cfg.K):
                    hp.hpsgd_local_step_ex(i, descs[i])
            else:
                hp.hpsgd_local_step_all_ex(descs)
        elif args.per_worker:
            for i in range(cfg.K):
                hp.hpsgd_local_step(i, self.grads[b, i])
        else:
            hp.hpsgd_local_step_all(self.grads[b], self.row * self.gsz)
        hp.hpsgd_sync_merge()

    def timed(self, steps, warmup, sampler=None, dist=None):
        """`warmup` untimed rounds, then `steps` rounds between two events on the main stream
        (the side stream joined before the second).  Returns (ms, launches, per-kernel event sums)."""
        hp, torch = self.hp, self.torch
        for t in range(warmup):
            self.one_round(t)
        hp.hpsgd_synchronize()
        hp.hpsgd_set_option(hp.HPSGD_OPT_PROFILE, 1)     # also launches anything the warm-up left held back
        for kind in range(len(self.KERNELS)):
            hp.hpsgd_profile_read(kind)
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(self.dev)
        if sampler is not None:
            sampler.mark_begin()
        launches0 = hp.hpsgd_launch_count()
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record(self.main)
        for t in range(steps):
            self.one_round(warmup + t)
        hp.hpsgd_flush()                                 # the last round's merge, if a schedule held it back
        self.main.wait_stream(self.side)
        end.record(self.main)
        torch.cuda.synchronize(self.dev)
        if sampler is not None:
            sampler.mark_end()
        if dist is not None:
            dist.barrier()
        ms = start.elapsed_time(end)
        launches = hp.hpsgd_launch_count() - launches0
        prof = {name: hp.hpsgd_profile_read(kind) for kind, name in enumerate(self.KERNELS)}
        hp.hpsgd_set_option(hp.HPSGD_OPT_PROFILE, 0)
        return ms, launches, prof

    def bytes_per_round(self):
        """HBM bytes each kind of kernel moves in one round of the current schedule (what the launch
        really reads and writes, not what an un-fused schedule would)."""
        cfg, K, P = self.cfg, self.cfg.K, self.cfg.P
        # gradient bytes of one round: dense buffers, minus the rows of a sparse-row tensor that carry
        # no gradient (never read), plus 4 bytes per listed row index
        grad_bytes = K * P * self.gsz
        if cfg.sparse:
            rows_total, cols = cfg.sparse[1], cfg.sparse[2]
            active = sum(pw[0].numel() for b in self.sparse_in for pw in b) / self.nbuf
            grad_bytes += active * 4 - (K * rows_total - active) * cols * self.gsz
        state_bytes = K * P * (8 + (8 if cfg.momentum else 0))        # r (and m) read and written
        return {"local_step_kernel": grad_bytes + state_bytes,
                "merge_staged_kernel": merge_bytes_per_index(cfg) * P,
                # pipelined: commit (w, D in; w out) + reduce (K r + w in; D out), two launches per merge
                "merge_kernel": (12 + (K + 2) * 4) * P if self.pipeline else
                                ((K + 4) * 4 * P if self.fuse == 2 else merge_bytes_per_index(cfg) * P),
                "merge_step_kernel": 16 * P + grad_bytes + state_bytes,
                # whole round in one kernel, one step per worker and period: no replica row is read
                # or written; w, D, K m, K g in and w, D, K m out
                "round_kernel": 16 * P + grad_bytes + (K * P * 8 if cfg.momentum else 0)}

    def write_share(self, kernel):
        """Share of the bytes a launch of `kernel` moves that are writes (HBM's rate depends on it)."""
        cfg, K, P = self.cfg, self.cfg.K, self.cfg.P
        mom = 4 if cfg.momentum else 0
        written = {"local_step_kernel": K * P * (4 + mom),
                   # pipelined: the commit writes w, the reduce writes D (two launches, one figure)
                   "merge_kernel": (8 * P if (self.pipeline or self.fuse == 2) else (K + 2) * 4 * P),
                   "merge_staged_kernel": (K + 2) * 4 * P,
                   "merge_step_kernel": 8 * P + K * P * (4 + mom),
                   "round_kernel": 8 * P + K * P * mom}[kernel]
        return written / self.bytes_per_round()[kernel]

    def kernel_table(self, prof, peak):
        per_round = self.bytes_per_round()
        kernels = {}
        for name, (ms, n) in prof.items():
            if n == 0:
                continue
            per_launch = per_round[name] / self.chunks
            if self.args.per_worker and name == "local_step_kernel":
                per_launch /= self.cfg.K
            if self.pipeline and name == "merge_kernel":
                per_launch /= 2
            gbs = per_launch * n / (ms * 1e-3) / 1e9
            kernels[name] = {"launches": n, "avg_ms": ms / n, "total_ms": ms, "bytes_per_launch": per_launch,
                             "achieved": gbs, "frac": gbs / peak, "frac_of_nominal_8TBs": gbs / NOMINAL_HBM_GBS}
        return kernels

    def parity(self):
        """The workload's T rounds from a fresh state in the schedule being timed, then w and D at a
        stratified sample of indices against the CPU oracle fed the HOST generator's gradients."""
        from oracle.ref import RefHPSGD
        hp, torch, cfg = self.hp, self.torch, self.cfg
        lay = cfg.layout
        self.setup(self.pipeline, self.fuse if not self.pipeline else 0, self.chunks, self.args.staging)
        for t in range(cfg.T):
            self.regenerate(0, t)         # every round its own gradients, as in a real run (untimed)
            self.one_round(0)
        hp.hpsgd_synchronize()
        idx = parity_sample(cfg)
        pos = torch.from_numpy(lay.padded_index(idx)).to(self.dev)
        got = {}
        for key, addr in (("w", hp.hpsgd_get_global()), ("D", hp.hpsgd_get_pending())):
            got[key] = torch.as_tensor(_RawDeviceArray(addr, lay.P_pad), device=self.dev)[pos].cpu().numpy()
        t0 = time.perf_counter()
        oracle = RefHPSGD(idx.size, cfg.K, cfg.lr, cfg.momentum, cfg.weight_decay, cfg.staleness)
        oracle.set_global(cfg.initial_global(idx))
        master = None
        if self.bf16:      # the same rule fed the gradients before their rounding to bf16
            master = RefHPSGD(idx.size, cfg.K, cfg.lr, cfg.momentum, cfg.weight_decay, cfg.staleness)
            master.set_global(cfg.initial_global(idx))
        for t in range(cfg.T):
            for i in range(cfg.K):
                oracle.local_step(i, cfg.stored_gradient(i, t, idx))
                if master:
                    master.local_step(i, cfg.gradient(i, t, idx))
            oracle.sync_merge()
            if master:
                master.sync_merge()
        want = {"w": oracle.get_global(), "D": oracle.get_pending()}
        out = {"rounds": cfg.T, "sampled_indices": int(idx.size),
               "inputs": "fresh gradients every round: device generator on the GPU, host generator for the oracle"}
        for key, floor in (("w", 1e-6), ("D", 1e-9)):
            g64, w64 = got[key].astype(np.float64), want[key].astype(np.float64)
            out[key] = {"max_rel_err": float(np.max(np.abs(g64 - w64) / np.maximum(np.abs(w64), floor))),
                        "max_ulp": int(ulp_distance(got[key], want[key]).max()),
                        "bit_equal_fraction": float(np.mean((got[key].view(np.uint32) == want[key].view(np.uint32))
                                                            | ((got[key] == 0) & (want[key] == 0))))}
        out["within_1e-6"] = bool(out["w"]["max_rel_err"] <= 1e-6)
        if master:
            m64 = master.get_global().astype(np.float64)
            out["w_vs_fp32_master_max_rel_err_floor_1e-4"] = float(
                np.max(np.abs(got["w"].astype(np.float64) - m64) / np.maximum(np.abs(m64), 1e-4)))
            out["within_1e-2_of_fp32_master"] = bool(out["w_vs_fp32_master_max_rel_err_floor_1e-4"] <= 1e-2)
            master.close()
        oracle.close()
        out["oracle_seconds"] = time.perf_counter() - t0
        return out

    def release(self):
        self.hp.hpsgd_destroy()
        self.arena = self.grads = self.sparse_in = self.keep = None
        self.torch.cuda.empty_cache()


def other_workload_entry(hp, torch, dev, name, args, peak):
    """A short timed run of another of the five workloads in the schedule being timed, with its
    parity figures (the oracle runs after the timed region)."""
    cfg = workloads.get(name)
    run = GpuWorkload(hp, torch, dev, cfg, args)
    steps = args.other_workload_steps
    ms, launches, prof = run.timed(steps, 3)
    kernels = run.kernel_table(prof, peak)
    dominant = max(kernels, key=lambda k: kernels[k]["total_ms"])
    entry = {"workload": "%s: %s" % (cfg.name, cfg.note), "K": cfg.K, "P": cfg.P, "steps": steps,
             "ms_per_step": ms / steps, "value": cfg.K * cfg.P * steps / (ms * 1e-3), "unit": UNIT,
             "gpu_launches": int(launches), "kernel": dominant, "kernel_avg_ms": kernels[dominant]["avg_ms"],
             "bytes_per_launch": kernels[dominant]["bytes_per_launch"], "achieved": kernels[dominant]["achieved"],
             "frac": kernels[dominant]["frac"], "frac_of_nominal_8TBs": kernels[dominant]["frac_of_nominal_8TBs"]}
    share = run.write_share(dominant)
    state_mb = run.nbytes / 1e6
    if state_mb + run.grads.numel() * run.gsz / 1e6 < 126:
        entry["note"] = "L2-resident (state + gradients below the 126 MB L2) and launch-bound: GB/s here is not an HBM figure"
    elif ms / steps < 0.5:
        entry["note"] = "sub-millisecond kernel: launch gaps and the tail of the grid weigh on the rate"
    if not args.per_worker and not args.pipeline and args.fuse != 0:
        # the same workload with separate local-step and merge kernels on two streams (the paper's schedule)
        run.setup(0, 0, 1)
        ms0, launches0, prof0 = run.timed(steps, 3)
        entry["separate_kernels"] = {
            "ms_per_step": ms0 / steps, "value": cfg.K * cfg.P * steps / (ms0 * 1e-3), "gpu_launches": int(launches0),
            "kernels": {k: {"launches": v["launches"], "avg_ms": v["avg_ms"], "bytes_per_launch": v["bytes_per_launch"],
                            "achieved": v["achieved"], "frac": v["frac"], "frac_of_nominal_8TBs": v["frac_of_nominal_8TBs"]}
                        for k, v in run.kernel_table(prof0, peak).items()}}
        run.setup(args.pipeline, args.fuse, args.chunks, args.staging)
    if args.parity:
        entry["parity"] = run.parity()
    run.release()
    if args.probe:
        rates = do_nothing_rates(hp, torch, dev, cfg)
        entry["do_nothing"] = {**rates, **against_do_nothing(rates, share, entry["achieved"])}
    return entry


def run_gpu(args, cfg):
    import torch
    import paper_2009_02701_b200 as hp
    from paper_2009_02701_b200 import build as cuda_build

    rank, world, local_rank, dist = dist_setup(args.gpus)
    # one GPU per rank; HPSGD_BENCH_DEVICE pins every rank to one device (single-GPU test runs of the
    # multi-rank code path: the ranks are independent replicas and never wait for each other)
    device_index = int(os.environ.get("HPSGD_BENCH_DEVICE", local_rank))
    torch.cuda.set_device(device_index)
    dev = torch.device("cuda", device_index)
    if local_rank == 0:
        cuda_build.build()              # no-op when the in-tree library is up to date
    if dist is not None:
        dist.barrier()
    K, P = cfg.K, cfg.P
    run = GpuWorkload(hp, torch, dev, cfg, args)

    # ---- warm-up, then the timed region (the clock sampler needs a moment to start)
    sampler = ClockSampler(device_index)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    elapsed_ms, launches, prof = run.timed(args.steps, args.warmup, sampler if rank == 0 else None, dist)
    clocks = sampler.stop() if rank == 0 else None
    units = K * P * args.steps
    job_ms, job_units = aggregate(dist, dev, elapsed_ms, units)
    value = job_units / (job_ms * 1e-3)

    # ---- roofline of the kernels from the event pairs recorded inside the timed region:
    # bytes one launch moves = bytes per parameter index x indices the launch covers
    peak, peak_src = measured_peak()
    kernels = run.kernel_table(prof, peak)
    dominant = max(kernels, key=lambda k: kernels[k]["total_ms"])
    per_round = run.bytes_per_round()
    roofline = {"bound": "hbm", "kernel": dominant, "achieved": kernels[dominant]["achieved"], "peak": peak,
                "unit": "GB/s", "frac": kernels[dominant]["frac"],
                "traffic": ncu_traffic(dominant, cfg, args.fuse) if (args.chunks == 1 and not args.per_worker) else None,
                "peak_source": peak_src, "nominal_peak": NOMINAL_HBM_GBS, "kernels": kernels,
                "note": "CUDA event pairs around each launch on its own stream inside the timed region; "
                        "bytes are the ones the launch actually moves: round_kernel (local steps + merge in one "
                        "pass, replicas never stored) 16 + K*(g + 8) per index with momentum, merge_step_kernel "
                        "16 + K*(g + 16), merge_kernel (2K + 4)*4, local_step_kernel K*(g + 16)"}
    moved = sum(k["bytes_per_launch"] * k["launches"] for k in kernels.values())
    roofline["round_achieved"] = moved / (elapsed_ms * 1e-3) / 1e9
    roofline["round_frac"] = roofline["round_achieved"] / peak
    # the same rounds priced at what separate local-step and merge kernels would have to move
    # (28K + 16 bytes per index with momentum): the rate the fusion is worth, not a bandwidth
    unfused_round = K * P * (run.gsz + 8 + (8 if cfg.momentum else 0)) + merge_bytes_per_index(cfg) * P
    roofline["round_unfused_equivalent"] = unfused_round * args.steps / (elapsed_ms * 1e-3) / 1e9

    # ---- the other schedules of the same path, timed briefly the same way (same inputs, same work)
    other = {}
    if args.other_schedule_steps > 0 and not args.per_worker:
        for name, pipe, fuse, staging in (
                ("separate merge and local-step kernels on two streams", 0, 0, 0),
                ("separate kernels, the merge's tiles staged through shared memory by bulk-async copies", 0, 0, 1),
                ("pipelined commit + reduce on double-buffered replicas", 1, 0, 0),
                ("merge fused into the next local step", 0, 1, 0),
                ("one kernel per round (local steps + merge), replicas never stored", 0, 2, 0)):
            if not staging and (pipe, fuse if not pipe else 0) == (args.pipeline, 0 if args.pipeline else args.fuse):
                continue
            run.setup(pipe, fuse, 1, staging)
            ms, n_launch, prof_o = run.timed(args.other_schedule_steps, 3)
            ms /= args.other_schedule_steps
            other[name] = {"ms_per_step": ms, "value": K * P / (ms * 1e-3), "steps": args.other_schedule_steps,
                           "gpu_launches": int(n_launch),
                           "kernels": {k: {"launches": v["launches"], "avg_ms": v["avg_ms"], "achieved": v["achieved"],
                                           "frac_of_nominal_8TBs": v["frac_of_nominal_8TBs"]}
                                       for k, v in run.kernel_table(prof_o, peak).items()}}
        run.setup(args.pipeline, args.fuse, args.chunks, args.staging)

    # ---- end to end: host gradient buffers in, host copy of the global model out, every step
    e2e = None
    if args.e2e_steps > 0:
        e2e = run_e2e(args, cfg, hp, torch, dev, run.grads, dist)

    line = None
    if rank == 0:
        parity = run.parity() if args.parity else None
        share = run.write_share(dominant)
        run.release()
        if args.probe:
            rates = do_nothing_rates(hp, torch, dev, cfg)
            roofline["do_nothing"] = {
                "method": "hpsgd_probe_hbm: R read + W write arrays as long as one flat buffer of the workload (at most "
                          "512 MB), one block per 128 groups of 8 floats, 256-bit accesses, sums only; best of two runs "
                          "of `launches_timed` launches each, CUDA events",
                **rates, **against_do_nothing(rates, share, kernels[dominant]["achieved"])}
        # ---- the other four workloads, briefly, each with its parity figures
        others = {}
        if args.other_workload_steps > 0 and not args.max_params:
            for name in workloads.names():
                if name != cfg.name:
                    others[name] = other_workload_entry(hp, torch, dev, name, args, peak)
        cpu = None
        if args.cpu_seconds > 0:
            eps, rounds, spent, desc, _ = oracle_sample_run(cfg, args.cpu_seconds)
            cpu = {"value": eps, "unit": UNIT, "cores": 1, "host_cores": os.cpu_count(), "kind": "oracle", "sample": desc,
                   "seconds": spent}
            if args.cpu_all_cores and not args.max_params:
                cpu["all_cores"] = oracle_all_cores(cfg)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": job_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic (counter-hash gradients generated on the device, %d rounds cycled)" % run.nbuf,
            "config": workload_config(cfg, {
                "schedule": {"overlap": args.overlap, "chunks": args.chunks,
                             "fuse": 0 if args.pipeline else args.fuse,
                             "fuse_meaning": "2: one kernel per round (batched local step inside the kernel of the merge "
                                             "that follows it); 1: merge carried into the next local step; 0: separate kernels",
                             "pipelined_commit_reduce": args.pipeline, "staged_merge": args.staging,
                             "local_step_call": "per worker" if args.per_worker else "all K in one call"},
                "l2": "inputs larger than L2 (state + gradients are tens of GB)",
                "multi_gpu": "independent replicas, no inter-GPU exchange"}),
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
            "roofline": roofline, "parity": parity, "cpu_baseline": cpu, "other_schedules": other,
            "workloads": others,
        }
    else:
        run.release()
    hp.hpsgd_destroy()
    if dist is not None:
        dist.destroy_process_group()
    if line is not None:
        print(json.dumps(line))


def run_e2e(args, cfg, hp, torch, dev, grads, dist):
    """Same metric with host buffers: every step copies each worker's gradient from pinned
    host memory (hpsgd_local_step_host) and reads the global model back (hpsgd_copy_global)."""
    K, P, P_pad = cfg.K, cfg.P, cfg.layout.P_pad
    gsz = 2 if cfg.grad_dtype == "bf16" else 4
    if cfg.sparse:
        hp.hpsgd_set_sparse_segment(-1, 0, 0)      # host path: dense gradients with zero rows
    nhost = min(K, args.e2e_host_buffers)
    host = [torch.empty(P_pad, dtype=grads.dtype).pin_memory() for _ in range(nhost)]
    for j in range(nhost):
        host[j].copy_(grads[0, j])
    out = [torch.empty(P, dtype=torch.float32).pin_memory() for _ in range(2)]
    torch.cuda.synchronize(dev)
    counter = [0]

    def one_step():
        # the read-back of step t runs beside the gradient uploads of step t+1 (PCIe is full duplex);
        # two result buffers, so that a result stays readable while the next one is written
        for i in range(K):
            hp.hpsgd_local_step_host(i, host[i % nhost])
        hp.hpsgd_sync_merge()
        hp.hpsgd_copy_global_async(out[counter[0] % 2])
        counter[0] += 1

    for _ in range(args.e2e_warmup):
        one_step()
    hp.hpsgd_synchronize()
    if dist is not None:
        dist.barrier()
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize(dev)
    start.record()
    t0 = time.perf_counter()
    for _ in range(args.e2e_steps):
        one_step()
    hp.hpsgd_synchronize()                 # the last read-back is part of the timed region
    end.record()
    torch.cuda.synchronize(dev)
    wall_ms = (time.perf_counter() - t0) * 1e3
    ms = max(start.elapsed_time(end), wall_ms)     # events on torch's stream do not see the library's streams
    job_ms, job_units = aggregate(dist, dev, ms, K * P * args.e2e_steps)
    if cfg.sparse:
        hp.hpsgd_set_sparse_segment(*cfg.sparse)
    return {"value": job_units / (job_ms * 1e-3), "unit": UNIT, "ms_per_step": job_ms / args.e2e_steps,
            "steps": args.e2e_steps, "h2d_bytes_per_step": K * P_pad * gsz, "d2h_bytes_per_step": P * 4,
            "host_buffers": "%d pinned gradient buffers cycled over the K workers" % nhost}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="own", choices=["own", "reference"])
    ap.add_argument("--workload", default="cfg4", choices=workloads.names())
    ap.add_argument("--overlap", type=int, default=1)
    ap.add_argument("--chunks", type=int, default=1)
    ap.add_argument("--fuse", type=int, default=2,
                    help="2: one kernel per round (the batched local step runs inside the kernel of the merge that "
                         "follows it, replicas never stored); 1: carry each merge into the next batched local step; "
                         "0: separate kernels on two streams")
    ap.add_argument("--pipeline", type=int, default=0,
                    help="paper timeline: commit on the main stream, K-way reduce on the side stream, double-buffered replicas")
    ap.add_argument("--other-schedule-steps", type=int, default=20,
                    help="steps used to time each of the other schedules for the record (0 = skip)")
    ap.add_argument("--per-worker", action="store_true", help="K hpsgd_local_step calls instead of one batched call")
    ap.add_argument("--grad-buffers", type=int, default=2, help="rounds of device-resident gradients to cycle")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--e2e-warmup", type=int, default=1)
    ap.add_argument("--e2e-host-buffers", type=int, default=4)
    ap.add_argument("--cpu-seconds", type=float, default=12.0, help="CPU oracle baseline budget (0 = skip)")
    ap.add_argument("--cpu-all-cores", type=int, default=1,
                    help="1: also time the oracle as one process per host core on disjoint index ranges")
    ap.add_argument("--other-workload-steps", type=int, default=10,
                    help="timed rounds for each of the other four workloads, reported under `workloads` (0 = skip)")
    ap.add_argument("--staging", type=int, default=0,
                    help="1: the stand-alone merge (fuse 0 or 1) stages its tiles through shared memory with bulk-async copies")
    ap.add_argument("--probe", type=int, default=1,
                    help="1: also measure what HBM gives a do-nothing kernel for each read/write mix (hpsgd_probe_hbm)")
    ap.add_argument("--parity", type=int, default=1,
                    help="1: after the timed regions, run each workload's T rounds and compare a sample with the CPU oracle")
    ap.add_argument("--max-params", type=int, default=0,
                    help="cut the workload to its first N parameters (for small profiler captures)")
    ap.add_argument("--ref-sample", type=int, default=4_000_000, help="parameters per step of --impl reference")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "own" else args.warmup
    cfg = workloads.get(args.workload)
    if args.max_params:
        cfg = cut_workload(cfg, args.max_params)

    if args.impl == "reference":
        if int(os.environ.get("RANK", "0")) != 0:
            return 0
        run_reference(args, cfg)
        return 0
    run_gpu(args, cfg)
    return 0


if __name__ == "__main__":
    sys.exit(main())
