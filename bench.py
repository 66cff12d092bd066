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


# DRAM bytes per parameter index (dram__bytes_read.sum + dram__bytes_write.sum of one ncu
# capture divided by the indices of that launch), keyed by (kernel, K, gradient dtype, fuse variant), with
# the SHA-1 of the kernel source the capture was taken from.  A changed source voids them.
NCU_TRAFFIC = {
    # profiles/merge_step_kernel_cfg4_cut16M.txt (last launch): 3.200047 GB read + 2.123349 GB written over 16,000,000 indices
    ('merge_step_kernel', 16, 'f32', 1): {"bytes_per_index": 5.323396e9 / 16e6, "source_sha1": "5d530923c7baf3340525993c3ad2d3ee08488a94"},
    # profiles/merge_step_implicit_kernel_cfg4_cut16M.txt (last launch): 2.176030 GB read + 1.126342 GB written over 16,000,000 indices
    ('merge_step_kernel', 16, 'f32', 2): {"bytes_per_index": 3.302372e9 / 16e6, "source_sha1": "5d530923c7baf3340525993c3ad2d3ee08488a94"},
    # profiles/merge_kernel_cfg4_cut16M.txt (last launch): 1.152017 GB read + 1.093487 GB written over 16,000,000 indices
    ('merge_kernel', 16, 'f32', 0): {"bytes_per_index": 2.245504e9 / 16e6, "source_sha1": "5d530923c7baf3340525993c3ad2d3ee08488a94"},
    # profiles/local_step_kernel_cfg4_cut16M.txt (last launch): 3.072011 GB read + 1.997550 GB written over 16,000,000 indices
    ('local_step_kernel', 16, 'f32', 0): {"bytes_per_index": 5.069561e9 / 16e6, "source_sha1": "5d530923c7baf3340525993c3ad2d3ee08488a94"},
}


def ncu_traffic(kernel, cfg, fuse):
    """Measured DRAM bytes of one full launch of that kernel on this workload, or None."""
    variant = fuse if kernel == "merge_step_kernel" else 0
    entry = NCU_TRAFFIC.get((kernel, cfg.K, cfg.grad_dtype, variant))
    if entry is None:
        return None
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
    lay = cfg.layout
    K, P, P_pad = cfg.K, cfg.P, lay.P_pad
    bf16 = cfg.grad_dtype == "bf16"
    gdt = torch.int16 if bf16 else torch.float32
    gsz = 2 if bf16 else 4
    kind = hp.HPSGD_GEN_UNIFORM if cfg.grad_kind == "uniform" else hp.HPSGD_GEN_GAUSS

    # ---- state: arena and streams come from torch, the library only computes.  The arena is
    # sized for the pipelined schedule too, so that every schedule can be timed in one run.
    nbytes = hp.hpsgd_arena_bytes(P_pad, K, (hp.HPSGD_ARENA_MOMENTUM if cfg.momentum else 0) | hp.HPSGD_ARENA_PIPELINE,
                                  cfg.sparse[1] if cfg.sparse else 0)
    arena = torch.empty(nbytes + 256, dtype=torch.uint8, device=dev)
    base = arena.data_ptr() + (-arena.data_ptr()) % 256
    main, side = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)

    def setup(pipeline, fuse, chunks):
        hp.hpsgd_destroy()
        if len(cfg.sizes) > 1:
            hp.hpsgd_set_layout(list(cfg.sizes))
        hp.hpsgd_set_pipeline(pipeline)
        hp.hpsgd_bind(base, nbytes, main, side)
        hp.hpsgd_init(P, K, cfg.lr, cfg.momentum, cfg.seed)
        if cfg.weight_decay:
            hp.hpsgd_set_option(hp.HPSGD_OPT_WEIGHT_DECAY, cfg.weight_decay)
        hp.hpsgd_set_option(hp.HPSGD_OPT_STALENESS, cfg.staleness)
        hp.hpsgd_set_option(hp.HPSGD_OPT_GRAD_DTYPE, hp.HPSGD_BF16 if bf16 else hp.HPSGD_F32)
        hp.hpsgd_set_option(hp.HPSGD_OPT_OVERLAP, args.overlap)
        hp.hpsgd_set_option(hp.HPSGD_OPT_CHUNKS, 1 if pipeline else chunks)
        hp.hpsgd_set_option(hp.HPSGD_OPT_FUSE, fuse)
        if cfg.sparse:
            hp.hpsgd_set_sparse_segment(*cfg.sparse)

    setup(args.pipeline, args.fuse, args.chunks)

    # ---- inputs: `nbuf` rounds of gradients for all K workers, generated on the device
    nbuf = args.grad_buffers
    row = -(-P_pad // 2048) * 2048          # every worker's gradient starts on a 4 KB boundary
    grads = torch.empty((nbuf, K, row), dtype=gdt, device=dev)[:, :, :P_pad]
    sparse_in = None
    if cfg.sparse:
        rows_max = cfg.sparse[1]
        cols = cfg.sparse[2]
        sparse_in = []
        for b in range(nbuf):
            per_worker = []
            for i in range(K):
                idx = torch.from_numpy(cfg.sparse_rows(i, b)).to(dev)
                vals = torch.empty(idx.numel() * cols, dtype=gdt, device=dev)
                hp.hpsgd_gen_row_vals(vals, i, b, kind, cfg.grad_scale, idx, idx.numel())
                per_worker.append((idx, vals))
            sparse_in.append(per_worker)
    for b in range(nbuf):
        for i in range(K):
            hp.hpsgd_gen_grads(grads[b, i], i, b, kind, cfg.grad_scale)
    hp.hpsgd_synchronize()

    def one_round(t):
        b = t % nbuf
        if cfg.sparse:
            descs = [hp.make_desc(grads[b, i], sparse_in[b][i][0], sparse_in[b][i][0].numel(), sparse_in[b][i][1])
                     for i in range(K)]
            if args.per_worker:
                for i in range(K):
                    hp.hpsgd_local_step_ex(i, descs[i])
            else:
                hp.hpsgd_local_step_all_ex(descs)
        elif args.per_worker:
            for i in range(K):
                hp.hpsgd_local_step(i, grads[b, i])
        else:
            hp.hpsgd_local_step_all(grads[b], row * gsz)
        hp.hpsgd_sync_merge()

    # ---- warm-up, then the timed region (the clock sampler needs a moment to start)
    sampler = ClockSampler(device_index)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    for t in range(args.warmup):
        one_round(t)
    hp.hpsgd_synchronize()
    hp.hpsgd_set_option(hp.HPSGD_OPT_PROFILE, 1)     # also launches a merge deferred by the warm-up
    for kind in range(4):
        hp.hpsgd_profile_read(kind)
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize(dev)
    sampler.mark_begin()
    launches0 = hp.hpsgd_launch_count()
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record(main)
    for t in range(args.steps):
        one_round(args.warmup + t)
    hp.hpsgd_flush()                                 # the last round's merge, if it was deferred
    main.wait_stream(side)
    end.record(main)
    torch.cuda.synchronize(dev)
    sampler.mark_end()
    if dist is not None:
        dist.barrier()
    clocks = sampler.stop() if rank == 0 else None
    elapsed_ms = start.elapsed_time(end)
    launches = hp.hpsgd_launch_count() - launches0
    prof = {name: hp.hpsgd_profile_read(kind) for kind, name in
            enumerate(("local_step_kernel", "merge_kernel", "merge_step_kernel", "round_kernel"))}
    hp.hpsgd_set_option(hp.HPSGD_OPT_PROFILE, 0)
    units = K * P * args.steps
    job_ms, job_units = aggregate(dist, dev, elapsed_ms, units)
    value = job_units / (job_ms * 1e-3)

    # ---- roofline of the kernels from the event pairs recorded inside the timed region.
    # Algorithmic bytes per launch = bytes per parameter index x indices one launch covers.
    peak, peak_src = measured_peak()
    # gradient bytes of one round: dense buffers, minus the rows of a sparse-row tensor that carry
    # no gradient (never read), plus 4 bytes per listed row index
    grad_bytes = K * P * gsz
    if cfg.sparse:
        rows_total, cols = cfg.sparse[1], cfg.sparse[2]
        active = sum(pw[0].numel() for b in sparse_in for pw in b) / nbuf
        grad_bytes += active * 4 - (K * rows_total - active) * cols * gsz
    state_bytes = K * P * (8 + (8 if cfg.momentum else 0))        # r (and m) read and written
    per_round = {"local_step_kernel": grad_bytes + state_bytes,
                 # pipelined: commit (w, D in; w out) + reduce (K r + w in; D out), two launches per merge
                 "merge_kernel": (12 + (K + 2) * 4) * P if args.pipeline else merge_bytes_per_index(cfg) * P,
                 "merge_step_kernel": 16 * P + grad_bytes + state_bytes,
                 # whole round in one kernel, one step per worker and period: no replica row is read
                 # or written; w, D, K m, K g in and w, D, K m out
                 "round_kernel": 16 * P + grad_bytes + (K * P * 8 if cfg.momentum else 0)}
    kernels = {}
    for name, (ms, n) in prof.items():
        if n == 0:
            continue
        per_launch = per_round[name] / (1 if args.pipeline else args.chunks) / (K if (args.per_worker and name == "local_step_kernel") else 1)
        if args.pipeline and name == "merge_kernel":
            per_launch /= 2
        gbs = per_launch * n / (ms * 1e-3) / 1e9
        kernels[name] = {"launches": n, "avg_ms": ms / n, "total_ms": ms, "algorithmic_bytes_per_launch": per_launch,
                         "achieved": gbs, "frac": gbs / peak, "frac_of_nominal_8TBs": gbs / NOMINAL_HBM_GBS}
    dominant = max(kernels, key=lambda k: kernels[k]["total_ms"])
    roofline = {"bound": "hbm", "kernel": dominant, "achieved": kernels[dominant]["achieved"], "peak": peak,
                "unit": "GB/s", "frac": kernels[dominant]["frac"],
                "traffic": ncu_traffic(dominant, cfg, args.fuse) if (args.chunks == 1 and not args.per_worker) else None,
                "peak_source": peak_src, "nominal_peak": NOMINAL_HBM_GBS, "kernels": kernels,
                "note": "CUDA event pairs around each launch on its own stream inside the timed region; "
                        "bytes are the ones the launch actually moves: round_kernel (local steps + merge in one "
                        "pass, replicas never stored) 16 + K*(g + 8) per index with momentum, merge_step_kernel "
                        "16 + K*(g + 16), merge_kernel (2K + 4)*4, local_step_kernel K*(g + 16)"}
    moved = sum(k["algorithmic_bytes_per_launch"] * k["launches"] for k in kernels.values())
    roofline["round_achieved"] = moved / (elapsed_ms * 1e-3) / 1e9
    roofline["round_frac"] = roofline["round_achieved"] / peak
    unfused_round = per_round["local_step_kernel"] + per_round["merge_kernel"]
    roofline["round_unfused_equivalent"] = unfused_round * args.steps / (elapsed_ms * 1e-3) / 1e9

    # ---- the other schedules of the same path, timed briefly the same way (same inputs, same work)
    other = {}
    if args.other_schedule_steps > 0 and not args.per_worker:
        for name, pipe, fuse in (("separate merge and local-step kernels on two streams", 0, 0),
                                 ("pipelined commit + reduce on double-buffered replicas", 1, 0),
                                 ("merge fused into the next local step", 0, 1),
                                 ("one kernel per round (local steps + merge), replicas never stored", 0, 2)):
            if (pipe, fuse if not pipe else 0) == (args.pipeline, 0 if args.pipeline else args.fuse):
                continue
            setup(pipe, fuse, 1)
            for t in range(3):
                one_round(t)
            hp.hpsgd_synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(main)
            for t in range(args.other_schedule_steps):
                one_round(3 + t)
            hp.hpsgd_flush()
            main.wait_stream(side)
            b.record(main)
            torch.cuda.synchronize(dev)
            ms = a.elapsed_time(b) / args.other_schedule_steps
            other[name] = {"ms_per_step": ms, "value": K * P / (ms * 1e-3), "steps": args.other_schedule_steps}
        setup(args.pipeline, args.fuse, args.chunks)

    # ---- end to end: host gradient buffers in, host copy of the global model out, every step
    e2e = None
    if args.e2e_steps > 0:
        e2e = run_e2e(args, cfg, hp, torch, dev, grads, dist)

    line = None
    if rank == 0:
        cpu = None
        if args.cpu_seconds > 0:
            eps, rounds, spent, desc, _ = oracle_sample_run(cfg, args.cpu_seconds)
            cpu = {"value": eps, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": desc,
                   "seconds": spent}
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": job_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic (counter-hash gradients generated on the device, %d rounds cycled)" % nbuf,
            "config": workload_config(cfg, {
                "schedule": {"overlap": args.overlap, "chunks": args.chunks,
                             "fuse_merge_into_next_step": 0 if args.pipeline else args.fuse,
                             "pipelined_commit_reduce": args.pipeline,
                             "local_step_call": "per worker" if args.per_worker else "all K in one call"},
                "l2": "inputs larger than L2 (state + gradients are tens of GB)",
                "multi_gpu": "independent replicas, no inter-GPU exchange"}),
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
            "roofline": roofline, "cpu_baseline": cpu, "other_schedules": other,
        }
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
