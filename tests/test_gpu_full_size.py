"""Full-size workloads (cfg4: 138M parameters x 16 workers, cfg5: GRU-shaped, bf16 + sparse
rows) in the launch configuration the benchmark times: gradients generated on the device,
one batched local-step call and one merge per round.  The oracle cannot run 2.2 G
parameters x T rounds in seconds, and every index is independent of every other, so it
recomputes a stratified sample of indices (both ends of every tensor plus 2^18 random
ones) from the HOST generator and those are compared."""
import numpy as np
import pytest
import torch

import paper_2009_02701_b200 as hp
import workloads
from oracle.ref import RefHPSGD
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def run_full(cfg, T, fuse, pipeline=0, fp32_master=False):
    lay = cfg.layout
    K, P_pad = cfg.K, lay.P_pad
    bf16 = cfg.grad_dtype == "bf16"
    gdt = torch.int16 if bf16 else torch.float32
    kind = hp.HPSGD_GEN_UNIFORM if cfg.grad_kind == "uniform" else hp.HPSGD_GEN_GAUSS
    idx = gu.stratified_sample(cfg)
    pos = lay.padded_index(idx)

    oracle = RefHPSGD(idx.size, K, cfg.lr, cfg.momentum, cfg.weight_decay, cfg.staleness)
    oracle.set_global(cfg.initial_global(idx))
    master = None
    if fp32_master:       # the same rule fed the gradients BEFORE their rounding to bf16
        master = RefHPSGD(idx.size, K, cfg.lr, cfg.momentum, cfg.weight_decay, cfg.staleness)
        master.set_global(cfg.initial_global(idx))

    with gu.session(cfg, fuse=fuse, pipeline=pipeline, lend_arena=True, streams=True, canary=True):
        # one gradient buffer, refilled every round by the device generator: generator and consumers
        # are all enqueued on the main stream, so no host synchronisation is needed (one would also
        # launch a deferred merge on its own and keep the fused kernel from ever running)
        grads = torch.empty((K, P_pad), dtype=gdt, device=gu.DEV)
        keep = []
        hp.hpsgd_set_option(hp.HPSGD_OPT_PROFILE, 1)
        for t in range(T):
            descs = []
            for i in range(K):
                hp.hpsgd_gen_grads(grads[i], i, t, kind, cfg.grad_scale)
                if cfg.sparse:
                    rows = gu.to_device(cfg.sparse_rows(i, t))
                    vals = torch.empty(rows.numel() * cfg.sparse[2], dtype=gdt, device=gu.DEV)
                    hp.hpsgd_gen_row_vals(vals, i, t, kind, cfg.grad_scale, rows, rows.numel())
                    keep += [rows, vals]
                    descs.append(hp.make_desc(grads[i], rows, rows.numel(), vals))
            if cfg.sparse:
                hp.hpsgd_local_step_all_ex(descs)
            else:
                hp.hpsgd_local_step_all(grads, P_pad * grads.element_size())
            hp.hpsgd_sync_merge()
            for i in range(K):
                oracle.local_step(i, cfg.stored_gradient(i, t, idx))
                if master is not None:
                    master.local_step(i, cfg.gradient(i, t, idx))
            oracle.sync_merge()
            if master is not None:
                master.sync_merge()
        hp.hpsgd_synchronize()
        ran = tuple(hp.hpsgd_profile_read(kind)[1] for kind in (hp.HPSGD_KERNEL_LOCAL_STEP, hp.HPSGD_KERNEL_MERGE,
                                                                hp.HPSGD_KERNEL_MERGE_STEP, hp.HPSGD_KERNEL_ROUND))
        # the schedule under test really ran (launches of: local step, merge, merge + next step, whole round)
        if pipeline:
            assert ran == (T, 2 * T, 0, 0)          # one commit and one reduce per merge
        elif fuse == 2:
            assert ran == (0, 0, 0, T)              # one kernel per round, nothing else
        elif fuse == 1:
            assert ran == (1, 1, T - 1, 0)          # T-1 merges inside fused kernels + the last one alone
        else:
            assert ran == (T, T, 0, 0)
        # properties that hold at every one of the K x P elements, checked on the device: the run
        # ends with a merge, so every replica is a clone of w, and nothing is NaN or infinite
        w_all = torch.as_tensor(gu._RawDeviceArray(hp.hpsgd_get_global(), P_pad, "<f4"), device=gu.DEV)
        assert bool(torch.isfinite(w_all).all())
        for i in range(K):
            r_i, m_i = hp.hpsgd_get_replica(i)
            assert torch.equal(torch.as_tensor(gu._RawDeviceArray(r_i, P_pad, "<f4"), device=gu.DEV), w_all), \
                "replica %d is not a clone of the global model after the last merge" % i
            if m_i:
                assert bool(torch.isfinite(torch.as_tensor(gu._RawDeviceArray(m_i, P_pad, "<f4"), device=gu.DEV)).all())
        got = {"w": gu.dev_gather(hp.hpsgd_get_global(), P_pad, pos),
               "D": gu.dev_gather(hp.hpsgd_get_pending(), P_pad, pos)}
        for i in (0, K // 2, K - 1):
            r, m = hp.hpsgd_get_replica(i)
            got["r%d" % i] = gu.dev_gather(r, P_pad, pos)
            if m:
                got["m%d" % i] = gu.dev_gather(m, P_pad, pos)
    want = {"w": oracle.get_global(), "D": oracle.get_pending()}
    for i in (0, K // 2, K - 1):
        want["r%d" % i] = oracle.get_replica(i)
        if cfg.momentum:
            want["m%d" % i] = oracle.get_momentum(i)
    oracle.close()
    if master is not None:
        want["w_fp32_master"] = master.get_global()
        master.close()
    return idx, got, want


@pytest.mark.parametrize("fuse", [2, 0, 1])
@pytest.mark.parametrize("name", ["cfg4", "cfg5"])
def test_full_size_sampled_parity(name, fuse):
    """fuse = 2 (one kernel per round) is the configuration bench.py times by default; 0 (separate
    kernels on two streams) and 1 (merge carried into the next local step) are its other schedules."""
    cfg = workloads.get(name)
    idx, got, want = run_full(cfg, cfg.T, fuse, fp32_master=(name == "cfg5" and fuse == 2))
    assert idx.size > 250_000
    if "w_fp32_master" in want:
        # bf16-stored gradients against an fp32 master, the full T = 30 rounds of the GRU-shaped
        # workload (K = 16, momentum 0.9, sparse embedding rows): 1e-2 per parameter.  Parameters are
        # O(0.1); the denominator is floored at 1e-4 because a parameter that happens to sit near
        # zero has no meaningful relative error.
        master = want.pop("w_fp32_master")
        assert gu.max_rel_err(got["w"], master, floor=1e-4) <= 1e-2
        w0 = cfg.initial_global(idx).astype(np.float64)
        assert np.linalg.norm(got["w"] - master) <= 1e-2 * np.linalg.norm(master - w0)
    for key in got:
        # parameters and replicas to 1e-6 relative (floor 1e-6); the momentum and pending-change
        # buffers are compared at the scale of the quantity they hold
        floor = 1e-6 if key[0] in "wr" else 1e-9
        err = gu.max_rel_err(got[key], want[key], floor=floor)
        assert err <= 1e-6, "%s: max relative error %g" % (key, err)
        equal = np.mean(got[key].view(np.uint32) == want[key].view(np.uint32))
        # device and host log/cos may round a Gaussian differently once in ~1e8 draws
        assert equal >= 0.999, "%s: only %.6f of the sample is bit-equal" % (key, equal)


def test_full_size_sampled_parity_pipelined_schedule():
    """cfg4 under the paper's timeline: commit on the main stream, reduce on the side stream."""
    cfg = workloads.get("cfg4")
    idx, got, want = run_full(cfg, cfg.T, 0, pipeline=1)
    for key in got:
        assert np.array_equal(got[key].view(np.uint32), want[key].view(np.uint32)) or \
            gu.max_rel_err(got[key], want[key], floor=1e-6 if key[0] in "wr" else 1e-9) <= 1e-6, key


@pytest.mark.parametrize("fuse", [2, 0])
def test_largest_supported_parameter_count(fuse):
    """Two tensors that together reach just below the 2^32 parameters the library accepts, the first one
    ending beyond element 2^31: every 32-bit shortcut in the index arithmetic of the kernels, the
    generators or the layout would show here.  K = 2, plain SGD with weight decay (~100 GB on the device),
    three rounds, a stratified sample against the oracle, in the schedule bench.py times and as separate
    kernels."""
    from workloads.configs import Workload
    free, _ = torch.cuda.mem_get_info()
    if free < 120 << 30:
        pytest.skip("needs 120 GB of free device memory")
    cfg = Workload("max_size", K=2, sizes=(2_147_483_648 + 1001, 2_147_479_000), T=3, lr=0.05, momentum=0.0,
                   weight_decay=1e-3, seed=77, grad_kind="uniform", grad_scale=1e-2)
    assert cfg.P < 1 << 32 and cfg.layout.offsets[1] > 1 << 31
    idx, got, want = run_full(cfg, cfg.T, fuse)
    assert idx.size > 250_000 and int(idx.max()) > (1 << 32) - 10_000
    for key in got:
        assert np.array_equal(got[key].view(np.uint32), want[key].view(np.uint32)), key     # uniform gradients: exact
    torch.cuda.empty_cache()
