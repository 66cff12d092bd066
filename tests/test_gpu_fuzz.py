"""Random call sequences against the oracle: batched and per-worker local steps, merges
(also back to back), synchronisations, option changes and checkpoints, under every schedule
option.  Whatever the library defers, fuses or rebuilds internally, its state must equal the
oracle's bit for bit."""
import numpy as np
import pytest

import paper_2009_02701_b200 as hp
from tests import gpu_util as gu
from workloads.configs import Workload

pytestmark = pytest.mark.gpu


def compare(cfg, o, what):
    w, D, rs, ms = gu.gpu_state(cfg)
    gu.assert_bitwise(w, o.get_global(), "%s: global model" % what)
    gu.assert_bitwise(D, o.get_pending(), "%s: pending change" % what)
    for i in range(cfg.K):
        gu.assert_bitwise(rs[i], o.get_replica(i), "%s: replica %d" % (what, i))
        if cfg.momentum:
            gu.assert_bitwise(ms[i], o.get_momentum(i), "%s: momentum %d" % (what, i))


@pytest.mark.parametrize("seed", range(24))
def test_random_call_sequences(seed):
    rng = np.random.default_rng(1000 + seed)
    K = int(rng.choice([1, 2, 3, 4, 5, 8, 16]))
    sizes = [int(x) for x in rng.integers(1, 20_000, size=int(rng.integers(1, 5)))]
    momentum = float(rng.choice([0.0, 0.9]))
    wd = float(rng.choice([0.0, 1e-3]))
    pipeline = int(rng.random() < 0.25)
    staleness = 1 if pipeline else int(rng.choice([0, 1]))
    cfg = Workload("fuzz", K=K, sizes=tuple(sizes), T=0, lr=0.05, momentum=momentum, weight_decay=wd,
                   seed=100 + seed, grad_kind="gauss", grad_scale=1e-2, staleness=staleness)
    fuse = int(rng.choice([0, 1, 2]))
    o = gu.oracle_for(cfg, staleness)
    keep = []
    step = 0
    with gu.session(cfg, staleness=staleness, overlap=int(rng.choice([0, 1])), chunks=1 if pipeline else int(rng.choice([1, 3])),
                    fuse=fuse, pipeline=pipeline, lend_arena=bool(rng.random() < 0.5), streams=bool(rng.random() < 0.5)):
        for op_no in range(30):
            op = rng.choice(["all", "all", "all", "some", "merge", "merge", "merge", "sync", "look", "chunks", "ckpt"])
            if op == "all":
                inputs = [gu.host_inputs(cfg, i, step) for i in range(K)]
                stacked = np.stack([inp["padded"] for inp in inputs])
                keep.append(gu.to_device(stacked.reshape(-1)))
                hp.hpsgd_local_step_all(keep[-1], stacked.shape[1] * 4)
                for i, inp in enumerate(inputs):
                    o.local_step(i, inp["flat"])
                step += 1
            elif op == "some":
                for i in rng.permutation(K)[:int(rng.integers(1, K + 1))]:
                    inp = gu.host_inputs(cfg, int(i), step)
                    gu.gpu_step(cfg, int(i), inp, keep)
                    o.local_step(int(i), inp["flat"])
                step += 1
            elif op == "merge":
                hp.hpsgd_sync_merge()
                o.sync_merge()
            elif op == "sync":
                hp.hpsgd_synchronize()
            elif op == "look":
                compare(cfg, o, "seed %d after op %d" % (seed, op_no))
            elif op == "chunks" and not pipeline:
                hp.hpsgd_set_option(hp.HPSGD_OPT_CHUNKS, int(rng.choice([1, 2, 5])))
                hp.hpsgd_set_option(hp.HPSGD_OPT_FUSE, int(rng.choice([0, 1, 2])))
            elif op == "ckpt":
                blob = np.empty(hp.hpsgd_state_bytes(), dtype=np.uint8)
                hp.hpsgd_export_state(blob)
                # wreck the live state, then restore it from the blob
                hp.hpsgd_set_global_host(np.zeros(cfg.P, dtype=np.float32))
                hp.hpsgd_import_state(blob)
        compare(cfg, o, "seed %d at the end" % seed)
    o.close()


@pytest.mark.parametrize("seed", range(8))
def test_random_call_sequences_gradient_accumulation_form(seed):
    """The same idea for Algorithms 2/3 as printed (explicit accumulated gradients)."""
    from oracle.ref import RefHPSGDAccum
    rng = np.random.default_rng(5000 + seed)
    K = int(rng.choice([1, 3, 4, 8, 16]))
    sizes = [int(x) for x in rng.integers(1, 20_000, size=int(rng.integers(1, 4)))]
    cfg = Workload("fuzz_acc", K=K, sizes=tuple(sizes), T=0, lr=0.05, momentum=0.0, weight_decay=0.0,
                   seed=200 + seed, grad_kind="uniform", grad_scale=1e-2)
    o = RefHPSGDAccum(cfg.P, K, cfg.lr)
    o.set_global(cfg.initial_global())
    keep = []
    step = 0

    def look(what):
        w, ghat, rs, accs = gu.gpu_state(cfg)
        gu.assert_bitwise(w, o.get_global(), what + ": global model")
        gu.assert_bitwise(ghat, o.get_synced(), what + ": AllReduce result")
        for i in range(K):
            gu.assert_bitwise(rs[i], o.get_replica(i), what + ": replica %d" % i)
            gu.assert_bitwise(accs[i], o.get_accumulated(i), what + ": accumulated gradient %d" % i)

    with gu.session(cfg, overlap=int(rng.choice([0, 1])), chunks=int(rng.choice([1, 3])), fuse=int(rng.choice([0, 1])),
                    form=hp.HPSGD_FORM_GRADIENT_ACCUMULATION):
        for op_no in range(25):
            op = rng.choice(["all", "all", "some", "merge", "merge", "sync", "look"])
            if op == "all":
                inputs = [gu.host_inputs(cfg, i, step) for i in range(K)]
                stacked = np.stack([inp["padded"] for inp in inputs])
                keep.append(gu.to_device(stacked.reshape(-1)))
                hp.hpsgd_local_step_all(keep[-1], stacked.shape[1] * 4)
                for i, inp in enumerate(inputs):
                    o.local_step(i, inp["flat"])
                step += 1
            elif op == "some":
                for i in rng.permutation(K)[:int(rng.integers(1, K + 1))]:
                    inp = gu.host_inputs(cfg, int(i), step)
                    gu.gpu_step(cfg, int(i), inp, keep)
                    o.local_step(int(i), inp["flat"])
                step += 1
            elif op == "merge":
                hp.hpsgd_sync_merge()
                o.sync_merge()
            elif op == "sync":
                hp.hpsgd_synchronize()
            else:
                look("seed %d after op %d" % (seed, op_no))
        look("seed %d at the end" % seed)
    o.close()


@pytest.mark.parametrize("seed", range(12))
def test_random_call_sequences_sparse_rows(seed):
    """The same with a sparse-row tensor in the layout: batched and per-worker sparse-row steps mixed with
    dense ones (which hold back, flush and share the per-worker row -> slot maps differently), fp32 and bf16."""
    rng = np.random.default_rng(9000 + seed)
    K = int(rng.choice([2, 3, 4, 8, 16]))
    rows, cols = int(rng.integers(5, 200)), int(rng.choice([8, 16, 64]))
    sizes = [int(rng.integers(1, 5000)), rows * cols, int(rng.integers(1, 5000))]
    momentum = float(rng.choice([0.0, 0.9]))
    wd = float(rng.choice([0.0, 1e-3]))
    pipeline = int(rng.random() < 0.2)
    cfg = Workload("fuzz_sparse", K=K, sizes=tuple(sizes), T=0, lr=0.05, momentum=momentum, weight_decay=wd,
                   seed=300 + seed, grad_kind="gauss", grad_scale=1e-2, grad_dtype=str(rng.choice(["f32", "bf16"])),
                   sparse=(1, rows, cols))
    o = gu.oracle_for(cfg)
    keep = []
    step = 0
    with gu.session(cfg, overlap=int(rng.choice([0, 1])), chunks=1 if pipeline else int(rng.choice([1, 3])),
                    fuse=int(rng.choice([0, 1, 2])), pipeline=pipeline, lend_arena=bool(rng.random() < 0.5)):
        for op_no in range(30):
            op = rng.choice(["all_ex", "all_ex", "all_ex", "some_ex", "some_dense", "merge", "merge", "merge", "sync",
                             "look", "fuse"])
            if op == "all_ex":
                descs = []
                for i in range(K):
                    inp = gu.host_inputs(cfg, i, step)
                    g, idx, vals = gu.to_device(inp["padded"]), gu.to_device(inp["rows"]), gu.to_device(inp["vals"].reshape(-1))
                    keep += [g, idx, vals]
                    descs.append(hp.make_desc(g, idx, len(inp["rows"]), vals))
                    gu.oracle_step(o, cfg, i, inp)
                hp.hpsgd_local_step_all_ex(descs)
                step += 1
            elif op in ("some_ex", "some_dense"):
                for i in rng.permutation(K)[:int(rng.integers(1, K + 1))]:
                    inp = gu.host_inputs(cfg, int(i), step)
                    gu.gpu_step(cfg, int(i), inp, keep, sparse_api=(op == "some_ex"))
                    gu.oracle_step(o, cfg, int(i), inp, sparse_api=(op == "some_ex"))
                step += 1
            elif op == "merge":
                hp.hpsgd_sync_merge()
                o.sync_merge()
            elif op == "sync":
                hp.hpsgd_synchronize()
            elif op == "look":
                compare(cfg, o, "seed %d after op %d" % (seed, op_no))
            elif op == "fuse" and not pipeline:
                hp.hpsgd_set_option(hp.HPSGD_OPT_FUSE, int(rng.choice([0, 1, 2])))
        compare(cfg, o, "seed %d at the end" % seed)
    o.close()
