"""CUDA path (through the C ABI) against the CPU oracle, element by element."""
import numpy as np
import pytest
import torch

import paper_2009_02701_b200 as hp
import workloads
from tests import gpu_util as gu
from tests.oracle_pins import GOLDEN, parse_worked
from workloads.configs import Workload

pytestmark = pytest.mark.gpu


def small(name, K, sizes, T=4, lr=0.1, momentum=0.9, wd=0.0, seed=7, kind="gauss", scale=1e-2,
          dtype="f32", sparse=None, staleness=1):
    return Workload(name, K=K, sizes=tuple(sizes), T=T, lr=lr, momentum=momentum, weight_decay=wd,
                    seed=seed, grad_kind=kind, grad_scale=scale, grad_dtype=dtype, sparse=sparse,
                    staleness=staleness)


def test_worked_examples_through_the_abi():
    """The hand-worked K=2, P=4 rounds (Algorithms 2/3, Eq. 1) reproduced by the kernels."""
    import os
    mu, w0, grads, cases = parse_worked(os.path.join(GOLDEN, "worked_k2_p4.txt"))
    for c in cases:
        cfg = small("worked", 2, [4], lr=mu, momentum=c["beta"], wd=c["lambda"], staleness=c["staleness"])
        with gu.session(cfg):
            hp.hpsgd_set_global_host(np.array(w0, dtype=np.float32))
            for t in range(3):
                keep = []
                for i in range(2):
                    g = np.zeros(32, dtype=np.float32)
                    g[:4] = grads[(t, i)]
                    keep.append(gu.to_device(g))
                    hp.hpsgd_local_step(i, keep[-1])
                w, D, rs, ms = gu.gpu_state(cfg)
                for i in range(2):
                    np.testing.assert_array_equal(rs[i], np.float32(c["r"][(t, i)]))
                hp.hpsgd_sync_merge()
                w, D, rs, ms = gu.gpu_state(cfg)
                np.testing.assert_array_equal(D, np.float32(c["D"][t]))
                np.testing.assert_array_equal(w, np.float32(c["w"][t]))
                np.testing.assert_array_equal(rs[0], w)
                np.testing.assert_array_equal(rs[1], w)


def test_cfg1_full():
    cfg = workloads.get("cfg1")
    got, want = gu.run_both(cfg, cfg.T, check_each_round=True)
    assert gu.max_rel_err(got, want) <= 1e-6


@pytest.mark.parametrize("P", [1, 3, 5, 31, 33, 127, 129, 1000, 4097, 70001])
@pytest.mark.parametrize("K,momentum,wd", [(1, 0.0, 0.0), (2, 0.9, 0.0), (3, 0.9, 5e-4), (5, 0.0, 1e-3),
                                           (4, 0.9, 0.0), (8, 0.9, 5e-4), (16, 0.9, 0.0), (9, 0.5, 0.0)])
def test_odd_sizes(P, K, momentum, wd):
    cfg = small("odd", K, [P], T=3, momentum=momentum, wd=wd)
    gu.run_both(cfg, cfg.T, check_each_round=(P <= 129))


def test_multi_tensor_ragged_layout():
    rng = np.random.default_rng(5)
    sizes = [int(x) for x in rng.integers(1, 3000, size=37)] + [64, 32, 1, 33, 100_003]
    cfg = small("ragged", 6, sizes, T=5, wd=5e-4)
    gu.run_both(cfg, cfg.T, session_kw=dict(lend_arena=True, canary=True, streams=True))


@pytest.mark.parametrize("staleness", [0, 1])
def test_staleness_modes_and_many_local_steps(staleness):
    cfg = small("hsteps", 4, [5000, 77], T=4, staleness=staleness)
    gu.run_both(cfg, cfg.T, staleness=staleness, steps_per_round=3, check_each_round=True)


def test_worker_without_a_step_contributes_zero():
    cfg = small("skip", 4, [3000], T=3)
    gu.run_both(cfg, cfg.T, skip_worker=2)


@pytest.mark.parametrize("overlap,chunks,batched", [(0, 1, False), (1, 1, False), (1, 3, False), (1, 7, True),
                                                    (0, 5, True), (1, 64, True)])
def test_schedule_does_not_change_results(overlap, chunks, batched):
    cfg = small("sched", 8, [300_000, 1234, 99_999], T=6, wd=1e-4)
    gu.run_both(cfg, cfg.T, overlap=overlap, chunks=chunks, batched=batched)


@pytest.mark.parametrize("batched", [False, True])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_sparse_rows_and_bf16_small(batched, dtype):
    # embedding-like [rows x cols] tensor in the middle of the layout, ~10 % rows active
    cfg = small("sparse", 5, [1000, 300 * 64, 777, 64], T=4, dtype=dtype, sparse=(1, 300, 64), scale=1e-3)
    gu.run_both(cfg, cfg.T, batched=batched, chunks=3)


def test_sparse_equals_dense_with_zero_rows():
    cfg = small("sparse_dense", 3, [128 * 16, 50], T=3, dtype="bf16", sparse=(0, 128, 16), scale=1e-3)
    results = []
    for sparse_api in (True, False):
        with gu.session(cfg):
            for t in range(cfg.T):
                keep = []
                for i in range(cfg.K):
                    gu.gpu_step(cfg, i, gu.host_inputs(cfg, i, t), keep, sparse_api=sparse_api)
                hp.hpsgd_sync_merge()
                hp.hpsgd_synchronize()
            results.append(gu.gpu_state(cfg))
    for a, b in zip(results[0][2] + results[0][3] + [results[0][0]], results[1][2] + results[1][3] + [results[1][0]]):
        gu.assert_bitwise(a, b, "sparse vs dense-with-zero-rows")


def test_bf16_gradients_against_fp32_master():
    """Stored-bf16 gradients vs an oracle fed the un-rounded fp32 gradients: within 1e-2."""
    cfg = small("bf16master", 4, [50_000], T=10, dtype="bf16", scale=1e-3, lr=0.01)
    o = gu.oracle_for(cfg)
    with gu.session(cfg):
        for t in range(cfg.T):
            keep = []
            for i in range(cfg.K):
                gu.gpu_step(cfg, i, gu.host_inputs(cfg, i, t), keep)
                o.local_step(i, cfg.gradient(i, t))              # fp32, not rounded to bf16
            hp.hpsgd_sync_merge()
            o.sync_merge()
            hp.hpsgd_synchronize()
        got = gu.gpu_global(cfg)
    want = o.get_global()
    # bf16 keeps 8 significand bits: each stored gradient is within 2^-9 of its fp32 value, so
    # the accumulated change agrees to well under 1e-2 of its size, and each parameter to 1e-2
    # relative.  Parameters are O(0.1); the denominator is floored at 1e-4 (0.1 % of that
    # scale) because a parameter that happens to sit at ~1e-6 has no meaningful relative error.
    assert gu.max_rel_err(got, want, floor=1e-4) <= 1e-2
    w0 = cfg.initial_global().astype(np.float64)
    change_err = np.linalg.norm((got - w0) - (want - w0)) / np.linalg.norm(want - w0)
    assert change_err <= 1e-2


def test_device_generator_matches_host_generator():
    for cfg in (small("gen_u", 3, [1000, 37, 5000], kind="uniform", scale=1e-2, seed=1),
                small("gen_g", 3, [1000, 37, 5000], kind="gauss", scale=1e-3, seed=2),
                small("gen_b", 3, [40 * 8, 100, 7], kind="gauss", scale=1e-3, seed=5, dtype="bf16",
                      sparse=(0, 40, 8))):
        with gu.session(cfg):
            gu.assert_bitwise(gu.gpu_global(cfg), cfg.initial_global(), "initial model from the device hash")
            kind = hp.HPSGD_GEN_UNIFORM if cfg.grad_kind == "uniform" else hp.HPSGD_GEN_GAUSS
            for worker, step in ((0, 0), (2, 9), (1, 1000)):
                want = cfg.layout.pack(cfg.stored_gradient(worker, step))
                if cfg.grad_dtype == "bf16":
                    out = torch.empty(cfg.layout.P_pad, dtype=torch.int16, device=gu.DEV)
                else:
                    out = torch.empty(cfg.layout.P_pad, dtype=torch.float32, device=gu.DEV)
                hp.hpsgd_gen_grads(out, worker, step, kind, cfg.grad_scale)
                hp.hpsgd_synchronize()
                got = out.cpu().numpy()
                if cfg.grad_dtype == "bf16":
                    got = got.view(np.uint16)
                    off = np.abs(got.astype(np.int64) - want.astype(np.int64))
                else:
                    off = np.abs(got.view(np.int32).astype(np.int64) - want.view(np.int32).astype(np.int64))
                if cfg.grad_kind == "uniform":
                    assert off.max() == 0
                else:
                    # host and device log/cos may differ in the last binary64 bit
                    assert off.max() <= 1 and (off > 0).mean() <= 1e-4
                if cfg.sparse:
                    rows = cfg.sparse_rows(worker, step)
                    idx = gu.to_device(rows)
                    vals = torch.empty(len(rows) * cfg.sparse[2], dtype=torch.int16, device=gu.DEV)
                    hp.hpsgd_gen_row_vals(vals, worker, step, kind, cfg.grad_scale, idx, len(rows))
                    hp.hpsgd_synchronize()
                    wantv = gu.host_inputs(cfg, worker, step)["vals"].reshape(-1)
                    offv = np.abs(vals.cpu().numpy().view(np.uint16).astype(np.int64) - wantv.astype(np.int64))
                    assert offv.max() <= 1 and (offv > 0).mean() <= 1e-4


@pytest.mark.parametrize("name", ["cfg2", "cfg3"])
def test_resnet_like_configs_full(name):
    """Full parameter count, every round, every element compared."""
    cfg = workloads.get(name)
    got, want = gu.run_both(cfg, cfg.T, batched=(name == "cfg3"), chunks=4)
    assert gu.max_rel_err(got, want) <= 1e-6


def test_host_buffer_entry_point():
    cfg = small("hostbuf", 3, [200_000, 333], T=3)
    o = gu.oracle_for(cfg)
    with gu.session(cfg):
        pinned = [torch.empty(cfg.layout.P_pad, dtype=torch.float32).pin_memory() for _ in range(cfg.K)]
        for t in range(cfg.T):
            for i in range(cfg.K):
                inp = gu.host_inputs(cfg, i, t)
                pinned[i].numpy()[:] = inp["padded"]
                hp.hpsgd_local_step_host(i, pinned[i])
                o.local_step(i, inp["flat"])
            hp.hpsgd_sync_merge()
            o.sync_merge()
            hp.hpsgd_synchronize()
        gu.assert_bitwise(gu.gpu_global(cfg), o.get_global(), "global via host buffers")


def test_argument_errors_enqueue_nothing():
    cfg = small("errors", 2, [1000], T=1)
    with gu.session(cfg):
        before = hp.hpsgd_launch_count()
        g = torch.zeros(cfg.layout.P_pad + 8, dtype=torch.float32, device=gu.DEV)
        for call, code in ((lambda: hp.hpsgd_local_step(2, g), hp.HPSGD_E_BADARG),
                           (lambda: hp.hpsgd_local_step(-1, g), hp.HPSGD_E_BADARG),
                           (lambda: hp.hpsgd_local_step(0, None), hp.HPSGD_E_BADARG),
                           (lambda: hp.hpsgd_local_step(0, g.data_ptr() + 4), hp.HPSGD_E_BADARG),
                           (lambda: hp.hpsgd_init(10, 2, 0.1, 0.0, 1), hp.HPSGD_E_STATE),
                           (lambda: hp.hpsgd_set_option(hp.HPSGD_OPT_CHUNKS, 0), hp.HPSGD_E_BADARG),
                           (lambda: hp.hpsgd_set_option(99, 0), hp.HPSGD_E_BADARG),
                           (lambda: hp.hpsgd_local_step_ex(0, hp.make_desc(g)), hp.HPSGD_E_STATE),
                           (lambda: hp.hpsgd_set_sparse_segment(0, 10, 10), hp.HPSGD_E_BADARG)):
            with pytest.raises(hp.HpsgdError) as err:
                call()
            assert err.value.code == code
        assert hp.hpsgd_launch_count() == before
    # an arena that is too small is refused before anything is touched
    hp.hpsgd_destroy()
    buf = torch.empty(4096, dtype=torch.uint8, device=gu.DEV)
    base = buf.data_ptr() + (-buf.data_ptr()) % 256
    hp.hpsgd_bind(base, 1024, None, None)
    with pytest.raises(hp.HpsgdError) as err:
        hp.hpsgd_init(100_000, 4, 0.1, 0.9, 1)
    assert err.value.code == hp.HPSGD_E_NOMEM
    hp.hpsgd_destroy()


def test_a_failed_call_does_not_poison_the_next_one():
    """A CUDA call that fails for its arguments (here: an allocation far beyond the device) is
    reported by the call that made it and by no later one."""
    hp.hpsgd_destroy()
    with pytest.raises(hp.HpsgdError) as err:
        hp.hpsgd_init((1 << 32) - 64, 64, 0.1, 0.9, 1)          # ~2.2 TB of state
    assert err.value.code == hp.HPSGD_E_NOMEM
    cfg = small("after_failure", 3, [5000, 33], T=2)
    gu.run_both(cfg, cfg.T)                                       # every call returns HPSGD_OK, results exact
    gu.run_both(cfg, cfg.T, batched=True)


def test_import_checks_the_staleness_it_is_given():
    """A checkpoint written without the one-synchronisation delay cannot be resumed under the
    pipelined schedule (whose commit kernel only knows the delayed form), and a blob whose
    staleness field is neither 0 nor 1 is refused."""
    cfg = small("ckpt_stale", 4, [3000, 17], T=2, staleness=0)
    with gu.session(cfg, staleness=0):
        keep = []
        for i in range(cfg.K):
            gu.gpu_step(cfg, i, gu.host_inputs(cfg, i, 0), keep)
        hp.hpsgd_sync_merge()
        blob = np.empty(hp.hpsgd_state_bytes(), dtype=np.uint8)
        hp.hpsgd_export_state(blob)
    delayed = small("ckpt_stale", 4, [3000, 17], T=2, staleness=1)
    with gu.session(delayed, pipeline=1):
        before = gu.gpu_state(delayed)
        with pytest.raises(hp.HpsgdError) as err:
            hp.hpsgd_import_state(blob)
        assert err.value.code == hp.HPSGD_E_BADARG
        after = gu.gpu_state(delayed)
        gu.assert_bitwise(after[0], before[0], "global model after a refused import")
    with gu.session(delayed):
        broken = blob.copy()
        # header: magic (8), P, P_pad, merges (3 x 8), K, form, has_aux (3 x 4), then staleness
        broken[44:48] = np.frombuffer(np.int32(7).tobytes(), dtype=np.uint8)
        with pytest.raises(hp.HpsgdError) as err:
            hp.hpsgd_import_state(broken)
        assert err.value.code == hp.HPSGD_E_BADARG
        hp.hpsgd_import_state(blob)                               # the plain schedule takes the staleness of the blob


# ---------------------------------------------------------------- merge fused into the next local step
@pytest.mark.parametrize("K,momentum,wd,staleness", [(16, 0.9, 0.0, 1), (8, 0.9, 5e-4, 1), (4, 0.0, 0.0, 1),
                                                      (3, 0.9, 0.0, 1), (5, 0.0, 1e-3, 0), (9, 0.5, 0.0, 1),
                                                      (1, 0.9, 0.0, 0), (16, 0.9, 1e-4, 0)])
def test_fused_merge_step_matches_oracle(K, momentum, wd, staleness):
    cfg = small("fused", K, [70_001, 33, 4096], T=5, momentum=momentum, wd=wd, staleness=staleness)
    got, want = gu.run_both(cfg, cfg.T, staleness=staleness, fuse=1, batched=True, chunks=3)
    assert gu.max_rel_err(got, want) <= 1e-6


def test_fused_launches_one_kernel_per_round():
    cfg = small("fused_count", 8, [50_000], T=4)
    with gu.session(cfg, fuse=1):
        stacked = np.stack([gu.host_inputs(cfg, i, 0)["padded"] for i in range(cfg.K)])
        g = gu.to_device(stacked.reshape(-1))
        hp.hpsgd_local_step_all(g, stacked.shape[1] * 4)
        hp.hpsgd_sync_merge()
        hp.hpsgd_synchronize()                       # launches that merge on its own
        base = hp.hpsgd_launch_count()
        for t in range(4):
            hp.hpsgd_local_step_all(g, stacked.shape[1] * 4)
            hp.hpsgd_sync_merge()
        assert hp.hpsgd_launch_count() - base == 4  # 1 local step, then 3 fused merge+step kernels
        hp.hpsgd_flush()
        assert hp.hpsgd_launch_count() - base == 5  # the last merge
        hp.hpsgd_flush()
        assert hp.hpsgd_launch_count() - base == 5


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_fused_sparse_rows(dtype):
    cfg = small("fused_sparse", 5, [1000, 300 * 64, 777, 64], T=5, dtype=dtype, sparse=(1, 300, 64), scale=1e-3)
    gu.run_both(cfg, cfg.T, fuse=1, batched=True, chunks=2)


def test_fused_mixed_with_other_calls():
    """Per-worker steps, several steps per round and back-to-back merges all force the
    deferred merge out on its own; the results stay those of the oracle."""
    cfg = small("fused_mixed", 4, [30_000, 17], T=3, wd=1e-4)
    gu.run_both(cfg, cfg.T, fuse=1, batched=False)                        # never fuses
    gu.run_both(cfg, cfg.T, fuse=1, batched=True, steps_per_round=3)      # first step of a round fuses
    o = gu.oracle_for(cfg)
    with gu.session(cfg, fuse=1):
        keep = []
        for t in range(3):
            for i in range(cfg.K):
                inp = gu.host_inputs(cfg, i, t)
                gu.gpu_step(cfg, i, inp, keep)
                o.local_step(i, inp["flat"])
            hp.hpsgd_sync_merge()
            hp.hpsgd_sync_merge()                                         # a merge with no step in between
            o.sync_merge()
            o.sync_merge()
        w, D, rs, ms = gu.gpu_state(cfg)
        gu.assert_bitwise(w, o.get_global(), "global after back-to-back merges")
        gu.assert_bitwise(D, o.get_pending(), "pending change after back-to-back merges")


# ---------------------------------------------------------------- Algorithms 2/3 as printed (accumulated gradients)
@pytest.mark.parametrize("K,sizes,batched,chunks,H", [(4, [1_048_576], True, 1, 1), (2, [4], False, 1, 1),
                                                      (16, [70_001, 33, 4096], True, 3, 1), (3, [5000, 77], False, 2, 3),
                                                      (5, [129], False, 1, 2), (8, [300_000], True, 5, 1)])
def test_gradient_accumulation_form(K, sizes, batched, chunks, H):
    cfg = small("accum", K, sizes, T=4, lr=0.01, momentum=0.0, kind="uniform", scale=1e-2, seed=1)
    got, want = gu.run_both_accum(cfg, cfg.T, batched=batched, chunks=chunks, steps_per_round=H)
    assert gu.max_rel_err(got, want) <= 1e-6


def test_gradient_accumulation_form_sparse_bf16():
    cfg = small("accum_sparse", 4, [1000, 200 * 32, 55], T=3, lr=0.01, momentum=0.0, dtype="bf16",
                sparse=(1, 200, 32), scale=1e-3)
    gu.run_both_accum(cfg, cfg.T)


def test_gradient_accumulation_form_agrees_with_replica_change_form():
    """Eq. 1 == Eq. 2: both forms give the same global model up to rounding."""
    cfg = small("forms", 8, [100_000], T=6, lr=0.01, momentum=0.0, kind="uniform", scale=1e-2, seed=1)
    a, _ = gu.run_both_accum(cfg, cfg.T, batched=True)
    b, _ = gu.run_both(cfg, cfg.T, batched=True)
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-7)


def test_gradient_accumulation_form_rejects_momentum():
    hp.hpsgd_destroy()
    hp.hpsgd_set_form(hp.HPSGD_FORM_GRADIENT_ACCUMULATION)
    with pytest.raises(hp.HpsgdError) as err:
        hp.hpsgd_init(1000, 2, 0.1, 0.9, 1)
    assert err.value.code == hp.HPSGD_E_BADARG
    hp.hpsgd_init(1000, 2, 0.1, 0.0, 1)
    with pytest.raises(hp.HpsgdError):
        hp.hpsgd_set_option(hp.HPSGD_OPT_WEIGHT_DECAY, 1e-3)
    hp.hpsgd_destroy()
    with pytest.raises(hp.HpsgdError):
        hp.hpsgd_set_form(7)


# ---------------------------------------------------------------- Local SGD (Algorithm 1) and SSGD as modes
@pytest.mark.parametrize("gamma", [1, 8])
def test_local_sgd_and_ssgd_modes(gamma):
    """staleness 0 with gamma plain-SGD local steps per merge is Algorithm 1 (the global model is
    the mean of the K local models); gamma = 1 is synchronous SGD on the mean gradient."""
    cfg = small("localsgd", 4, [20_000, 31], T=3, lr=0.01, momentum=0.0, kind="uniform", scale=1e-2, seed=9,
                staleness=0)
    w = cfg.initial_global().astype(np.float64)
    with gu.session(cfg, staleness=0):
        step = 0
        for loop in range(cfg.T):
            local = np.repeat(w[None, :], cfg.K, axis=0)
            keep = []
            for e in range(gamma):
                for i in range(cfg.K):
                    inp = gu.host_inputs(cfg, i, step)
                    gu.gpu_step(cfg, i, inp, keep)
                    local[i] -= np.float64(np.float32(cfg.lr)) * inp["flat"]
                step += 1
            hp.hpsgd_sync_merge()
            hp.hpsgd_synchronize()
            w = local.mean(axis=0)                      # AllReduce(model) / n, Algorithm 1
            np.testing.assert_allclose(gu.gpu_global(cfg), w, rtol=0, atol=2e-7)
    gu.run_both(cfg, cfg.T, staleness=0, steps_per_round=gamma)     # and bit-exact against the oracle


# ---------------------------------------------------------------- pipelined synchronisation (the paper's timeline)
@pytest.mark.parametrize("K,momentum,wd,H,batched", [(16, 0.9, 0.0, 1, True), (8, 0.9, 5e-4, 3, False), (4, 0.0, 0.0, 1, False),
                                                     (3, 0.9, 0.0, 2, True), (5, 0.0, 1e-3, 1, True), (1, 0.9, 0.0, 1, False)])
def test_pipelined_sync_matches_oracle(K, momentum, wd, H, batched):
    cfg = small("pipe", K, [70_001, 33, 4096], T=5, momentum=momentum, wd=wd)
    gu.run_both(cfg, cfg.T, pipeline=1, batched=batched, steps_per_round=H)
    gu.run_both(cfg, 3, pipeline=1, batched=batched, steps_per_round=H, check_each_round=True,
                session_kw=dict(lend_arena=True, canary=True, streams=True))


def test_pipelined_sync_idle_worker_and_sparse_rows():
    cfg = small("pipe_skip", 4, [3000], T=4)
    gu.run_both(cfg, cfg.T, pipeline=1, skip_worker=2, check_each_round=True)
    cfg = small("pipe_sparse", 5, [1000, 300 * 64, 777, 64], T=4, dtype="bf16", sparse=(1, 300, 64), scale=1e-3)
    gu.run_both(cfg, cfg.T, pipeline=1, batched=True)
    gu.run_both(cfg, cfg.T, pipeline=1, batched=False)


def test_pipelined_sync_argument_checks():
    hp.hpsgd_destroy()
    hp.hpsgd_set_pipeline(1)
    hp.hpsgd_set_form(hp.HPSGD_FORM_GRADIENT_ACCUMULATION)
    with pytest.raises(hp.HpsgdError):
        hp.hpsgd_init(1000, 2, 0.1, 0.0, 1)
    hp.hpsgd_destroy()
    hp.hpsgd_set_pipeline(1)
    with pytest.raises(hp.HpsgdError) as err:
        hp.hpsgd_init(1000, 33, 0.1, 0.0, 1)
    assert err.value.code == hp.HPSGD_E_UNSUPPORTED
    hp.hpsgd_init(1000, 4, 0.1, 0.0, 1)
    for key, val in ((hp.HPSGD_OPT_STALENESS, 0), (hp.HPSGD_OPT_CHUNKS, 4)):
        with pytest.raises(hp.HpsgdError):
            hp.hpsgd_set_option(key, val)
    hp.hpsgd_destroy()


# ---------------------------------------------------------------- checkpoint
@pytest.mark.parametrize("mode", ["plain", "fuse", "round", "pipeline", "accum"])
def test_export_import_resumes_bit_identically(mode):
    momentum = 0.0 if mode == "accum" else 0.9
    cfg = small("ckpt", 4, [20_000, 77], T=6, momentum=momentum, lr=0.05)
    kw = dict(fuse={"fuse": 1, "round": 2}.get(mode, 0), pipeline=int(mode == "pipeline"),
              form=hp.HPSGD_FORM_GRADIENT_ACCUMULATION if mode == "accum" else 0)

    def rounds(t0, t1, keep):
        for t in range(t0, t1):
            stacked = np.stack([gu.host_inputs(cfg, i, t)["padded"] for i in range(cfg.K)])
            keep.append(gu.to_device(stacked.reshape(-1)))
            hp.hpsgd_local_step_all(keep[-1], stacked.shape[1] * 4)
            hp.hpsgd_sync_merge()

    with gu.session(cfg, **kw):
        keep = []
        rounds(0, cfg.T, keep)
        straight = gu.gpu_state(cfg)
    with gu.session(cfg, **kw):
        keep = []
        rounds(0, 3, keep)
        blob = np.empty(hp.hpsgd_state_bytes(), dtype=np.uint8)
        hp.hpsgd_export_state(blob)
    with gu.session(cfg, **kw):
        with pytest.raises(hp.HpsgdError):
            hp.hpsgd_import_state(blob[:100])
        hp.hpsgd_import_state(blob)
        assert hp.hpsgd_get_sizes()[3] == 3
        keep = []
        rounds(3, cfg.T, keep)
        resumed = gu.gpu_state(cfg)
    gu.assert_bitwise(resumed[0], straight[0], "global model after resume")
    gu.assert_bitwise(resumed[1], straight[1], "pending change after resume")
    for a, b in zip(resumed[2] + resumed[3], straight[2] + straight[3]):
        gu.assert_bitwise(a, b, "replica / momentum after resume")


def test_more_workers_than_one_batched_launch_addresses():
    """K = 40 > 32: batched calls are issued in groups of 32 workers, the fused path steps aside."""
    cfg = small("k40", 40, [5000, 33], T=3, momentum=0.9)
    gu.run_both(cfg, cfg.T, batched=True)
    gu.run_both(cfg, cfg.T, batched=True, fuse=1, chunks=2)
    gu.run_both(cfg, cfg.T, batched=True, fuse=2)
    gu.run_both(cfg, cfg.T, batched=False)


# ---------------------------------------------------------------- one kernel per round, lazy clones
@pytest.mark.parametrize("K,momentum,wd,staleness,H", [(16, 0.9, 0.0, 1, 1), (8, 0.9, 5e-4, 1, 1), (4, 0.5, 1e-3, 0, 1),
                                                        (16, 0.9, 0.0, 1, 2), (3, 0.9, 0.0, 1, 1), (8, 0.0, 0.0, 1, 1),
                                                        (1, 0.9, 0.0, 1, 1), (5, 0.0, 1e-3, 0, 3), (9, 0.9, 0.0, 1, 1),
                                                        (32, 0.9, 0.0, 1, 1), (17, 0.0, 0.0, 1, 2)])
def test_round_kernel_matches_oracle(K, momentum, wd, staleness, H):
    """HPSGD_OPT_FUSE = 2: the batched local step runs inside the kernel of the merge that follows it
    and no replica row is written; with several steps per period only the last one is fused and the
    earlier ones read w (the lazy clone) or their row.  All of it bit-identical."""
    cfg = small("round", K, [70_001, 33, 4096], T=6, momentum=momentum, wd=wd, staleness=staleness)
    gu.run_both(cfg, cfg.T, staleness=staleness, fuse=2, batched=True, chunks=2, steps_per_round=H)
    gu.run_both(cfg, 3, staleness=staleness, fuse=2, batched=True, steps_per_round=H, check_each_round=True,
                session_kw=dict(lend_arena=True, canary=True, streams=True))


@pytest.mark.parametrize("K", [1, 2, 3, 5, 6, 7, 9, 10, 11, 12, 13, 14, 15, 17, 20, 23, 24, 31])
def test_round_kernel_any_worker_count(K):
    """Every way the whole-round kernel cuts K workers into batches: fewer workers than a batch holds (one
    batch of exactly K), a multiple of the batch size, and the rest (batches of as equal a size as possible),
    for gradients and optimisers of different register weight, with one step per period (replicas read
    from w) and with two (replica rows read)."""
    for momentum, wd, dtype, H in ((0.9, 0.0, "f32", 1), (0.0, 0.0, "f32", 1), (0.9, 1e-3, "bf16", 1), (0.0, 0.0, "bf16", 1),
                                   (0.9, 0.0, "f32", 2)):
        cfg = small("round_k", K, [9001, 33, 1024], T=3, momentum=momentum, wd=wd, dtype=dtype)
        gu.run_both(cfg, cfg.T, fuse=2, batched=True, steps_per_round=H)
    for dtype in ("f32", "bf16"):
        cfg = small("round_k_sparse", K, [520, 90 * 64, 77], T=3, dtype=dtype, sparse=(1, 90, 64), scale=1e-3)
        gu.run_both(cfg, cfg.T, fuse=2, batched=True)


@pytest.mark.parametrize("P", [1, 31, 33, 129, 1000, 4097])
def test_round_kernel_odd_sizes(P):
    for K, momentum in ((2, 0.9), (7, 0.0), (16, 0.9)):
        cfg = small("round_odd", K, [P], T=3, momentum=momentum)
        gu.run_both(cfg, cfg.T, fuse=2, batched=True, check_each_round=True)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("batched", [True, False])
def test_round_kernel_sparse_rows(dtype, batched):
    cfg = small("round_sparse", 4, [1000, 300 * 64, 777, 64], T=5, dtype=dtype, sparse=(1, 300, 64), scale=1e-3)
    gu.run_both(cfg, cfg.T, fuse=2, batched=batched)
    cfg = small("round_sparse16", 16, [64, 200 * 128, 5], T=4, dtype=dtype, sparse=(1, 200, 128), scale=1e-3, wd=1e-4)
    gu.run_both(cfg, cfg.T, fuse=2, batched=batched, chunks=3)


def test_round_kernel_launches_one_kernel_per_round_and_writes_no_replica_row():
    cfg = small("round_count", 8, [50_000], T=4)
    with gu.session(cfg, fuse=2, lend_arena=True):
        stacked = np.stack([gu.host_inputs(cfg, i, 0)["padded"] for i in range(cfg.K)])
        g = gu.to_device(stacked.reshape(-1))
        rows = []
        for i in range(cfg.K):
            r, _ = hp.hpsgd_get_replica(i)               # before any merge the rows are real
            rows.append(r)
        assert len(set(rows)) == cfg.K and hp.hpsgd_get_global() not in rows
        poison = torch.full((cfg.layout.P_pad,), float("nan"), dtype=torch.float32, device=gu.DEV)
        hp.hpsgd_set_option(hp.HPSGD_OPT_PROFILE, 1)
        base = hp.hpsgd_launch_count()
        for t in range(4):
            hp.hpsgd_local_step_all(g, stacked.shape[1] * 4)
            assert hp.hpsgd_launch_count() - base == t          # held back
            hp.hpsgd_sync_merge()
            assert hp.hpsgd_launch_count() - base == t + 1      # one kernel: K local steps + the merge
            if t == 0:
                # from here on the rows are dead storage: whatever they hold must never be read
                hp.hpsgd_synchronize()
                for r in rows:
                    gu.dev_tensor(r, cfg.layout.P_pad).copy_(poison)
                torch.cuda.synchronize()
        hp.hpsgd_flush()
        assert hp.hpsgd_launch_count() - base == 4
        assert hp.hpsgd_profile_read(hp.HPSGD_KERNEL_ROUND)[1] == 4
        assert hp.hpsgd_profile_read(hp.HPSGD_KERNEL_LOCAL_STEP)[1] == 0
        assert hp.hpsgd_profile_read(hp.HPSGD_KERNEL_MERGE)[1] == 0
        w = hp.hpsgd_get_global()
        for i in range(cfg.K):
            assert hp.hpsgd_get_replica(i)[0] == w               # lazy clones: the replica is w itself
        for r in rows:
            assert bool(torch.isnan(gu.dev_tensor(r, cfg.layout.P_pad)).all()), "a replica row was written"
        assert bool(torch.isfinite(gu.dev_tensor(w, cfg.layout.P_pad)).all())


def test_the_four_core_calls_alone_reach_the_round_kernel():
    """hpsgd_init, hpsgd_local_step per worker, hpsgd_sync_merge, hpsgd_get_global with HPSGD_OPT_FUSE = 2:
    K per-worker calls and the merge that follows are one launch; a worker that steps twice, or a merge
    that finds only some workers stepped, falls back to separate launches.  Results as the oracle's."""
    cfg = small("four_calls", 8, [30_000, 77], T=6, momentum=0.9, wd=1e-4)
    o = gu.oracle_for(cfg)
    with gu.session(cfg, fuse=2):
        keep = []
        hp.hpsgd_set_option(hp.HPSGD_OPT_PROFILE, 1)
        for t in range(cfg.T):
            before = hp.hpsgd_launch_count()
            order = list(range(cfg.K)) if t % 2 == 0 else list(reversed(range(cfg.K)))   # any order of workers
            if t == 3:
                order.remove(5)                          # worker 5 sits this round out
            for i in order:
                inp = gu.host_inputs(cfg, i, t)
                gu.gpu_step(cfg, i, inp, keep)
                o.local_step(i, inp["flat"])
            if t == 4:                                   # worker 2 steps a second time before the merge
                inp = gu.host_inputs(cfg, 2, 100 + t)
                gu.gpu_step(cfg, 2, inp, keep)
                o.local_step(2, inp["flat"])
            hp.hpsgd_sync_merge()
            o.sync_merge()
            launched = hp.hpsgd_launch_count() - before
            if t == 3:
                assert launched == 3                     # workers 0-4, workers 6-7, the merge
            elif t == 4:
                assert launched == 3                     # all eight, worker 2 again, the merge
            else:
                assert launched == 1
        assert hp.hpsgd_profile_read(hp.HPSGD_KERNEL_ROUND)[1] == cfg.T - 2
        w, D, rs, ms = gu.gpu_state(cfg)
        gu.assert_bitwise(w, o.get_global(), "global model")
        gu.assert_bitwise(D, o.get_pending(), "pending change")
        for i in range(cfg.K):
            gu.assert_bitwise(rs[i], o.get_replica(i), "replica %d" % i)
            gu.assert_bitwise(ms[i], o.get_momentum(i), "momentum %d" % i)
    o.close()


def test_lazy_clones_under_every_other_call():
    """Interleave whole-round kernels with per-worker steps, idle workers, merges on their own,
    inspection and a change of schedule: replicas that exist only as 'w' must behave like rows."""
    cfg = small("round_mixed", 8, [40_000, 17], T=10, momentum=0.9, wd=1e-4)
    o = gu.oracle_for(cfg)
    with gu.session(cfg, fuse=2, chunks=2):
        keep = []
        for t in range(cfg.T):
            inputs = [gu.host_inputs(cfg, i, t) for i in range(cfg.K)]
            if t in (4, 7):                              # per-worker calls; in round 7 worker 3 sits out
                for i, inp in enumerate(inputs):
                    if t == 7 and i == 3:
                        continue
                    gu.gpu_step(cfg, i, inp, keep)
                    o.local_step(i, inp["flat"])
            else:
                stacked = np.stack([inp["padded"] for inp in inputs])
                keep.append(gu.to_device(stacked.reshape(-1)))
                hp.hpsgd_local_step_all(keep[-1], stacked.shape[1] * 4)
                for i, inp in enumerate(inputs):
                    o.local_step(i, inp["flat"])
            if t == 2:                                   # look at the replicas between step and merge
                w, D, rs, ms = gu.gpu_state(cfg)
                for i in range(cfg.K):
                    gu.assert_bitwise(rs[i], o.get_replica(i), "replica %d after a flushed step" % i)
            if t == 5:
                hp.hpsgd_set_option(hp.HPSGD_OPT_FUSE, 1)    # rows are written out, the other fused schedule takes over
            if t == 8:
                hp.hpsgd_set_option(hp.HPSGD_OPT_FUSE, 2)
            hp.hpsgd_sync_merge()
            o.sync_merge()
            if t == 3:
                hp.hpsgd_sync_merge()                    # a merge with no step before it
                o.sync_merge()
        w, D, rs, ms = gu.gpu_state(cfg)
        gu.assert_bitwise(w, o.get_global(), "global model")
        gu.assert_bitwise(D, o.get_pending(), "pending change")
        for i in range(cfg.K):
            gu.assert_bitwise(rs[i], o.get_replica(i), "replica %d" % i)
            gu.assert_bitwise(ms[i], o.get_momentum(i), "momentum %d" % i)


def test_fill_global_reseeds_like_a_fresh_init():
    """hpsgd_fill_global(seed): w from hash stream 2 of that seed, everything else as after hpsgd_init."""
    cfg = small("fill", 4, [5000, 77, 33], T=2, momentum=0.9)
    other = small("fill", 4, [5000, 77, 33], T=2, momentum=0.9, seed=cfg.seed + 1000)
    with gu.session(other):
        fresh = gu.gpu_state(other)
    for fuse in (0, 2):
        with gu.session(cfg, fuse=fuse):
            keep = []
            for t in range(2):                               # leave every buffer dirty
                for i in range(cfg.K):
                    gu.gpu_step(cfg, i, gu.host_inputs(cfg, i, t), keep)
                hp.hpsgd_sync_merge()
            hp.hpsgd_fill_global(other.seed)
            assert hp.hpsgd_get_sizes()[3] == 0
            w, D, rs, ms = gu.gpu_state(cfg)
            gu.assert_bitwise(w, other.initial_global(), "re-seeded global model vs the host generator")
            gu.assert_bitwise(w, fresh[0], "re-seeded global model vs a fresh hpsgd_init")
            assert not D.any()
            for i in range(cfg.K):
                gu.assert_bitwise(rs[i], w, "replica %d after the re-seed" % i)
                assert not ms[i].any()
            # and the run that follows is the run of a fresh state with that seed
            o = gu.oracle_for(other)
            for t in range(3):
                for i in range(cfg.K):
                    inp = gu.host_inputs(other, i, t)
                    gu.gpu_step(other, i, inp, keep)
                    o.local_step(i, inp["flat"])
                hp.hpsgd_sync_merge()
                o.sync_merge()
            gu.assert_bitwise(gu.gpu_state(cfg)[0], o.get_global(), "global model of the run after the re-seed")
            # the device generator follows the new seed too
            out = torch.empty(cfg.layout.P_pad, dtype=torch.float32, device=gu.DEV)
            hp.hpsgd_gen_grads(out, 1, 3, hp.HPSGD_GEN_UNIFORM, 1e-2)
            hp.hpsgd_synchronize()
            import workloads.hashgen as hg
            gu.assert_bitwise(cfg.layout.unpack(out.cpu().numpy()),
                              hg.grad_uniform(other.seed, 3, 1, scale=1e-2, idx0=0, n=cfg.P), "gradients of the new seed")
            o.close()


@pytest.mark.parametrize("mode", ["two_streams", "one_stream", "fuse", "round", "pipeline"])
def test_async_host_copy_sees_the_model_of_its_merge(mode):
    """hpsgd_copy_global_async after merge t must deliver w as of merge t, although later local
    steps and merges are enqueued before anything is waited for."""
    cfg = small("d2h", 4, [60_000, 99], T=5, momentum=0.9)
    kw = dict(overlap=0 if mode == "one_stream" else 1, fuse={"fuse": 1, "round": 2}.get(mode, 0),
              pipeline=int(mode == "pipeline"))
    o = gu.oracle_for(cfg)
    outs = [torch.empty(cfg.P, dtype=torch.float32).pin_memory() for _ in range(cfg.T)]
    want = []
    with gu.session(cfg, **kw):
        keep = []
        for t in range(cfg.T):
            inputs = [gu.host_inputs(cfg, i, t) for i in range(cfg.K)]
            stacked = np.stack([inp["padded"] for inp in inputs])
            keep.append(gu.to_device(stacked.reshape(-1)))
            hp.hpsgd_local_step_all(keep[-1], stacked.shape[1] * 4)
            for i, inp in enumerate(inputs):
                o.local_step(i, inp["flat"])
            hp.hpsgd_sync_merge()
            o.sync_merge()
            hp.hpsgd_copy_global_async(outs[t])
            want.append(o.get_global())
        hp.hpsgd_synchronize()
        for t in range(cfg.T):
            gu.assert_bitwise(outs[t].numpy(), want[t], "host copy taken after merge %d" % t)


def test_async_host_copy_after_a_fused_kernel():
    """The fused merge + step kernel writes w on the main stream; a host copy requested right
    after it (before the next merge) must wait for it."""
    cfg = small("d2h_fused", 8, [400_000], T=4, momentum=0.9)
    o = gu.oracle_for(cfg)
    outs = [torch.empty(cfg.P, dtype=torch.float32).pin_memory() for _ in range(cfg.T)]
    want = []
    with gu.session(cfg, fuse=1):
        keep = []
        for t in range(cfg.T):
            inputs = [gu.host_inputs(cfg, i, t) for i in range(cfg.K)]
            stacked = np.stack([inp["padded"] for inp in inputs])
            keep.append(gu.to_device(stacked.reshape(-1)))
            hp.hpsgd_local_step_all(keep[-1], stacked.shape[1] * 4)     # carries merge t-1 from round 1 on
            for i, inp in enumerate(inputs):
                o.local_step(i, inp["flat"])
            hp.hpsgd_copy_global_async(outs[t])                          # w as of merge t-1
            want.append(o.get_global())
            hp.hpsgd_sync_merge()
            o.sync_merge()
        hp.hpsgd_synchronize()
        for t in range(cfg.T):
            gu.assert_bitwise(outs[t].numpy(), want[t], "host copy taken after the step of round %d" % t)
