"""The checked build of the library (-DHPSGD_DEBUG): same results, plus what it exists for.

In that build every hot kernel tests the group index it is about to touch (and every row -> slot
entry it is about to follow) before the access, records a violation and skips it, and the entry
points that take a sparse row list copy the list to the host and refuse a bad one.  Nothing here
makes the GPU fault: the kernel guard is shown to work by lowering the limit it tests against
below the real size, so that the "violations" are accesses that are in fact in bounds.
"""
import numpy as np
import pytest
import torch

import paper_2009_02701_b200 as hp
from paper_2009_02701_b200 import build
from tests import gpu_util as gu
from workloads.configs import Workload

pytestmark = pytest.mark.gpu


@pytest.fixture()
def checked_library():
    path = build.build(debug=True)
    hp.hpsgd_destroy()
    hp.use_library(path)
    try:
        yield path
    finally:
        hp.hpsgd_destroy()
        hp.use_library(None)


def small(name, K, sizes, T=3, momentum=0.9, wd=0.0, dtype="f32", sparse=None, scale=1e-2):
    return Workload(name, K=K, sizes=tuple(sizes), T=T, lr=0.1, momentum=momentum, weight_decay=wd, seed=9,
                    grad_kind="gauss", grad_scale=scale, grad_dtype=dtype, sparse=sparse)


def test_checked_build_gives_the_same_results(checked_library):
    for P in (1, 33, 129, 4097):
        for K, momentum in ((3, 0.9), (16, 0.9), (5, 0.0)):
            cfg = small("chk_odd", K, [P], momentum=momentum)
            gu.run_both(cfg, cfg.T, check_each_round=True)
            gu.run_both(cfg, cfg.T, fuse=2, batched=True)
    cfg = small("chk_multi", 8, [70_001, 33, 4096], T=4, wd=5e-4)
    for kw in (dict(), dict(fuse=1, batched=True, chunks=3), dict(fuse=2, batched=True, chunks=2),
               dict(pipeline=1, batched=True), dict(batched=True, chunks=5, overlap=0),
               dict(chunks=2, session_kw=dict(staging=1))):
        gu.run_both(cfg, cfg.T, **kw)
    for dtype in ("f32", "bf16"):
        cfg = small("chk_sparse", 5, [1000, 300 * 64, 777, 64], T=4, dtype=dtype, sparse=(1, 300, 64), scale=1e-3)
        for kw in (dict(), dict(batched=True, chunks=3), dict(fuse=1, batched=True), dict(fuse=2, batched=True),
                   dict(pipeline=1, batched=True)):
            gu.run_both(cfg, cfg.T, **kw)
    cfg = small("chk_accum", 4, [5000, 77], momentum=0.0)
    gu.run_both_accum(cfg, cfg.T, batched=True, chunks=2)


def test_checked_build_refuses_bad_row_lists_before_launching(checked_library):
    rows, cols = 40, 16
    cfg = small("chk_rows", 2, [64, rows * cols, 32], sparse=(1, rows, cols))
    lay = cfg.layout
    g = torch.zeros(lay.P_pad, dtype=torch.float32, device=gu.DEV)
    vals = torch.zeros(4 * cols, dtype=torch.float32, device=gu.DEV)
    good = torch.tensor([1, 5, 9, 30], dtype=torch.int32, device=gu.DEV)
    bad = {"not ascending": [5, 1, 9, 30], "listed twice": [1, 5, 5, 30], "outside": [1, 5, 9, rows],
           "outside ": [-1, 5, 9, 30]}
    with gu.session(cfg):
        hp.hpsgd_synchronize()
        before = hp.hpsgd_launch_count()
        for what, lst in bad.items():
            idx = torch.tensor(lst, dtype=torch.int32, device=gu.DEV)
            torch.cuda.synchronize()
            for call in (lambda: hp.hpsgd_local_step_ex(0, hp.make_desc(g, idx, 4, vals)),
                         lambda: hp.hpsgd_local_step_all_ex([hp.make_desc(g, good, 4, vals), hp.make_desc(g, idx, 4, vals)])):
                with pytest.raises(hp.HpsgdError) as err:
                    call()
                assert err.value.code == hp.HPSGD_E_BADARG
                assert what.strip() in hp.last_error()
        assert hp.hpsgd_launch_count() == before, "a refused call launched something"
        hp.hpsgd_local_step_ex(0, hp.make_desc(g, good, 4, vals))        # and a good list still goes through
        hp.hpsgd_synchronize()
    # the entry point that allocates nothing checks its list the same way
    r = torch.zeros(lay.P_pad, dtype=torch.float32, device=gu.DEV)
    keep = r.clone()
    for what, lst in bad.items():
        idx = torch.tensor(lst, dtype=torch.int32, device=gu.DEV)
        torch.cuda.synchronize()
        with pytest.raises(hp.HpsgdError) as err:
            hp.hpsgd_local_step_sparse_noalloc(r, None, lay.P_pad, hp.make_desc(g, idx, 4, vals), hp.HPSGD_F32,
                                               lay.offsets[1], rows, cols, 0.1, 0.0, 0.0, None)
        assert err.value.code == hp.HPSGD_E_BADARG
    torch.cuda.synchronize()
    assert torch.equal(r, keep)


@pytest.mark.parametrize("fuse,batched,staging", [(0, False, 0), (0, True, 0), (1, True, 0), (2, True, 0), (0, True, 1)])
def test_kernel_guard_records_and_skips(checked_library, fuse, batched, staging):
    """With the limit lowered to half the buffer the kernels skip the upper half (in-bounds memory
    that the guard now calls out of range), the next synchronisation reports it, and the state
    stays usable."""
    cfg = small("chk_guard", 4, [8192 * 8], T=1, momentum=0.9)
    groups = cfg.layout.P_pad // 8
    half = groups // 2
    with gu.session(cfg, fuse=fuse, staging=staging):
        inputs = [gu.host_inputs(cfg, i, 0) for i in range(cfg.K)]
        stacked = np.stack([inp["padded"] for inp in inputs])
        dev_g = gu.to_device(stacked.reshape(-1))
        w_before = gu.dev_view(hp.hpsgd_get_global(), cfg.layout.P_pad)
        m_before = gu.dev_view(hp.hpsgd_get_replica(0)[1], cfg.layout.P_pad)
        hp.hpsgd_set_option(hp.HPSGD_OPT_DEBUG_GROUP_LIMIT, half)

        def one_round():
            if batched:
                hp.hpsgd_local_step_all(dev_g, stacked.shape[1] * 4)
            else:
                for i in range(cfg.K):
                    hp.hpsgd_local_step(i, dev_g[i * stacked.shape[1]:])
            hp.hpsgd_sync_merge()

        one_round()
        with pytest.raises(hp.HpsgdError) as err:
            hp.hpsgd_synchronize()
        assert err.value.code == hp.HPSGD_E_CUDA
        text = hp.last_error()
        assert "checked build" in text and "group index" in text and "[0, %d)" % half in text
        hp.hpsgd_synchronize()                                   # reported once, then the record is clear
        m_after = gu.dev_view(hp.hpsgd_get_replica(0)[1], cfg.layout.P_pad)
        assert torch.equal(m_after[half * 8:], m_before[half * 8:]), "a group beyond the limit was touched"
        assert not torch.equal(m_after[:half * 8], m_before[:half * 8])
        w_after = gu.dev_view(hp.hpsgd_get_global(), cfg.layout.P_pad)
        assert torch.equal(w_after, w_before)                    # the first merge commits nothing anyway
        # back to the real limit: everything runs, nothing is reported
        hp.hpsgd_set_option(hp.HPSGD_OPT_DEBUG_GROUP_LIMIT, -1)
        one_round()
        hp.hpsgd_synchronize()
        assert bool(torch.isfinite(gu.dev_view(hp.hpsgd_get_global(), cfg.layout.P_pad)).all())


def test_staged_merge_wait_that_runs_out_is_reported(checked_library):
    """The one device-side wait of the library (the staged merge waiting for its own bulk loads) is bounded:
    with its barrier told to expect bytes that never arrive, every block gives up after a second, writes
    nothing, and the next synchronisation returns HPSGD_E_TIMEOUT; the context stays usable."""
    import time
    cfg = small("chk_stall", 3, [2000, 40], T=1)           # three tiles, three blocks
    with gu.session(cfg, staging=1):
        keep = []
        for i in range(cfg.K):
            gu.gpu_step(cfg, i, gu.host_inputs(cfg, i, 0), keep)
        hp.hpsgd_synchronize()
        n = cfg.layout.P_pad
        w_before = gu.dev_view(hp.hpsgd_get_global(), n)
        rows = [hp.hpsgd_get_replica(i)[0] for i in range(cfg.K)]
        r_before = [gu.dev_view(r, n) for r in rows]
        hp.hpsgd_set_option(hp.HPSGD_OPT_DEBUG_STAGE_STALL, 1)
        hp.hpsgd_sync_merge()
        t0 = time.perf_counter()
        with pytest.raises(hp.HpsgdError) as err:
            hp.hpsgd_synchronize()
        waited = time.perf_counter() - t0
        assert err.value.code == hp.HPSGD_E_TIMEOUT and "gave up waiting" in hp.last_error()
        assert 1.0 < waited < 30.0
        hp.hpsgd_set_option(hp.HPSGD_OPT_DEBUG_STAGE_STALL, 0)
        hp.hpsgd_synchronize()                               # reported once
        assert torch.equal(gu.dev_view(hp.hpsgd_get_global(), n), w_before), "a block that gave up wrote w"
        for r, before in zip(rows, r_before):
            assert torch.equal(gu.dev_view(r, n), before), "a block that gave up wrote a replica"
    # and the library carries on: the same kernel, unstalled, against the oracle
    gu.run_both(small("chk_after_stall", 3, [2000, 40], T=2), 2, session_kw=dict(staging=1))


def test_normal_build_has_no_guard_option():
    cfg = small("chk_none", 2, [1000])
    with gu.session(cfg):
        with pytest.raises(hp.HpsgdError) as err:
            hp.hpsgd_set_option(hp.HPSGD_OPT_DEBUG_GROUP_LIMIT, 10)
        assert err.value.code == hp.HPSGD_E_UNSUPPORTED
        with pytest.raises(hp.HpsgdError) as err:
            hp.hpsgd_set_option(hp.HPSGD_OPT_DEBUG_STAGE_STALL, 1)
        assert err.value.code == hp.HPSGD_E_UNSUPPORTED
