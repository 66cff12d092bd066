"""The merge with its tiles staged through shared memory by bulk-async copies (HPSGD_OPT_STAGING)
against the CPU oracle, bit for bit, and the HBM bandwidth probe's contract."""
import numpy as np
import pytest
import torch

import paper_2009_02701_b200 as hp
from tests import gpu_util as gu
from workloads.configs import Workload

pytestmark = pytest.mark.gpu


def small(name, K, sizes, T=4, momentum=0.9, wd=0.0, staleness=1):
    return Workload(name, K=K, sizes=tuple(sizes), T=T, lr=0.1, momentum=momentum, weight_decay=wd, seed=21,
                    grad_kind="gauss", grad_scale=1e-2, staleness=staleness)


def staged_launches():
    return hp.hpsgd_profile_read(hp.HPSGD_KERNEL_MERGE_STAGED)[1], hp.hpsgd_profile_read(hp.HPSGD_KERNEL_MERGE)[1]


@pytest.mark.parametrize("K,momentum,wd,staleness,overlap,chunks,fuse", [
    (16, 0.9, 0.0, 1, 1, 1, 0), (8, 0.9, 5e-4, 1, 1, 3, 0), (4, 0.0, 0.0, 1, 0, 1, 0), (4, 0.5, 1e-3, 0, 1, 2, 0),
    (1, 0.9, 0.0, 1, 1, 1, 0), (3, 0.0, 0.0, 0, 0, 5, 0), (9, 0.9, 0.0, 1, 1, 1, 1), (32, 0.9, 0.0, 1, 1, 2, 0)])
def test_staged_merge_matches_oracle(K, momentum, wd, staleness, overlap, chunks, fuse):
    """Several tiles, a ragged last tile and several tensors, every round compared."""
    cfg = small("staged", K, [70_001, 1234, 8 * 1024 * 3, 33], T=4, momentum=momentum, wd=wd, staleness=staleness)
    gu.run_both(cfg, cfg.T, staleness=staleness, overlap=overlap, chunks=chunks, fuse=fuse, batched=bool(fuse),
                check_each_round=not fuse, session_kw=dict(staging=1, lend_arena=True, canary=True))


@pytest.mark.parametrize("P", [1, 8, 31, 33, 1000, 1023, 1024, 1025, 2048, 4097])
def test_staged_merge_odd_sizes(P):
    """One group, exactly one tile, one element more than a tile, ..."""
    cfg = small("staged_odd", 5, [P], T=3)
    gu.run_both(cfg, cfg.T, check_each_round=True, session_kw=dict(staging=1, lend_arena=True, canary=True))


def test_staged_merge_is_the_kernel_that_ran_and_gives_way_where_it_does_not_apply():
    cfg = small("staged_ran", 8, [50_000], T=3)
    for fuse, want_staged in ((0, True), (2, False)):       # lazy clones (fuse 2) have their own merge kernel
        with gu.session(cfg, fuse=fuse, staging=1):
            hp.hpsgd_set_option(hp.HPSGD_OPT_PROFILE, 1)
            keep = []
            for t in range(cfg.T):
                gu.gpu_step(cfg, 0, gu.host_inputs(cfg, 0, t), keep)     # one worker only: no whole-round kernel
                hp.hpsgd_sync_merge()
            hp.hpsgd_synchronize()
            staged, plain = staged_launches()
            assert (staged, plain) == ((cfg.T, 0) if want_staged else (0, cfg.T))
    # more workers than the staged kernel takes: the plain merge runs, same results
    cfg = small("staged_k33", 33, [3000], T=2)
    gu.run_both(cfg, cfg.T, session_kw=dict(staging=1))
    with gu.session(cfg):
        with pytest.raises(hp.HpsgdError) as err:
            hp.hpsgd_set_option(hp.HPSGD_OPT_STAGING, 2)
        assert err.value.code == hp.HPSGD_E_BADARG


def test_staging_can_be_switched_between_rounds():
    cfg = small("staged_switch", 4, [9000, 77], T=6)
    o = gu.oracle_for(cfg)
    with gu.session(cfg):
        keep = []
        for t in range(cfg.T):
            hp.hpsgd_set_option(hp.HPSGD_OPT_STAGING, t % 2)
            for i in range(cfg.K):
                inp = gu.host_inputs(cfg, i, t)
                gu.gpu_step(cfg, i, inp, keep)
                gu.oracle_step(o, cfg, i, inp)
            hp.hpsgd_sync_merge()
            o.sync_merge()
        w, D, rs, ms = gu.gpu_state(cfg)
        gu.assert_bitwise(w, o.get_global(), "global model")
        gu.assert_bitwise(D, o.get_pending(), "pending change")
        for i in range(cfg.K):
            gu.assert_bitwise(rs[i], o.get_replica(i), "replica %d" % i)
    o.close()


def test_bandwidth_probe_contract():
    row = 8 << 20
    buf = torch.empty(24 * row, dtype=torch.uint8, device=gu.DEV)
    torch.cuda.synchronize()
    for n_read, n_write in ((16, 0), (12, 4), (16, 4), (13, 7), (12, 8), (8, 8), (4, 16), (0, 16)):
        rate = hp.hpsgd_probe_hbm(buf, buf.numel(), n_read, n_write, row, 3)
        assert np.isfinite(rate) and rate > 0
    # the rows were zero-filled and only sums of zeros were written
    assert not bool(buf[: 20 * row].any())
    for args, code in (((buf, buf.numel(), 5, 5, row, 3), hp.HPSGD_E_UNSUPPORTED),
                       ((buf, buf.numel(), 16, 4, row + 32, 3), hp.HPSGD_E_BADARG),
                       ((buf, 19 * row, 16, 4, row, 3), hp.HPSGD_E_NOMEM),
                       ((buf.data_ptr() + 256, buf.numel() - 256, 8, 8, row, 3), hp.HPSGD_E_BADARG),
                       ((buf, buf.numel(), 8, 8, row, 0), hp.HPSGD_E_BADARG),
                       ((None, 0, 8, 8, row, 3), hp.HPSGD_E_BADARG)):
        with pytest.raises(hp.HpsgdError) as err:
            hp.hpsgd_probe_hbm(*args)
        assert err.value.code == code
