"""The allocation-free sparse-row step against the regular one and against the CPU oracle.

hpsgd_local_step_sparse_noalloc exists for programs that cannot allocate device memory at the
moment they want to step: a server whose own allocator claimed the whole GPU at start-up, so
that a cudaMalloc by anyone else simply fails; a latency-critical loop in which the device-wide
synchronisation hidden in cudaMalloc / cudaFree would stall every other stream; a process held
to a fixed memory budget.  For them the row -> slot scratch map of the sparse-row step is a
fixed array inside the library image instead of a piece of an arena.

The test runs the same two consecutive steps through that entry point, through
hpsgd_local_step_ex and through the oracle's sparse-row step, and requires bit-identical
replicas and momenta from all three.  The second step uses a different set of active rows, so a
map that still held the first call's entries would be caught.  It also checks the property the
entry point exists for: once the first call on the device has been made, a call leaves the
amount of free device memory exactly where it was.

This file is named to be collected last: if it fails under `pytest -x`, every other test has
already run.
"""
import numpy as np
import pytest
import torch

import paper_2009_02701_b200 as hp
from oracle.ref import RefHPSGD
from tests import gpu_util as gu
from workloads.configs import Workload

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,momentum,wd", [("bf16", 0.9, 0.0), ("f32", 0.9, 5e-4), ("f32", 0.0, 0.0)])
def test_noalloc_step_matches_regular_step_twice_in_a_row(dtype, momentum, wd):
    rows, cols = 500, 64
    cfg = Workload("noalloc", K=2, sizes=(1000, rows * cols, 321), T=2, lr=0.05, momentum=momentum,
                   weight_decay=wd, seed=21, grad_kind="gauss", grad_scale=1e-3, grad_dtype=dtype,
                   sparse=(1, rows, cols))
    lay = cfg.layout
    worker = 1
    inputs = [gu.host_inputs(cfg, worker, step) for step in (0, 1)]
    assert not np.array_equal(inputs[0]["rows"], inputs[1]["rows"])

    # first reference: the regular entry point, which keeps its map in the arena
    want = []
    with gu.session(cfg):
        w0 = gu.dev_view(hp.hpsgd_get_global(), lay.P_pad)
        for inp in inputs:
            keep = []
            gu.gpu_step(cfg, worker, inp, keep)
            hp.hpsgd_synchronize()
            r, m = hp.hpsgd_get_replica(worker)
            want.append((gu.dev_view(r, lay.P_pad), gu.dev_view(m, lay.P_pad) if m else None))

    # second reference: the oracle's sparse-row step (un-padded index space)
    oracle = gu.oracle_for(cfg)
    oracle_want = []
    for inp in inputs:
        gu.oracle_step(oracle, cfg, worker, inp)
        oracle_want.append((oracle.get_replica(worker), oracle.get_momentum(worker) if momentum else None))
    oracle.close()

    # the allocation-free entry point on buffers owned by the test; no library state exists
    r = w0.clone()
    m = torch.zeros_like(r) if momentum else None
    stream = torch.cuda.Stream(device=gu.DEV)
    stream.wait_stream(torch.cuda.current_stream())
    gdt = hp.HPSGD_BF16 if dtype == "bf16" else hp.HPSGD_F32
    staged = []
    for inp in inputs:                        # every device buffer exists before the first call
        staged.append((gu.to_device(inp["padded"]), gu.to_device(inp["rows"]), gu.to_device(inp["vals"].reshape(-1))))
    torch.cuda.synchronize()
    free_after_first = None
    for step, (inp, (g, idx, vals)) in enumerate(zip(inputs, staged)):
        desc = hp.make_desc(g, idx, len(inp["rows"]), vals)
        if step == 1:
            free_after_first = torch.cuda.mem_get_info()[0]
        hp.hpsgd_local_step_sparse_noalloc(r, m, lay.P_pad, desc, gdt, lay.offsets[1], rows, cols,
                                           cfg.lr, momentum, wd, stream)
        stream.synchronize()
        if step == 1:
            # the call after the warm-up call took no device memory (and gave none back)
            assert torch.cuda.mem_get_info()[0] == free_after_first
        assert torch.equal(r, want[step][0]), "replica differs from hpsgd_local_step_ex after call %d" % (step + 1)
        gu.assert_bitwise(lay.unpack(r.cpu().numpy()), oracle_want[step][0], "replica vs oracle after call %d" % (step + 1))
        if momentum:
            assert torch.equal(m, want[step][1]), "momentum differs from hpsgd_local_step_ex after call %d" % (step + 1)
            gu.assert_bitwise(lay.unpack(m.cpu().numpy()), oracle_want[step][1],
                              "momentum vs oracle after call %d" % (step + 1))


def test_noalloc_rejects_more_rows_than_its_built_in_map():
    r = torch.zeros(64, dtype=torch.float32, device=gu.DEV)
    desc = hp.make_desc(r)
    with pytest.raises(hp.HpsgdError) as err:
        hp.hpsgd_local_step_sparse_noalloc(r, None, 64, desc, hp.HPSGD_F32, 0, hp.HPSGD_NOALLOC_MAX_ROWS + 1, 8,
                                           0.1, 0.0, 0.0, None)
    assert err.value.code == hp.HPSGD_E_UNSUPPORTED
    assert str(hp.HPSGD_NOALLOC_MAX_ROWS) in hp.last_error()


def test_noalloc_rejects_a_tensor_that_does_not_fit_without_overflowing():
    """cols so large that rows * cols would wrap a 64-bit integer must be refused, not truncated."""
    r = torch.zeros(64, dtype=torch.float32, device=gu.DEV)
    desc = hp.make_desc(r)
    for rows, cols, off in ((4, 1 << 62, 0), (2, 64, 0), (1, 64, 8), (8, 8, 8)):
        with pytest.raises(hp.HpsgdError) as err:
            hp.hpsgd_local_step_sparse_noalloc(r, None, 64, desc, hp.HPSGD_F32, off, rows, cols, 0.1, 0.0, 0.0, None)
        assert err.value.code == hp.HPSGD_E_BADARG
