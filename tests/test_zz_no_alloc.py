"""The allocation-free sparse-row step against the regular one.

hpsgd_local_step_sparse_noalloc exists for programs that cannot allocate device memory at the
moment they want to step: a server whose own allocator claimed the whole GPU at start-up, so
that a cudaMalloc by anyone else simply fails; a latency-critical loop in which the device-wide
synchronisation hidden in cudaMalloc / cudaFree would stall every other stream; a process held
to a fixed memory budget.  For them the row -> slot scratch map of the sparse-row step is a
fixed array inside the library image instead of a piece of an arena.

The test runs the same two consecutive steps through that entry point and through
hpsgd_local_step_ex and requires bit-identical replicas and momenta.  The second step uses a
different set of active rows, so a map that still held the first call's entries would be caught.

This file is named to be collected last: if it fails under `pytest -x`, every other test has
already run.
"""
import numpy as np
import pytest
import torch

import paper_2009_02701_b200 as hp
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

    # reference: the regular entry point, which keeps its map in the arena
    want = []
    with gu.session(cfg):
        w0 = gu.dev_view(hp.hpsgd_get_global(), lay.P_pad)
        for inp in inputs:
            keep = []
            gu.gpu_step(cfg, worker, inp, keep)
            hp.hpsgd_synchronize()
            r, m = hp.hpsgd_get_replica(worker)
            want.append((gu.dev_view(r, lay.P_pad), gu.dev_view(m, lay.P_pad) if m else None))

    # the allocation-free entry point on buffers owned by the test; no library state exists
    r = w0.clone()
    m = torch.zeros_like(r) if momentum else None
    stream = torch.cuda.Stream(device=gu.DEV)
    stream.wait_stream(torch.cuda.current_stream())
    gdt = hp.HPSGD_BF16 if dtype == "bf16" else hp.HPSGD_F32
    for step, inp in enumerate(inputs):
        g = gu.to_device(inp["padded"])
        idx = gu.to_device(inp["rows"])
        vals = gu.to_device(inp["vals"].reshape(-1))
        torch.cuda.synchronize()
        desc = hp.make_desc(g, idx, len(inp["rows"]), vals)
        hp.hpsgd_local_step_sparse_noalloc(r, m, lay.P_pad, desc, gdt, lay.offsets[1], rows, cols,
                                           cfg.lr, momentum, wd, stream)
        stream.synchronize()
        assert torch.equal(r, want[step][0]), "replica differs after call %d" % (step + 1)
        if momentum:
            assert torch.equal(m, want[step][1]), "momentum differs after call %d" % (step + 1)


def test_noalloc_rejects_more_rows_than_its_built_in_map():
    r = torch.zeros(64, dtype=torch.float32, device=gu.DEV)
    desc = hp.make_desc(r)
    with pytest.raises(hp.HpsgdError) as err:
        hp.hpsgd_local_step_sparse_noalloc(r, None, 64, desc, hp.HPSGD_F32, 0, hp.HPSGD_NOALLOC_MAX_ROWS + 1, 8,
                                           0.1, 0.0, 0.0, None)
    assert err.value.code == hp.HPSGD_E_UNSUPPORTED
    assert str(hp.HPSGD_NOALLOC_MAX_ROWS) in hp.last_error()
