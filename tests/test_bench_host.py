"""Host logic of bench.py for N > 1: independent replicas, time = max over ranks, units = sum.
Run as two gloo ranks on CPU."""
import json
import os
import subprocess
import sys

import pytest
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world), LOCAL_RANK=str(rank), HPSGD_BENCH_BACKEND="gloo")
    sys.path.insert(0, ROOT)
    import bench
    r, w, local, dist = bench.dist_setup(world)
    assert (r, w, local) == (rank, world, rank) and dist is not None
    dist.barrier()
    ms, units = bench.aggregate(dist, torch.device("cpu"), 10.0 + 5.0 * rank, 1000 * (rank + 1))
    out[rank] = (ms, units)
    dist.barrier()
    dist.destroy_process_group()


def test_aggregate_takes_max_time_and_sums_units():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank_main, args=(world, 29517, out), nprocs=world, join=True)
        assert out[0] == out[1] == (15.0, 3000.0)


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    env = {k: os.environ.pop(k) for k in ("WORLD_SIZE", "RANK") if k in os.environ}
    try:
        assert bench.dist_setup(1) == (0, 1, 0, None)
        assert bench.aggregate(None, None, 7.0, 42) == (7.0, 42)
    finally:
        os.environ.update(env)


def test_reference_arm_prints_one_line_on_rank0_only():
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0",
           "--workload", "cfg1", "--ref-sample", "200000"]
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    other = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=300)
    assert other.returncode == 0 and other.stdout.strip() == ""
    env = dict(os.environ, RANK="0", WORLD_SIZE="2")
    first = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=300)
    assert first.returncode == 0
    line = json.loads(first.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["unit"] == "K*P elems/s"
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] == 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["vs_baseline"] is None


def test_roofline_byte_counts():
    sys.path.insert(0, ROOT)
    import bench
    import workloads
    assert bench.merge_bytes_per_index(workloads.get("cfg1")) == 48
    assert bench.merge_bytes_per_index(workloads.get("cfg2")) == 80
    assert bench.merge_bytes_per_index(workloads.get("cfg4")) == 144
    assert bench.local_bytes_per_elem(workloads.get("cfg1")) == 12
    assert bench.local_bytes_per_elem(workloads.get("cfg4")) == 20
    assert bench.local_bytes_per_elem(workloads.get("cfg5")) == 18


def test_oracle_on_all_cores_and_do_nothing_interpolation():
    sys.path.insert(0, ROOT)
    import bench
    import workloads
    out = bench.oracle_all_cores(workloads.get("cfg1"), per_core_params=20_000, rounds=2)
    assert out["cores"] == os.cpu_count() and out["value"] > 0 and out["unit"] == "K*P elems/s"
    rates = {"rates": [{"write_share": 0.0, "GB/s": 7500.0}, {"write_share": 0.5, "GB/s": 6800.0},
                       {"write_share": 1.0, "GB/s": 7300.0}]}
    got = bench.against_do_nothing(rates, 0.25, 3575.0)
    assert got["do_nothing_GB/s"] == pytest.approx(7150.0) and got["kernel_over_do_nothing"] == pytest.approx(0.5)
