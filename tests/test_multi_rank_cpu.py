"""The N > 1 plumbing of the benchmark on CPU: two gloo ranks, each with its own instances, no
data-path collective; the job time is the MAX over ranks and the value counts every rank's work."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        my_ms = 10.0 + 5.0 * rank  # rank 1 is the slow one
        ms = bench.max_over_ranks(torch, dist, my_ms, "cpu")
        value = bench.shard_report(world, 7, 2.0e9, 3, ms)
        dist.barrier()
        out[rank] = (ms, value)
    finally:
        dist.destroy_process_group()


def test_two_ranks_max_time_and_aggregate_value():
    world = 2
    port = 29500 + (os.getpid() % 2000)
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for ms, value in res.values():
        assert ms == 15.0  # both ranks agree on the slowest rank's time
        assert value == pytest.approx(2 * 7 * 2.0e9 * 3 / 15.0e-3 / 1e12)


def test_single_rank_helpers():
    sys.path.insert(0, ROOT)
    import bench

    assert bench.max_over_ranks(torch, None, 3.5, "cpu") == 3.5
    assert bench.shard_report(1, 10, 1e12, 2, 1000.0) == pytest.approx(20.0)
    peaks = {"hbm_gbs": 6551.0, "bf16_tflops": 1645.6}
    from paper_2104_04731_b200.synth import CONFIGS

    bounds = [bench.roofline_time_us(c, peaks)[1] for c in CONFIGS]
    assert bounds == ["hbm", "hbm", "hbm", "hbm", "tensor"]
    big = bench.scaled_shape(CONFIGS[4], peaks)
    assert big.N % CONFIGS[4].N == 0 and bench.roofline_time_us(big, peaks)[0] >= 50.0
