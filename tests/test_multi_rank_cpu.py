"""The N > 1 host logic of bench.py on CPU: two gloo ranks, each with its own tokens of the same
layer, no data-path collective; the job's time is the max over ranks and the throughput is the
sum of what all ranks processed over that time."""
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
    import gen
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        spec = gen.scaled(gen.CONFIGS["cfg2"], M=16, N=64, K=16, B=8)
        x = gen.make_x(bench.rank_spec(spec, rank))
        # every rank's replica packs the same layer (weights from `spec`) and gets its own tokens
        my_ms = 10.0 * (rank + 1)                         # rank 1 is the slow one
        ms = bench.max_over_ranks(dist, my_ms, "cpu")
        val = bench.aggregate_tokens_per_s(world, spec.B, ms)
        out[rank] = (ms, val, x[:2].tolist())
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_max_time_and_sum_of_tokens():
    world, port = 2, 29500 + (os.getpid() % 2000)
    mgr = mp.get_context("spawn").Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    assert out[0][0] == out[1][0] == 20.0                 # max over ranks
    assert out[0][1] == out[1][1] == pytest.approx(2 * 8 / 20e-3)
    assert out[0][2] != out[1][2]                         # different tokens per rank


def test_rank_spec_changes_tokens_only_by_seed():
    sys.path.insert(0, ROOT)
    import bench
    import gen
    spec = gen.CONFIGS["cfg2"]
    assert bench.rank_spec(spec, 0) is spec
    s1 = bench.rank_spec(spec, 1)
    assert (s1.M, s1.N, s1.K, s1.B, s1.density) == (spec.M, spec.N, spec.K, spec.B, spec.density)
    assert s1.seed != spec.seed
