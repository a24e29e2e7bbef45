"""The multi-rank bookkeeping of bench.py on CPU: two gloo ranks, max-over-ranks timing, whole-job value.

The layer shards without an exchange step, so `bench.py --gpus N` runs N replicas of the step; the only
collective is the reduction of the per-rank timings.
"""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _rank_main(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    per_rank = [10.0 + rank, 3.0 - rank, 7.0]          # rank 0: 10, 3, 7; rank 1: 11, 2, 7
    got = bench.max_over_ranks(per_rank, dist, torch.device("cpu"))
    out[rank] = got
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_two_gloo_ranks():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank_main, args=(world, 29581, out), nprocs=world, join=True)
        assert out[0] == out[1] == [11.0, 3.0, 7.0]


def test_single_rank_passthrough_and_whole_job_value():
    import bench
    assert bench.max_over_ranks([1.5, 2.5], None, None) == [1.5, 2.5]
    # two ranks, each 1e12 flop per step in 1 ms -> 2 PFLOP/s... in TFLOP/s
    assert abs(bench.whole_job_value(1e12, 1.0, 2) - 2000.0) < 1e-9
    assert bench.layer_flops(2, 4, 8, 1) == 2.0 * 2 * ((4 + 1) * 8 + 4 * 1)
    assert bench.layer_weight_bytes(4096, 4096, 32) == 0.5625 * 4096 * 4096 + 1.0625 * 32 * 8192
