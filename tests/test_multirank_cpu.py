"""The N>1 path of the benchmark on CPU: two gloo ranks.  The attention path shards over independent batch elements
with no collective; what the ranks share is only the timing reduction (max over ranks) and the per-rank workload
derivation, which is what this test exercises."""
import os
import sys

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
        ms = bench.max_over_ranks(10.0 + 5.0 * rank, world, "cpu")
        w = bench.rank_workload("tiny", rank)
        q = bench.da2_inputs.make_tensor(w, 0, "cpu")
        out[rank] = (ms, w.seed, float(q.float().abs().sum()))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_take_max_time_and_distinct_batches():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    port = 29500 + (os.getpid() % 2000)
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    assert out[0][0] == out[1][0] == 15.0          # the slowest rank's time on every rank
    assert out[0][1] != out[1][1]                  # each rank draws its own batch element
    assert out[0][2] != out[1][2]


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, 1, "cpu") == 3.5
    assert bench.rank_workload("wan14b_720p", 0) == bench.da2_inputs.WORKLOADS["wan14b_720p"]
