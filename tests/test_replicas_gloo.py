"""Host-side logic of the N > 1 benchmark path on CPU: two gloo ranks, no GPU.

The learner path does not shard (one learner GPU by design), so `bench.py --gpus N` runs independent replicas;
what the ranks exchange is only the timing: the whole-job throughput divides by the slowest rank's time.
"""
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
        ms = [10.0 + 5.0 * rank, 100.0 - 30.0 * rank]   # rank 1 is slower on the first, faster on the second
        red = bench.max_over_ranks(ms, torch.device("cpu"))
        out[rank] = (red, bench.replicas_throughput(world, 16384, 5, red[0]))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_timing_is_the_max_over_ranks_and_value_is_the_whole_job():
    world = 2
    port = 29500 + os.getpid() % 2000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for rank in (0, 1):
        red, value = res[rank]
        assert red == [15.0, 100.0]
        assert abs(value - 2 * 16384 * 5 / 15.0e-3) < 1e-6 * value


def test_single_process_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5], torch.device("cpu")) == [1.5, 2.5]
    assert bench.replicas_throughput(1, 100, 2, 4.0) == 100 * 2 / 4.0e-3
