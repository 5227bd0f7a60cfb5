"""The N > 1 path of the benchmark is "replicas only": every rank runs the whole workload, the only exchange is
the max-over-ranks of the measured time.  Two gloo ranks on CPU check that aggregation (no GPU needed)."""
import os
import sys

import pytest

torch = pytest.importorskip("torch")
import torch.multiprocessing as mp  # noqa: E402

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms_local = 100.0 + 25.0 * rank                    # rank 1 is the slow one
    dist.barrier()
    ms = bench.max_over_ranks(ms_local, world, torch.device("cpu"))
    value = bench.aggregate_tokens_per_s(world, 8, 50, ms)
    out[rank] = (ms, value)
    dist.destroy_process_group()


def test_two_rank_aggregation_uses_the_slowest_rank():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    port = 29500 + os.getpid() % 1000
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    for rank in range(world):
        ms, value = out[rank]
        assert ms == 125.0                             # every rank reports the slowest rank's time
        assert abs(value - 2 * 8 * 50 / 0.125) < 1e-6  # whole-job tokens/s of two replicas


def test_single_rank_is_a_no_op():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(12.5, 1, None) == 12.5
    assert bench.aggregate_tokens_per_s(1, 8, 100, 1000.0) == 800.0
