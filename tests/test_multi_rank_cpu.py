"""The path does not shard across GPUs ("replicas only"): bench.py --gpus N runs N independent replicas
and reports units of all ranks over the slowest rank's time.  This checks that reduction with two gloo
ranks on the CPU, and that each rank's bookkeeping-only cache evolves independently."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2503_19950_b200 import LQ_DEVICE_NONE, LogQuantCache
    # every rank owns a private replica of the cache state: no collective touches it
    c = LogQuantCache(2, 1, 8, 2, 128, 32, max_tokens=4096, device=LQ_DEVICE_NONE)
    n = 500 + 300 * rank
    c.append(0, None, None, n_tokens=n)
    assert c.info(0).n_seen == n and c.info(1).n_seen == 0
    ms = [10.0 + 5.0 * rank, 100.0 - 30.0 * rank]
    ms_max = bench.reduce_max_over_ranks(ms, world, torch.device("cpu"))
    out[rank] = (ms_max, bench.aggregate_throughput(1000, world, ms_max[0]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_report_units_of_all_ranks_over_the_slowest_time():
    world = 2
    port = 29500 + os.getpid() % 2000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        for rank in range(world):
            ms_max, value = out[rank]
            assert ms_max == [15.0, 100.0]
            assert abs(value - 2 * 1000 / 15e-3) < 1e-6
