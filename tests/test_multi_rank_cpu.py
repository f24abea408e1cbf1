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


def test_gpus_flag_without_a_launcher_starts_that_many_replica_ranks():
    """`bench.py --gpus 2` with no WORLD_SIZE in the environment re-runs itself as two ranks; the CPU-only
    self-test arm takes them through the same max-over-ranks reduction as the real run (gloo, no GPU)."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR",
                                                            "MASTER_PORT")}
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "replica-selftest"],
                         capture_output=True, text=True, env=env, timeout=300)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [json.loads(l) for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1  # rank 0 alone prints
    assert lines[0]["n_gpus"] == 2 and lines[0]["ms_per_step"] == 15.0
    assert abs(lines[0]["value"] - 2 * 1000 / 15e-3) < 1e-6


def test_gpus_flag_fails_loudly_without_that_many_devices():
    import subprocess
    if torch.cuda.device_count() >= 2:
        return
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "1"],
                         capture_output=True, text=True, env=env, timeout=300)
    assert res.returncode != 0 and "CUDA device" in res.stderr
