"""The multi-rank bookkeeping of bench.py on CPU: two gloo ranks, no GPU.

The path has no exchange step (replicas only), so all that crosses ranks is the maximum of the
timings; the whole-job value is the units of all ranks over the slowest rank's time."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms, e2e = bench.max_over_ranks([10.0 + 5.0 * rank, 40.0 - 3.0 * rank], dist, "cpu")
    rate = bench.whole_job_rate(4096.0 * 32, world, ms)
    with open(os.path.join(out_dir, f"r{rank}.txt"), "w") as f:
        f.write(f"{ms} {e2e} {rate} {bench.replica_seed_base(rank)}")
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_reduction(tmp_path):
    world, port = 2, 29500 + (os.getpid() % 2000)
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    rows = [open(tmp_path / f"r{r}.txt").read().split() for r in range(world)]
    for r in rows:
        assert float(r[0]) == 15.0 and float(r[1]) == 40.0          # max over ranks, element-wise
        assert float(r[2]) == pytest.approx(4096.0 * 32 * 2 / 15e-3)
    assert rows[0][3] != rows[1][3]                                  # replicas use different seeds


def test_single_process_is_identity():
    import bench
    assert bench.max_over_ranks([3.0, 4.0]) == [3.0, 4.0]
    assert bench.whole_job_rate(100.0, 1, 50.0) == pytest.approx(2000.0)
