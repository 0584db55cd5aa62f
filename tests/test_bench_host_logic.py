"""Host-side logic of the benchmark that only matters with more than one rank, on CPU with gloo."""
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
    import workloads as W
    slow = bench.max_over_ranks(10.0 + 5.0 * rank, world, torch.device("cpu"))
    wl = W.get_config("c1_tiny")
    mine = bench.rank_workload(wl, rank)
    q, _, _ = W.make_step(mine, 0, 1)
    gathered = [torch.zeros_like(q) for _ in range(world)]
    dist.all_gather(gathered, q)
    out[rank] = (slow, bool(torch.equal(gathered[0], gathered[1])), bench.whole_job_rate(slow, world))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_take_the_slowest_time_and_distinct_shards():
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, 29611, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == 15.0 and res[1][0] == 15.0          # max over ranks, seen by both
    assert res[0][1] is False                                # ranks draw different batch rows (weak scaling)
    assert abs(res[0][2] - 2 * 1e3 / 15.0) < 1e-9            # whole-job steps/s = ranks x steps / slowest time


def test_algorithmic_bytes_formula():
    sys.path.insert(0, ROOT)
    import bench
    import workloads as W
    wl = W.get_config("c4_cerebras")
    per_unit = 4 * 128 * 2049 + 12 * 2049 + 12 * 128
    assert bench.algorithmic_bytes_per_launch(wl) == 1024 * per_unit
