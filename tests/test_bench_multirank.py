"""The N > 1 path of bench.py on CPU: two gloo ranks, each with its own timing; rank 0 must see the
slowest rank's time and the whole-job throughput built from it; every rank draws its own problem."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    my_ms = 10.0 + 5.0 * rank                       # rank 1 is the slow one
    dist.barrier()
    total = bench.max_over_ranks(my_ms, dist, torch.device("cpu"))
    value = bench.whole_job_throughput(1000, world, total)
    seeds = [torch.zeros(1, dtype=torch.int64) for _ in range(world)]
    dist.all_gather(seeds, torch.tensor([bench.rank_seed(3, rank)]))
    out[rank] = (total, value, [int(s) for s in seeds])
    dist.destroy_process_group()


def test_two_gloo_ranks_report_the_slowest_time_and_the_aggregate():
    world, port = 2, 29500 + os.getpid() % 2000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    for rank in range(world):
        total, value, seeds = res[rank]
        assert total == 15.0                                   # max over ranks, on every rank
        assert abs(value - 2 * 1000 / 15e-3) < 1e-6            # units of all ranks / slowest time
        assert seeds == [3, 4]                                 # independent problems


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.max_over_ranks(7.5, None, torch.device("cpu")) == 7.5
    assert bench.whole_job_throughput(35552, 1, 80.0) == 35552 / 0.08
