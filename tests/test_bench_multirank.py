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


def _split_worker(rank, world, port, out):
    """Each rank runs the oracle on its share of ONE problem's batch; rank 0 gathers the pieces."""
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import numpy as np
    import bench
    from oracle import hero_oracle as O
    from workloads import synthetic as S
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfgd = dict(S.CONFIGS["tiny"], batch=2, hidden=32, n_heads=2, head_dim=16, ffn_dim=64, temb_dim=16, frames=2,
                grid_h=4, grid_w=6, n_text=3, full_interval=3)
    mine, part = bench.shard_cfg_pair(cfgd, rank, world)
    weights = [S.block_weights(cfgd, l) for l in range(cfgd["n_blocks"])]
    orc = O.HeroOracle(O.Config.from_dict(mine), weights)
    x = S.tokens(cfgd)[part].astype(np.float64)
    lists = []
    for s in range(5):
        x = orc.step(s, x, S.temb(cfgd, s)[part])
        lists.append(orc.blocks[0].ages.copy())
    pieces = [torch.zeros(mine["batch"], *x.shape[1:], dtype=torch.float64) for _ in range(world)]
    dist.all_gather(pieces, torch.from_numpy(np.ascontiguousarray(x)))
    out[rank] = (torch.cat(pieces).numpy(), np.stack(lists), (part.start, part.stop), mine["batch"])
    dist.destroy_process_group()


def test_batch_items_of_one_problem_split_over_two_ranks_reproduce_the_unsplit_run():
    """The classifier-free-guidance pair is two independent sequences that share the selection lists (one
    draw per step and block for the whole batch): split over two ranks, with no exchange, the gathered
    result is the unsplit run's, and both ranks track the same ages."""
    import numpy as np
    from oracle import hero_oracle as O
    from workloads import synthetic as S
    world, port = 2, 31500 + os.getpid() % 2000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_split_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    cfgd = dict(S.CONFIGS["tiny"], batch=2, hidden=32, n_heads=2, head_dim=16, ffn_dim=64, temb_dim=16, frames=2,
                grid_h=4, grid_w=6, n_text=3, full_interval=3)
    weights = [S.block_weights(cfgd, l) for l in range(cfgd["n_blocks"])]
    orc = O.HeroOracle(O.Config.from_dict(cfgd), weights)
    x = S.tokens(cfgd).astype(np.float64)
    ages = []
    for s in range(5):
        x = orc.step(s, x, S.temb(cfgd, s))
        ages.append(orc.blocks[0].ages.copy())
    assert [res[r][2] for r in range(world)] == [(0, 1), (1, 2)] and res[0][3] == 1
    for r in range(world):
        np.testing.assert_allclose(res[r][0], x, rtol=1e-12, atol=1e-13)       # every rank gathered the whole batch
        assert np.array_equal(res[r][1], np.stack(ages))                       # same lists on every rank


def test_shard_cfg_pair_rejects_uneven_splits():
    import bench
    import pytest
    with pytest.raises(ValueError):
        bench.shard_cfg_pair(dict(batch=2), 0, 3)
    cfg, part = bench.shard_cfg_pair(dict(batch=4, seed=9), 1, 2)
    assert cfg == dict(batch=2, seed=9) and (part.start, part.stop) == (2, 4)
