"""bench.py's multi-rank glue on CPU: two gloo ranks, the job's step time is the slowest
rank's, the value counts every rank's parameters (replicas, weak scaling)."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank: int, world: int, port: int, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert bench.dist_env() == (rank, rank, world)
    mine = 2.0 + rank            # rank 1 is the slower replica
    dist.barrier()
    slowest = bench.max_over_ranks(mine, world)
    out[rank] = (slowest, bench.aggregate_value(1_000_000, world, slowest))
    dist.destroy_process_group()


def test_max_over_ranks_and_aggregate_value_two_gloo_ranks():
    world, port = 2, 29000 + os.getpid() % 2000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    slowest, value = res[0]
    assert slowest == 3.0
    assert abs(value - 2 * 1_000_000 / 3.0e-3 / 1e9) < 1e-12


def test_single_rank_passthrough():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(1.25, 1) == 1.25
    assert bench.aggregate_value(138_357_544, 1, 2.0) == 138_357_544 / 2.0e-3 / 1e9
    b = bench.model_bytes(138_357_544, 8, 6_917_877, 1_314_396)
    assert b["score"] == 5_534_301_760 and b["round"] == 8_366_342_045     # the byte model's VGG-16-shaped totals
