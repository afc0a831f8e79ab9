"""Selection over a range-sharded model: the host logic (shard bounds, tie quotas, the order of
steps and reductions) on CPU, in one process and as two gloo ranks; the oracle's whole-vector
selection is the reference in every case."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

import oracle
from _shard_numpy import NumpyBackend
from paper_1709_09393_b200.sharded import select_core_sharded, shard_bounds, tie_quotas


def test_shard_bounds_cover_the_vector_in_order():
    for n, g in ((10, 3), (7, 7), (5, 8), (138_357_544, 8), (1, 1)):
        b = shard_bounds(n, g)
        assert len(b) == g and b[0][0] == 0 and b[-1][1] == n
        assert all(b[i][1] == b[i + 1][0] for i in range(g - 1))
        sizes = [e - s for s, e in b]
        assert max(sizes) - min(sizes) <= 1 and sizes == sorted(sizes, reverse=True)


def test_tie_quotas_hand_the_ties_to_the_lowest_shards():
    # 9 wanted, 6 above the threshold, so 3 ties: shard 0 has 2 equal keys, shard 1 none, shard 2 five
    assert tie_quotas([3, 2, 1], [2, 0, 5], 9) == [2, 0, 1]
    assert tie_quotas([0, 0], [4, 4], 8) == [4, 4]
    assert tie_quotas([5], [1], 5) == [0]
    with pytest.raises(ValueError):
        tie_quotas([3], [1], 6)            # more ties wanted than exist
    with pytest.raises(ValueError):
        tie_quotas([7], [1], 6)            # more keys above the threshold than wanted


def _scores(case, n, rng):
    if case == "random":
        return np.abs(rng.standard_normal(n)).astype(np.float32)
    if case == "ties":          # a 16-value grid: the threshold's tie group straddles shard boundaries
        return (rng.integers(0, 16, n) / 16.0).astype(np.float32)
    if case == "all_equal":
        return np.full(n, 0.5, np.float32)
    raise ValueError(case)


@pytest.mark.parametrize("case", ["random", "ties", "all_equal"])
@pytest.mark.parametrize("shards", [1, 2, 4, 7])
def test_sharded_selection_equals_the_whole_vector_selection(case, shards):
    rng = np.random.default_rng(5)
    n = 20_011
    S = _scores(case, n, rng)
    for k in (0, 1, n // 10, n // 2 + 3, n):
        ref = oracle.select_core(S, k)
        parts = [torch.from_numpy(S[b:e].copy()) for b, e in shard_bounds(n, shards)]
        out = select_core_sharded(parts, k, NumpyBackend())
        got = np.concatenate([o[0].numpy().view(np.uint32).astype(np.int64) + b
                              for o, (b, e) in zip(out, shard_bounds(n, shards))])
        assert np.array_equal(got, ref.astype(np.int64)), (case, shards, k)
        assert sum(o[2] for o in out) == k


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, n, k, case, q):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    rng = np.random.default_rng(6)
    S = _scores(case, n, rng)                       # every rank draws the same vector and keeps its shard
    b, e = shard_bounds(n, world)[rank]
    (core, _, k_shard), = select_core_sharded([torch.from_numpy(S[b:e].copy())], k, NumpyBackend())
    q.put((rank, (core.numpy().view(np.uint32).astype(np.int64) + b).tolist(), k_shard))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("case", ["random", "ties"])
def test_sharded_selection_as_two_gloo_ranks(case):
    n, k, world = 30_007, 4_321, 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, n, k, case, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    S = _scores(case, n, np.random.default_rng(6))
    ref = oracle.select_core(S, k)
    assert np.array_equal(np.array(got[0][1] + got[1][1], dtype=np.int64), ref.astype(np.int64))
    assert got[0][2] + got[1][2] == k
