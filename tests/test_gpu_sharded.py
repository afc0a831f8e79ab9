"""Selection over a range-sharded model on the GPU: the shards of one vector are processed one
after the other on one device (histograms summed on the device, counts collected on the host), and
the concatenation of the shards' results must be, bit for bit, the oracle's core of the whole vector."""
import numpy as np
import pytest
import torch

import oracle
from test_gpu_parity import check_aux

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P():
    import paper_1709_09393_b200 as P
    return P


def _scores(case, n, rng):
    if case == "random":
        return np.abs(rng.standard_normal(n)).astype(np.float32)
    if case == "ties":          # a 64-value grid: the threshold's tie group straddles shard boundaries
        return (rng.integers(0, 64, n) / 64.0).astype(np.float32)
    if case == "bits":          # arbitrary bit patterns, NaNs and infinities included
        return rng.integers(0, 2 ** 32, n, dtype=np.uint64).astype(np.uint32).view(np.float32)
    raise ValueError(case)


@pytest.mark.parametrize("case", ["random", "ties", "bits"])
@pytest.mark.parametrize("shards", [2, 4, 7])
def test_sharded_selection_matches_the_oracle(P, case, shards):
    rng = np.random.default_rng(31 + shards)
    n = 1_000_003
    S = _scores(case, n, rng)
    bounds = P.shard_bounds(n, shards)
    parts = [torch.from_numpy(S[b:e].copy()).cuda() for b, e in bounds]
    for k in (1, n // 20, n // 2 + 7):
        ref = oracle.select_core(S, k).astype(np.int64)
        out = P.select_core_sharded(parts, k, P.CudaBackend())
        got = np.concatenate([o[0].cpu().numpy().view(np.uint32).astype(np.int64) + b for o, (b, e) in zip(out, bounds)])
        assert np.array_equal(got, ref), (case, shards, k)
        # every shard's core_aux describes its own part of the core (bitmap and directory on local indices)
        for (core_idx, core_aux, k_shard), (b, e) in zip(out, bounds):
            local = ref[(ref >= b) & (ref < e)] - b
            assert k_shard == local.size
            check_aux(P, core_aux, local.astype(np.uint32), e - b)


def test_sharded_selection_with_an_empty_shard_result(P):
    # all large scores sit in the last shard: the others contribute nothing to the core
    n, shards, k = 300_000, 3, 1000
    S = np.full(n, 0.25, np.float32)
    S[-5000:] = np.linspace(1.0, 2.0, 5000, dtype=np.float32)
    bounds = P.shard_bounds(n, shards)
    parts = [torch.from_numpy(S[b:e].copy()).cuda() for b, e in bounds]
    out = P.select_core_sharded(parts, k, P.CudaBackend())
    assert [o[2] for o in out] == [0, 0, k]
    got = out[2][0].cpu().numpy().view(np.uint32).astype(np.int64) + bounds[2][0]
    assert np.array_equal(got, oracle.select_core(S, k).astype(np.int64))
