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
    for k in (0, 1, n // 20, n // 2 + 7, n):
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


@pytest.mark.parametrize("shards", [2, 4, 7])
def test_sharded_explorer_and_exchange_match_the_oracle(P, shards):
    """The rest of a round on the shards of one vector: every shard draws its share of each worker's
    explorer and runs the exchange on shard-local indices; shifted by the shards' offsets and put together,
    explorers, packed values, merged model and pulled values are the oracle's round on the whole vector."""
    rng = np.random.default_rng(41 + shards)
    n, K, k_core, k_exp = 700_003, 3, 70_001, 31_003
    w = rng.standard_normal(n).astype(np.float32)
    gs = [(rng.standard_normal(n) * 1e-2).astype(np.float32) for _ in range(K)]
    ref = oracle.run_round(w, gs, 1.0, k_core, k_exp, 9, 4, 1.0 / K)
    bounds = P.shard_bounds(n, shards)
    S = oracle.score(w, gs, 1.0)
    parts = [torch.from_numpy(S[b:e].copy()).cuda() for b, e in bounds]
    sel = P.select_core_sharded(parts, k_core, P.CudaBackend())
    k_shard = [s[2] for s in sel]
    noncore = [(e - b) - k for (b, e), k in zip(bounds, k_shard)]        # what the all-gather of core sizes tells everyone
    noncore_total = sum(noncore)
    got_exp = [[] for _ in range(K)]
    merged = np.empty(n, np.float32)
    got_val = [np.zeros(k_core + k_exp, np.float32) for _ in range(K)]
    got_pull = [np.zeros(k_core + k_exp, np.float32) for _ in range(K)]
    core_at, exp_at = 0, [0] * K
    for g, ((b, e), (core_idx, core_aux, kc)) in enumerate(zip(bounds, sel)):
        ns = e - b
        below = sum(noncore[:g])
        ws = torch.empty(P.explore_shard_workspace_bytes(ns, noncore_total, k_exp), dtype=torch.uint8, device="cuda")
        exps = []
        for k in range(K):
            cap = min(k_exp, noncore[g])
            buf = torch.empty(cap, dtype=torch.int32, device="cuda")
            count = torch.zeros(1, dtype=torch.int32, device="cuda")
            P.slimdp_sample_explore_shard(core_aux, ns, kc, noncore_total, below, k_exp, 9, k, 4, buf, count, ws)
            P.read_status(ws)
            exps.append(buf[:int(count.item())].clone())
            got_exp[k].append(exps[k].cpu().numpy().view(np.uint32).astype(np.int64) + b)
        # the exchange runs per worker-list length, so each worker's share is exchanged on its own here:
        # pack, merge in worker order, pull (three calls; the shard's explorers have different lengths)
        d_w = torch.from_numpy(w[b:e].copy()).cuda()
        d_gs = [torch.from_numpy(gk[b:e].copy()).cuda() for gk in gs]
        vals = []
        for k in range(K):
            v = torch.empty(kc + exps[k].numel(), dtype=torch.float32, device="cuda")
            P.slimdp_pack(d_gs[k], core_idx, exps[k], v)
            vals.append(v)
        for k in range(K):          # one worker at a time keeps the worker order with lists of different lengths
            none = torch.empty(0, dtype=torch.int32, device="cuda")
            if k == 0:              # the core once, with all workers' core values
                P.slimdp_merge(d_w, core_idx, [none] * K, [v[:kc].contiguous() for v in vals], 1.0 / K)
            P.slimdp_merge(d_w, none, [exps[k]], [vals[k][kc:].contiguous()], 1.0 / K)
        merged[b:e] = d_w.cpu().numpy()
        for k in range(K):
            out = torch.empty(kc + exps[k].numel(), dtype=torch.float32, device="cuda")
            P.slimdp_pull(d_w, core_idx, exps[k], out)
            ne = exps[k].numel()
            got_val[k][core_at:core_at + kc] = vals[k][:kc].cpu().numpy()
            got_pull[k][core_at:core_at + kc] = out[:kc].cpu().numpy()
            got_val[k][k_core + exp_at[k]:k_core + exp_at[k] + ne] = vals[k][kc:].cpu().numpy()
            got_pull[k][k_core + exp_at[k]:k_core + exp_at[k] + ne] = out[kc:].cpu().numpy()
            exp_at[k] += ne
        core_at += kc
    u32 = lambda a: np.ascontiguousarray(a).view(np.uint32)
    for k in range(K):
        assert np.array_equal(np.concatenate(got_exp[k]), ref["exp_idx"][k].astype(np.int64)), f"explorer {k}"
        assert np.array_equal(u32(got_val[k]), u32(ref["val"][k])), f"packed values {k}"
        assert np.array_equal(u32(got_pull[k]), u32(ref["pulled"][k])), f"pulled values {k}"
    assert np.array_equal(u32(merged), u32(ref["w"]))
