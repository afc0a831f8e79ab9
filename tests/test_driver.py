"""Algorithm 1's schedule: the oracle driver against what the paper fixes (CPU), and the
device driver against the oracle driver round by round (GPU)."""
import numpy as np
import pytest

import oracle
from oracle.driver import Driver


def bits(a):
    return np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)


def _updates(rng, n, K, scale=1e-2):
    return [(rng.standard_normal(n) * scale).astype(np.float32) for _ in range(K)]


def test_worker_merge_overwrites_exactly_the_communication_set():
    # Section 3.3 step 5
    w = np.arange(10, dtype=np.float32)
    out = oracle.worker_merge(w, np.array([1, 4], np.uint32), np.array([7], np.uint32),
                              np.array([-1.0, -4.0, -7.0], np.float32))
    assert out.tolist() == [0, -1, 2, 3, -4, 5, 6, -7, 8, 9]


@pytest.mark.parametrize("q", [1, 2, 5])
def test_full_communication_ratio_is_plump_dp_for_any_core_size_and_q(q):
    # alpha = 100 %: every round transfers everything, whatever beta and q are (Sections 2.1, 3.5):
    # the global model follows the dense merge and every local model equals it after the pull
    rng = np.random.default_rng(q)
    n, K, k_core = 3000, 3, 700
    w = rng.standard_normal(n).astype(np.float32)
    d = Driver(w, K, k_core, n - k_core, q, 1.0, 1.0 / K, seed=5)
    ref = w.copy()
    for t in range(6):
        ds = _updates(rng, n, K)
        d.round(ds)
        ref = oracle.dense_merge(ref, ds, 1.0 / K)
        assert np.array_equal(bits(d.w), bits(ref)), t
        for k in range(K):
            assert np.array_equal(bits(d.local[k]), bits(ref)), (t, k)


def test_schedule_of_dense_pushes_and_reselections():
    rng = np.random.default_rng(11)
    n, K, k_core, k_exp, q = 4000, 2, 400, 200, 3
    w = rng.standard_normal(n).astype(np.float32)
    d = Driver(w, K, k_core, k_exp, q, 1.0, 0.5, seed=1)
    # the first core is the magnitude top-k of the initial model
    assert np.array_equal(d.core, oracle.select_core(np.abs(w), k_core))
    cores = [d.core.copy()]
    for t in range(7):
        before = d.w.copy()
        ds = _updates(rng, n, K, 0.3)
        d.round(ds)
        cores.append(d.core.copy())
        changed = np.flatnonzero(bits(d.w) != bits(before))
        if (t + 1) % q == 0:
            # dense push: the whole model moves, and the core is reselected from the updated model
            assert changed.size > 0.99 * n
            assert np.array_equal(d.core, oracle.select_core(oracle.score(d.w, ds, 1.0), k_core))
        else:
            # sparse push: only the communication sets move, the core stays
            allowed = np.union1d(cores[t], np.concatenate(d.exp))
            assert np.all(np.isin(changed, allowed))
            assert np.array_equal(cores[t + 1], cores[t])
        for k in range(K):
            tc = np.concatenate([cores[t], d.exp[k]])
            assert np.array_equal(bits(d.local[k][tc]), bits(d.w[tc]))       # pulled values are in the local model
    assert d.t == 7
    assert not np.array_equal(cores[0], cores[3]) and not np.array_equal(cores[3], cores[6])


@pytest.mark.gpu
@pytest.mark.parametrize("n,K,k_core,k_exp,q", [(200_003, 4, 20_000, 9_000, 3), (50_001, 2, 0, 5_000, 2),
                                                (50_001, 3, 5_000, 0, 1), (3_000_017, 3, 300_000, 60_000, 2)])
def test_device_driver_follows_the_oracle_driver(n, K, k_core, k_exp, q):
    import torch
    import paper_1709_09393_b200 as P
    rng = np.random.default_rng(n + q)
    w = (rng.standard_normal(n) * 0.05).astype(np.float32)
    ref = Driver(w, K, k_core, k_exp, q, 1.0, 1.0 / K, seed=9)
    dev = P.SlimDPDriver(torch.from_numpy(w).cuda(), K, k_core, k_exp, q, 1.0, 1.0 / K, seed=9)
    u32 = lambda t: t.cpu().numpy().view(np.uint32)
    assert np.array_equal(u32(dev.buf.core_idx), ref.core)
    for t in range(2 * q + 1):
        ds = _updates(rng, n, K, 1e-2)
        ref.round(ds)
        dev.round([torch.from_numpy(d).cuda() for d in ds])
        dev.check()
        assert np.array_equal(u32(dev.w), bits(ref.w)), ("global model", t)
        assert np.array_equal(u32(dev.buf.core_idx), ref.core), ("core", t)
        for k in range(K):
            assert np.array_equal(u32(dev.buf.exp_idx[k]), ref.exp[k]), ("explorer", t, k)
            assert np.array_equal(u32(dev.buf.pulled[k]), bits(ref.pulled[k])), ("pulled", t, k)
            assert np.array_equal(u32(dev.local[k]), bits(ref.local[k])), ("local model", t, k)


@pytest.mark.gpu
def test_dense_merge_score_and_worker_merge_parity():
    import torch
    import paper_1709_09393_b200 as P
    rng = np.random.default_rng(3)
    for n, K in [(1, 1), (5, 3), (100_007, 8), (100_007, 17)]:
        w = rng.standard_normal(n).astype(np.float32)
        ds = _updates(rng, n, K, 0.1)
        merged = oracle.dense_merge(w, ds, 0.3)
        S = oracle.score(merged, ds, 0.7)
        d_w = torch.from_numpy(w).cuda()
        scores = torch.empty(n, dtype=torch.float32, device="cuda")
        P.slimdp_dense_merge_score(d_w, [torch.from_numpy(d).cuda() for d in ds], 0.3, 0.7, scores)
        assert np.array_equal(d_w.cpu().numpy().view(np.uint32), bits(merged))
        assert np.array_equal(scores.cpu().numpy().view(np.uint32), bits(S))
        # unaligned views and no scores: the scalar path
        big = torch.zeros(n + 3, dtype=torch.float32, device="cuda")
        big[1:n + 1] = torch.from_numpy(w).cuda()
        P.slimdp_dense_merge_score(big[1:n + 1], [torch.from_numpy(d).cuda() for d in ds], 0.3, 0.7, None)
        assert np.array_equal(big[1:n + 1].cpu().numpy().view(np.uint32), bits(merged))
        assert float(big[0]) == 0.0 and float(big[n + 1]) == 0.0
