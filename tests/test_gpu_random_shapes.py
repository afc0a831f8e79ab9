"""GPU parity on seeded random shapes: the whole round as one call against the oracle's round, bit for bit.

The fixed cases of test_gpu_parity.py pick their sizes and ratios by hand; here vector length, worker count,
core and explorer ratios and the value pattern (continuous, quantised with ties by the thousand, all equal,
layers of very different scale, a handful of distinct values) are drawn from a seeded generator, so that
combinations nobody thought of are met as well: short vectors (the selection's full path), vectors above
2^21 parameters (the sampled bracket, the fused scoring pass), empty and full cores, empty explorers.
"""
import numpy as np
import pytest
import torch

import oracle
from test_gpu_parity import assert_round_equal, gpu_round

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    import paper_1709_09393_b200 as pkg
    return pkg


def _draw(case: int):
    rng = np.random.default_rng(7_000_003 + case)
    scale = rng.choice([1e3, 1e4, 1e5, 3e6], p=[0.15, 0.2, 0.25, 0.4])
    n = int(rng.integers(1, int(scale))) + ((1 << 21) if scale >= 3e6 and rng.random() < 0.8 else 0)
    K = int(rng.choice([1, 2, 3, 4, 8, 9, 16]))
    alpha = rng.choice([0.0, 0.001, 0.01, 0.05, 0.2, 0.5, 0.9, 1.0])
    beta = rng.choice([0.0, 0.001, 0.01, 0.05, 0.3, 1.0])
    k_core = min(n, int(alpha * n))
    k_exp = min(n - k_core, int(beta * (n - k_core)))
    pattern = str(rng.choice(["normal", "quantised", "equal", "layers", "few_values"]))
    w = rng.standard_normal(n).astype(np.float32)
    if pattern == "normal":
        gs = [(0.01 * rng.standard_normal(n)).astype(np.float32) for _ in range(K)]
    elif pattern == "quantised":
        w = (np.round(w * 4) / 4).astype(np.float32)
        gs = [(np.round(rng.standard_normal(n) * 2) / 64).astype(np.float32) for _ in range(K)]
    elif pattern == "equal":
        w = np.full(n, 0.5, np.float32)
        gs = [np.zeros(n, np.float32) for _ in range(K)]
    elif pattern == "layers":
        sc = np.repeat(rng.choice([1e-3, 1.0, 30.0], size=(n + 4095) // 4096), 4096)[:n].astype(np.float32)
        w = (w * sc).astype(np.float32)
        gs = [(0.01 * rng.standard_normal(n) * sc).astype(np.float32) for _ in range(K)]
    else:
        w = rng.choice(np.array([0.0, 0.25, 1.0, 3.0], np.float32), size=n)
        gs = [rng.choice(np.array([0.0, 0.5], np.float32), size=n) for _ in range(K)]
    seed, rnd = int(rng.integers(0, 2 ** 62)), int(rng.integers(0, 1000))
    return w, gs, k_core, k_exp, seed, rnd, pattern


@pytest.mark.parametrize("case", range(48))
def test_round_one_call_on_a_random_shape(P, case):
    w, gs, k_core, k_exp, seed, rnd, pattern = _draw(case)
    c, eta = 0.7, 0.05
    ref = oracle.run_round(w, gs, c, k_core, k_exp, seed, rnd, eta)
    d_w, buf = gpu_round(P, w, gs, c, k_core, k_exp, seed, rnd, eta, True, True, False)
    assert_round_equal(P, d_w, buf, ref, w.size, scores=False)
