"""The synthetic input recipes: sizes, determinism, distributions."""
import numpy as np

from workloads import CONFIGS, grads, scaled_config, weights
from workloads.generate import CHUNK


def test_sizes_match_the_published_architectures():
    c = CONFIGS
    assert (c["tiny"].N, c["tiny"].K, c["tiny"].k_core, c["tiny"].k_exp) == (1_000_000, 4, 100_000, 45_000)
    assert c["googlenet"].N == 6_998_552                       # inception-v1 main branch with biases
    assert c["vgg16"].N == 138_357_544                         # VGG-16 with biases
    assert (c["vgg16"].k_core, c["vgg16"].M, c["vgg16"].k_exp) == (6_917_877, 131_439_667, 1_314_396)
    assert c["resnet50_ties"].N == 25_557_032                  # ResNet-50 with BN affine parameters
    assert (c["resnet50_ties"].k_core, c["resnet50_ties"].k_exp) == (5_111_406, 1_022_281)
    assert c["large"].N == 10 ** 9 and c["large"].with_core_pct(30).k_core == 3 * 10 ** 8
    fc6 = [s for s in c["vgg16"].segments if s.name == "fc6.weight"][0]
    assert fc6.size == 25088 * 4096


def test_slices_are_reproducible_and_chunk_independent():
    cfg = CONFIGS["googlenet"]
    a, b = CHUNK - 1000, CHUNK + 5000
    w = weights(cfg, a, b)
    assert np.array_equal(w, weights(cfg, 0, b)[a:])
    g = grads(cfg, 3, a, b)
    assert np.array_equal(g, grads(cfg, 3, a, b))
    assert not np.array_equal(g, grads(cfg, 4, a, b))


def test_value_distributions():
    cfg = CONFIGS["tiny"]
    w, g = weights(cfg), grads(cfg, 0)
    assert abs(w.std() - 0.05) < 5e-4 and abs(g.std() - 1e-3) < 1e-5
    v = CONFIGS["vgg16"]
    lo, hi, seg = [b for b in v.bounds() if b[2].name == "fc7.weight"][0]
    w = weights(v, lo, lo + 500_000)
    assert abs(w.std() / seg.sigma - 1) < 0.01
    g = grads(v, 1, lo, lo + 500_000)
    assert abs(np.abs(g).mean() / 1e-4 - 1) < 0.01            # Laplace(0, b): E|x| = b
    assert abs(g.var() / (2e-8) - 1) < 0.02                   # variance 2 b^2
    lo, hi, seg = [b for b in v.bounds() if b[2].name == "fc7.bias"][0]
    assert np.all(weights(v, lo, hi) == 0)


def test_tie_stress_grid():
    r = CONFIGS["resnet50_ties"]
    w = weights(r, 0, 2_000_000)
    g = grads(r, 0, 0, 2_000_000)
    assert np.all(w * 512 == np.rint(w * 512)) and np.abs(w * 512).max() <= 128
    assert np.all(g * 65536 == np.rint(g * 65536)) and np.abs(g * 65536).max() <= 128
    assert len(np.unique(w)) <= 256 and len(np.unique(g)) <= 256


def test_scaled_config_is_a_prefix():
    v = CONFIGS["vgg16"]
    s = scaled_config(v, 3_000_000)
    assert s.N == 3_000_000 and s.K == v.K and s.seed == v.seed
    assert np.array_equal(weights(s), weights(v, 0, 3_000_000))
    assert np.array_equal(grads(s, 2), grads(v, 2, 0, 3_000_000))
