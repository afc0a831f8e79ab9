"""CPU-only pins of the oracle against what the paper and the mathematics fix.

Each test names the passage it pins.  None of the expected values comes from
the oracle itself or from the CUDA path: they are hand-computed exact binary
values, exact rational arithmetic, brute force over all subsets, published
known answers of the counter-based generator, or invariants stated in the
paper.
"""
import itertools
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from _exact import (explore_py, fma_f32, frac, perm_py, philox_py, round_f32,
                    round_keys_py)

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bits(a):
    return np.asarray(a, dtype=np.float32).view(np.uint32)


# ----------------------------------------------------------------- generator

def _kat_rows():
    rows = []
    with open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            v = [int(x, 16) for x in line.split()]
            rows.append((v[0:4], v[4:6], v[6:10]))
    assert len(rows) == 3
    return rows


@pytest.mark.parametrize("ctr,key,out", _kat_rows())
def test_philox_known_answers(ctr, key, out):
    # published known answers of Philox-4x32-10 (Salmon et al., SC'11)
    assert oracle.philox4x32_10(key, ctr) == out
    assert philox_py(key, ctr) == out


def test_round_keys_and_permutation_match_bigint_restatement():
    rng = np.random.default_rng(7)
    for _ in range(40):
        seed = int(rng.integers(0, 2 ** 63)) * 2 + int(rng.integers(0, 2))
        worker, rnd = int(rng.integers(0, 64)), int(rng.integers(0, 2 ** 32))
        rk = oracle.round_keys(seed, worker, rnd)
        assert [int(x) for x in rk] == round_keys_py(seed, worker, rnd)
        M = int(rng.integers(1, 2 ** 32))
        for j in rng.integers(0, M, size=8):
            assert oracle.feistel_perm(int(j), M, rk) == perm_py(int(j), M, list(map(int, rk)))


def test_permutation_is_a_bijection_for_every_small_M():
    # cycle-walking a bijection of [0, 2^(2h)) restricted to [0, M) is a bijection of [0, M)
    for M in range(1, 301):
        rk = oracle.round_keys(12345 + M, M % 7, M % 5)
        img = sorted(oracle.feistel_perm(j, M, rk) for j in range(M))
        assert img == list(range(M)), M


def test_permutation_bijection_at_power_of_two_edges():
    for M in (255, 256, 257, 4095, 4096, 4097, 65536, 65537):
        rk = oracle.round_keys(99, 1, M)
        img = np.array([oracle.feistel_perm(j, M, rk) for j in range(M)])
        assert np.array_equal(np.sort(img), np.arange(M)), M


# --------------------------------------------------------------------- score

def test_score_hand_example_eq1():
    # Eq. 1 with values exact in binary: S = |w| + c|g|
    w = np.array([0.5, -0.25, 0.0, 1.0], np.float32)
    g = np.array([0.0, 1.0, -2.0, 0.125], np.float32)
    S = oracle.score(w, [g], 0.5)
    assert S.tolist() == [0.5, 0.75, 1.0, 1.0625]


def test_score_reduces_to_magnitude_and_to_gradient():
    rng = np.random.default_rng(0)
    w = rng.standard_normal(1000).astype(np.float32)
    g = rng.standard_normal(1000).astype(np.float32)
    z = np.zeros(1000, np.float32)
    # g = 0: pure magnitude ranking (the weight-pruning measure of Section 3.2)
    assert np.array_equal(bits(oracle.score(w, [z], 3.0)), bits(np.abs(w)))
    # w = 0, c = 1: |g|
    assert np.array_equal(bits(oracle.score(z, [g], 1.0)), bits(np.abs(g)))
    # sign symmetry of both terms
    assert np.array_equal(bits(oracle.score(-w, [-g], 0.7)), bits(oracle.score(w, [g], 0.7)))


def test_score_is_one_rounding_of_the_exact_value():
    rng = np.random.default_rng(1)
    n = 400
    w = (rng.standard_normal(n) * 10.0 ** rng.integers(-42, 3, n)).astype(np.float32)
    g = (rng.standard_normal(n) * 10.0 ** rng.integers(-42, 3, n)).astype(np.float32)
    c = np.float32(0.3)
    S = oracle.score(w, [g], float(c))
    for i in range(n):
        exact = abs(frac(w[i])) + frac(c) * abs(frac(g[i]))
        assert bits(S[i]) == bits(round_f32(exact)), i


def test_score_sums_workers_left_to_right_in_fp32():
    # (a + b) + c differs from a + (b + c) in binary32 for these values
    a, b, c_ = np.float32(1.0), np.float32(2.0 ** -24), np.float32(2.0 ** -24)
    left = np.float32(np.float32(a + b) + c_)
    right = np.float32(a + np.float32(b + c_))
    assert left != right
    z = np.zeros(1, np.float32)
    S = oracle.score(z, [np.array([a]), np.array([b]), np.array([c_])], 1.0)
    assert S[0] == left
    rng = np.random.default_rng(2)
    gs = [rng.standard_normal(500).astype(np.float32) for _ in range(5)]
    acc = gs[0].copy()
    for g in gs[1:]:
        acc = (acc + g).astype(np.float32)
    assert np.array_equal(bits(oracle.score(np.zeros(500, np.float32), gs, 1.0)), bits(np.abs(acc)))


def test_score_nonfinite():
    w = np.array([np.inf, 1.0, np.nan, 0.0, -0.0], np.float32)
    g = np.array([0.0, np.inf, 0.0, np.nan, -0.0], np.float32)
    S = oracle.score(w, [g], 1.0)
    assert bits(S).tolist() == [0x7F800000, 0x7F800000, 0x7FC00000, 0x7FC00000, 0]


# -------------------------------------------------------------------- select

def _valid_core(S, C):
    """C is the top set under (score descending, index ascending): every member beats every non-member."""
    key = bits(S)
    inside = set(C)
    for a in C:
        for b in range(len(S)):
            if b in inside:
                continue
            if not (key[a] > key[b] or (key[a] == key[b] and a < b)):
                return False
    return True


def test_select_brute_force_over_all_subsets():
    rng = np.random.default_rng(3)
    for trial in range(30):
        n = int(rng.integers(1, 11))
        S = rng.integers(0, 4, n).astype(np.float32) * np.float32(0.25)   # many ties
        for k in range(n + 1):
            valid = [C for C in itertools.combinations(range(n), k) if _valid_core(S, C)]
            assert len(valid) == 1
            assert oracle.select_core(S, k).tolist() == list(valid[0])


def test_select_closed_cases():
    n, k = 1000, 137
    assert oracle.select_core(np.full(n, 0.5, np.float32), k).tolist() == list(range(k))
    inc = np.arange(n, dtype=np.float32)
    assert oracle.select_core(inc, k).tolist() == list(range(n - k, n))
    assert oracle.select_core(inc[::-1].copy(), k).tolist() == list(range(k))
    assert oracle.select_core(inc, 0).size == 0
    assert oracle.select_core(inc, n).tolist() == list(range(n))
    # NaN (canonical) ranks above +inf, +inf above everything finite
    S = np.array([1.0, np.inf, 3.0, 2.0], np.float32)
    S[3] = np.uint32(0x7FC00000).view(np.float32)
    assert oracle.select_core(S, 2).tolist() == [1, 3]


def test_select_against_partition_on_random_scores():
    rng = np.random.default_rng(4)
    n, k = 200_000, 20_000
    S = np.abs(rng.standard_normal(n)).astype(np.float32)
    S[rng.integers(0, n, 5000)] = S[17]          # a tie group
    core = oracle.select_core(S, k)
    assert core.size == k and np.all(np.diff(core.astype(np.int64)) > 0)
    kth = np.partition(S, n - k)[n - k]           # library routine: k-th largest value
    inside = np.zeros(n, bool)
    inside[core] = True
    assert S[inside].min() == kth
    assert np.all(S[~inside] <= kth) and np.all(S[inside] >= kth)
    tied = np.flatnonzero(S == kth)
    sel_tied, unsel_tied = tied[inside[tied]], tied[~inside[tied]]
    if sel_tied.size and unsel_tied.size:
        assert sel_tied.max() < unsel_tied.min()  # ties go to the smaller indices


# ------------------------------------------------------------------- explore

def _random_core(rng, n, k):
    return np.sort(rng.choice(n, size=k, replace=False)).astype(np.uint32)


def test_explore_invariants():
    # Section 3.1 item 2 / Section 3.3 step 2: exact size, outside the core, distinct
    rng = np.random.default_rng(5)
    for n, k_core, k_exp in [(1000, 100, 45), (1000, 0, 300), (1000, 1000, 0), (1000, 999, 1),
                             (4097, 1234, 2863), (50_000, 5000, 2250), (1, 0, 1), (2, 1, 1)]:
        core = _random_core(rng, n, k_core)
        e = oracle.sample_explore(core, n, k_exp, seed=11, worker=2, rnd=3)
        assert e.size == k_exp
        assert np.all(np.diff(e.astype(np.int64)) > 0)
        assert e.size == 0 or int(e.max()) < n
        assert np.intersect1d(core, e).size == 0
        if k_exp == n - k_core:           # everything outside the core
            assert np.array_equal(e, np.setdiff1d(np.arange(n, dtype=np.uint32), core))


def test_explore_resampled_per_worker_and_per_round_but_reproducible():
    rng = np.random.default_rng(6)
    n = 20_000
    core = _random_core(rng, n, 2000)
    a = oracle.sample_explore(core, n, 900, 5, 0, 0)
    assert np.array_equal(a, oracle.sample_explore(core, n, 900, 5, 0, 0))
    for seed, worker, rnd in [(5, 1, 0), (5, 0, 1), (6, 0, 0), (5 + 2 ** 32, 0, 0)]:
        b = oracle.sample_explore(core, n, 900, seed, worker, rnd)
        assert not np.array_equal(a, b)
        # two independent 5 % samples overlap in about 5 % of their members, not in most
        assert np.intersect1d(a, b).size < 200


def test_explore_matches_bigint_restatement():
    rng = np.random.default_rng(8)
    for n, k_core, k_exp in [(300, 30, 40), (1025, 100, 925), (5000, 4000, 100)]:
        core = _random_core(rng, n, k_core)
        got = oracle.sample_explore(core, n, k_exp, seed=2 ** 40 + 17, worker=3, rnd=9)
        assert got.tolist() == explore_py(core, n, k_exp, 2 ** 40 + 17, 3, 9)


def test_explore_inclusion_is_uniform_over_the_noncore():
    # "randomly picking ... from those other than the core": every non-core
    # parameter is included equally often (chi-square over many rounds)
    n, k_core, k_exp, rounds = 1100, 100, 50, 4000
    core = np.arange(0, n, 11, dtype=np.uint32)         # every 11th parameter is core
    assert core.size == k_core
    counts = np.zeros(n, np.int64)
    for t in range(rounds):
        counts[oracle.sample_explore(core, n, k_exp, seed=0, worker=0, rnd=t)] += 1
    assert counts[core].sum() == 0
    M = n - k_core
    noncore = np.setdiff1d(np.arange(n), core)
    expect = rounds * k_exp / M
    chi2 = float(((counts[noncore] - expect) ** 2 / expect).sum())
    dof = M - 1
    assert abs(chi2 - dof) < 5 * np.sqrt(2 * dof), chi2
    # per-worker streams are independent as well
    counts_w = np.zeros(n, np.int64)
    for k in range(64):
        for t in range(60):
            counts_w[oracle.sample_explore(core, n, k_exp, seed=1, worker=k, rnd=t)] += 1
    expect = 64 * 60 * k_exp / M
    chi2 = float(((counts_w[noncore] - expect) ** 2 / expect).sum())
    assert abs(chi2 - dof) < 5 * np.sqrt(2 * dof), chi2


# --------------------------------------------------------- pack / merge / pull

def test_pack_and_pull_identity_and_layout():
    rng = np.random.default_rng(9)
    n = 1000
    d = rng.standard_normal(n).astype(np.float32)
    allidx = np.arange(n, dtype=np.uint32)
    none = np.zeros(0, np.uint32)
    assert np.array_equal(oracle.pack(d, allidx, none), d)
    assert np.array_equal(oracle.pack(d, none, allidx), d)
    core, exp = np.array([3, 10, 999], np.uint32), np.array([0, 7], np.uint32)
    assert oracle.pack(d, core, exp).tolist() == [d[3], d[10], d[999], d[0], d[7]]
    assert oracle.pull(d, core, exp).tolist() == [d[3], d[10], d[999], d[0], d[7]]


def test_merge_single_worker_closed_form_and_sign():
    # Section 3.3 step 3: w <- w - eta' * delta on the communication set
    w = np.array([1.0, 2.0, 3.0, 4.0], np.float32)
    core, exp = np.array([1], np.uint32), [np.array([3], np.uint32)]
    val = [np.array([0.5, -2.0], np.float32)]
    out = oracle.merge(w, core, exp, val, 0.5)
    assert out.tolist() == [1.0, 1.75, 3.0, 5.0]
    rng = np.random.default_rng(10)
    n = 300
    w = rng.standard_normal(n).astype(np.float32)
    d = rng.standard_normal(n).astype(np.float32)
    eta = np.float32(0.37)
    idx = np.arange(n, dtype=np.uint32)
    out = oracle.merge(w, idx, [np.zeros(0, np.uint32)], [d], float(eta))
    for i in range(n):      # one rounding of the exact w - eta*d
        assert bits(out[i]) == bits(fma_f32(-eta, d[i], w[i])), i


def test_merge_applies_workers_in_ascending_order():
    # two workers whose explorers collide on one parameter; values chosen so
    # the two application orders round differently in binary32
    w0 = np.float32(1.0)
    a, b = np.float32(2.0 ** -24), np.float32(-1.5 * 2.0 ** -23)
    first_a = fma_f32(-1.0, b, fma_f32(-1.0, a, w0))
    first_b = fma_f32(-1.0, a, fma_f32(-1.0, b, w0))
    assert bits(first_a) != bits(first_b)
    w = np.array([w0, 5.0], np.float32)
    none = np.zeros(0, np.uint32)
    e = [np.array([0], np.uint32), np.array([0], np.uint32)]
    out = oracle.merge(w, none, e, [np.array([a]), np.array([b])], 1.0)
    assert bits(out[0]) == bits(first_a) and out[1] == 5.0
    out = oracle.merge(w, none, e, [np.array([b]), np.array([a])], 1.0)
    assert bits(out[0]) == bits(first_b)


def test_merge_stores_every_nan_result_as_the_canonical_quiet_nan():
    # Section 3.3 step 3 defines the merged value; which NaN payload comes out of an update is open in
    # IEEE 754, so the contract fixes it: any NaN result is stored as 0x7FC00000.  Pack and pull move bits.
    odd_nans = np.array([0x7F800001, 0xFFC12345, 0x7FFFFFFF, 0xFF800001], np.uint32).view(np.float32)
    inf = np.float32(np.inf)
    #            NaN model x4 (signalling, negative, all-ones, negative signalling), inf - inf, finite
    w = np.concatenate([odd_nans, np.array([inf, -inf, 1.0, 2.0], np.float32)])
    d = np.array([1.0, 2.0, 3.0, 4.0, inf, -inf, odd_nans[1], 0.5], np.float32)
    d.view(np.uint32)[6] = 0xFFC12345
    n = w.size
    core = np.array([0, 2, 4, 6], np.uint32)
    exp = [np.array([1, 3, 5, 7], np.uint32)]
    val = [oracle.pack(d, core, exp[0])]
    assert bits(val[0]).tolist() == bits(d[[0, 2, 4, 6, 1, 3, 5, 7]]).tolist()      # payloads kept by pack
    out = oracle.merge(w, core, exp, val, 0.5)
    canon = 0x7FC00000
    assert bits(out).tolist() == [canon] * 7 + [int(bits(np.float32(1.75)))]
    assert bits(oracle.pull(out, core, exp[0])).tolist() == bits(out[[0, 2, 4, 6, 1, 3, 5, 7]]).tolist()
    dense = oracle.dense_merge(w, [d], 0.5)
    assert bits(dense).tolist() == bits(out).tolist()
    # an untouched NaN keeps its payload: only results of updates are canonical
    untouched = oracle.merge(w, np.array([7], np.uint32), [np.zeros(0, np.uint32)], [np.array([0.5], np.float32)], 0.5)
    assert bits(untouched[:4]).tolist() == bits(odd_nans).tolist()


def test_dense_merge_is_sequential_rounding_of_exact_updates():
    rng = np.random.default_rng(11)
    n, K = 200, 3
    w = rng.standard_normal(n).astype(np.float32)
    gs = [rng.standard_normal(n).astype(np.float32) for _ in range(K)]
    eta = np.float32(1.0 / 3.0)
    out = oracle.dense_merge(w, gs, float(eta))
    for i in range(n):
        x = w[i]
        for k in range(K):
            x = fma_f32(-eta, gs[k][i], x)
        assert bits(out[i]) == bits(x), i


@pytest.mark.parametrize("form", ["all_core", "all_explore", "core_plus_rest"])
def test_full_communication_ratio_reproduces_plump_dp(form):
    # alpha = 100 %: Slim-DP transfers everything, i.e. Plump-DP (Sections 2.1, 3.5)
    rng = np.random.default_rng(12)
    n, K = 5000, 4
    w = rng.standard_normal(n).astype(np.float32)
    gs = [(rng.standard_normal(n) * 1e-2).astype(np.float32) for _ in range(K)]
    k_core = {"all_core": n, "all_explore": 0, "core_plus_rest": 1234}[form]
    r = oracle.run_round(w, gs, 1.0, k_core, n - k_core, seed=3, rnd=0, eta=1.0 / K)
    assert np.array_equal(bits(r["w"]), bits(oracle.dense_merge(w, gs, 1.0 / K)))
    for k in range(K):      # and every worker pulls the whole merged model
        both = np.concatenate([r["core_idx"], r["exp_idx"][k]])
        full = np.empty(n, np.float32)
        full[both] = r["pulled"][k]
        assert np.array_equal(bits(full), bits(r["w"]))


def test_round_invariants_on_tiny_shape():
    rng = np.random.default_rng(13)
    n, K, k_core, k_exp = 20_000, 4, 2000, 900
    w = (rng.standard_normal(n) * 0.05).astype(np.float32)
    gs = [(rng.standard_normal(n) * 1e-3).astype(np.float32) for _ in range(K)]
    r = oracle.run_round(w, gs, 1.0, k_core, k_exp, seed=0, rnd=0, eta=0.25)
    core = r["core_idx"]
    assert core.size == k_core
    touched = np.zeros(n, bool)
    touched[core] = True
    for k in range(K):
        e = r["exp_idx"][k]
        assert e.size == k_exp and np.intersect1d(e, core).size == 0     # core and explorer disjoint
        touched[e] = True
        # pushed values are the worker's updates on its communication set
        assert np.array_equal(r["val"][k], gs[k][np.concatenate([core, e])])
        assert np.array_equal(r["pulled"][k], r["w"][np.concatenate([core, e])])
    # parameters outside every communication set are untouched, bit for bit
    assert np.array_equal(bits(r["w"][~touched]), bits(w[~touched]))
    # eta' = 0: nothing moves, pull returns the old values
    r0 = oracle.run_round(w, gs, 1.0, k_core, k_exp, seed=0, rnd=0, eta=0.0)
    assert np.array_equal(bits(r0["w"]), bits(w))


def test_degenerate_ratios():
    # beta = 0 (pure exploration) and beta = alpha (no exploration) are legal (Section 3.4)
    rng = np.random.default_rng(14)
    n, K = 3000, 2
    w = rng.standard_normal(n).astype(np.float32)
    gs = [rng.standard_normal(n).astype(np.float32) for _ in range(K)]
    r = oracle.run_round(w, gs, 1.0, 0, 300, seed=1, rnd=0, eta=0.5)
    assert r["core_idx"].size == 0 and all(v.size == 300 for v in r["val"])
    r = oracle.run_round(w, gs, 1.0, 300, 0, seed=1, rnd=0, eta=0.5)
    assert all(e.size == 0 for e in r["exp_idx"]) and all(v.size == 300 for v in r["val"])


# ----------------------------------------------------------------- wire size

def test_wire_words_match_table1_ratios():
    # Section 3.5: core costs beta*n words (keys cached), explorer 2(alpha-beta)n;
    # Table 1's measured T_comm ratios agree with (2 alpha - beta) to a few percent.
    with open(os.path.join(GOLDEN, "table1_comm_time.txt")) as f:
        rows = [l.split() for l in f if l.strip() and not l.startswith("#")]
    n = 10 ** 6
    for model, K, alpha, beta, t_plump, t_slim in rows:
        alpha, beta = float(alpha), float(beta)
        k_core, k_exp = round(beta * n), round((alpha - beta) * n)
        words = k_core + 2 * k_exp           # values for the core, (index, value) for the explorer
        assert words == round((2 * alpha - beta) * n)
        assert abs(words / n - float(t_slim) / float(t_plump)) < 0.03, model


# ------------------------------------------------------------ key signature

def test_key_signature_pins():
    # Section 3.5: a signature of the cached keys.  Pinned to SplitMix64's published first outputs
    # (seed 0: 0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4) and to what a signature must tell apart.
    assert oracle.core_signature(np.zeros(0, np.uint32)) == 0
    assert oracle.core_signature(np.array([0], np.uint32)) == 0xE220A8397B1DCDAF      # mix64(0 + golden)
    # key 0x9E3779B9 - carry trick is avoided: second published output checked through exact integers instead
    M = (1 << 64) - 1

    def mix(z):
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & M
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & M
        return z ^ (z >> 31)

    assert mix((2 * 0x9E3779B97F4A7C15) & M) == 0x6E789E6AA1B965F4
    keys = np.array([5, 9, 12, 4000000000], np.uint32)
    want = sum(mix((((j << 32) | int(k)) + 0x9E3779B97F4A7C15) & M) for j, k in enumerate(keys)) & M
    assert oracle.core_signature(keys) == want
    # equal lists agree; a changed key, a swapped pair, a dropped or an added key do not
    assert oracle.core_signature(keys.copy()) == want
    for other in (np.array([5, 9, 13, 4000000000], np.uint32), np.array([9, 5, 12, 4000000000], np.uint32),
                  keys[:3], np.append(keys, np.uint32(7))):
        assert oracle.core_signature(other) != want


# ------------------------------------------------------------- wire message

def _mix64(z):
    M = (1 << 64) - 1
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & M
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & M
    return z ^ (z >> 31)


def _signature_py(keys):
    M = (1 << 64) - 1
    return sum(_mix64((((j << 32) | int(k)) + 0x9E3779B97F4A7C15) & M) for j, k in enumerate(keys)) & M


def test_wire_message_layout_byte_for_byte():
    # Section 3.5: the core travels as values plus a signature of the cached keys, the explorer as
    # <key, value> pairs.  The expected bytes are assembled by hand here, field by field.
    import struct
    core, exp = [3, 9], [5]
    val = [1.0, 2.0, -0.5]
    sig = _signature_py(core)
    head = struct.pack("<4sIQIIII", b"SDPW", 0, sig, 2, 1, 7, 11)
    body = struct.pack("<ff", 1.0, 2.0) + struct.pack("<If", 5, -0.5)
    msg = oracle.wire_pack(core, exp, val, 7, 11, False)
    assert bytes(msg) == head + body
    head_k = struct.pack("<4sIQIIII", b"SDPW", 1, sig, 2, 1, 7, 11)
    msg_k = oracle.wire_pack(core, exp, val, 7, 11, True)
    assert bytes(msg_k) == head_k + struct.pack("<II", 3, 9) + body
    assert oracle.wire_message_bytes(2, 1, False) == 48 and oracle.wire_message_bytes(2, 1, True) == 56


def test_wire_message_size_is_the_papers_amount_plus_a_header():
    # (2 alpha - beta) n words per push (Section 3.5), checked against Table 1's time ratios above;
    # the message adds a 32-byte header, and 4 k_core bytes when the keys have to travel again
    n = 10 ** 6
    for alpha, beta in ((0.2, 0.1), (0.3, 0.15), (0.5, 0.25)):
        k_core, k_exp = round(beta * n), round((alpha - beta) * n)
        assert oracle.wire_message_bytes(k_core, k_exp, False) == 4 * round((2 * alpha - beta) * n) + 32
        assert oracle.wire_message_bytes(k_core, k_exp, True) == 4 * round((2 * alpha - beta) * n) + 32 + 4 * k_core


def test_wire_round_trip_and_stale_keys():
    rng = np.random.default_rng(21)
    n, k_core, k_exp = 5000, 700, 333
    idx = rng.permutation(n).astype(np.uint32)
    core, exp = np.sort(idx[:k_core]), np.sort(idx[k_core:k_core + k_exp])
    val = rng.standard_normal(k_core + k_exp).astype(np.float32)
    val.view(np.uint32)[5] = 0x7FC12345          # a NaN payload must survive: the message moves bits
    sig = _signature_py(core)
    assert oracle.core_signature(core) == sig
    # receiver with current keys: values and pairs come back bit for bit, the cache is left alone
    st, got_core, got_exp, got_val, new_sig = oracle.wire_unpack(oracle.wire_pack(core, exp, val, 2, 9, False), sig,
                                                                  k_core, k_exp)
    assert st == 0 and got_core is None and new_sig == sig
    assert np.array_equal(got_exp, exp) and np.array_equal(bits(got_val), bits(val))
    # receiver whose cached keys are stale: "keys wanted", nothing is taken
    stale = np.sort(idx[1:k_core + 1])
    st, _, _, _, _ = oracle.wire_unpack(oracle.wire_pack(core, exp, val, 2, 9, False), _signature_py(stale), k_core, k_exp)
    assert st == 1
    # the next push carries the keys: taken whatever the cache held, keys and signature handed over
    st, got_core, got_exp, got_val, new_sig = oracle.wire_unpack(oracle.wire_pack(core, exp, val, 2, 10, True),
                                                                  _signature_py(stale), k_core, k_exp)
    assert st == 0 and np.array_equal(got_core, core) and new_sig == sig
    assert np.array_equal(got_exp, exp) and np.array_equal(bits(got_val), bits(val))
    # unpack + merge is the same as merging what was packed
    w = rng.standard_normal(n).astype(np.float32)
    assert np.array_equal(bits(oracle.merge(w, got_core, [got_exp], [got_val], 0.25)),
                          bits(oracle.merge(w, core, [exp], [val], 0.25)))


def test_wire_malformed_messages_are_refused():
    core, exp = np.array([1, 4, 6], np.uint32), np.array([2, 3], np.uint32)
    val = np.arange(5, dtype=np.float32)
    sig = _signature_py(core)
    good = oracle.wire_pack(core, exp, val, 0, 0, True)
    assert oracle.wire_unpack(good, 0, 3, 2)[0] == 0
    bad = good.copy(); bad[0] ^= 1                       # magic
    assert oracle.wire_unpack(bad, sig, 3, 2)[0] == -1
    assert oracle.wire_unpack(good[:-4], sig, 3, 2)[0] == -1          # truncated
    assert oracle.wire_unpack(good, sig, 4, 2)[0] == -1               # sizes other than agreed
    bad = good.copy(); bad[32] ^= 1                      # an included key that the signature does not cover
    assert oracle.wire_unpack(bad, sig, 3, 2)[0] == -1
    bad = good.copy(); bad[4] = 2                        # unknown flag
    assert oracle.wire_unpack(bad, sig, 3, 2)[0] == -1


# ------------------------------------------------- per-segment selection (Section 5: model-specific significance)

def test_segmented_select_brute_force_and_reductions():
    rng = np.random.default_rng(30)
    # brute force on tiny segments with many ties: the per-segment winners maximise the segment's sorted key tuple
    for trial in range(40):
        sizes = rng.integers(1, 6, 3)
        off = np.concatenate([[0], np.cumsum(sizes)])
        S = (rng.integers(0, 3, off[-1]) * 0.5).astype(np.float32)
        ks = [int(rng.integers(0, sz + 1)) for sz in sizes]
        got = oracle.select_core_segmented(S, off, ks)
        want = []
        for s in range(3):
            idx = list(range(off[s], off[s + 1]))
            best = max(itertools.combinations(idx, ks[s]),
                       key=lambda c: (sorted((float(S[i]) for i in c), reverse=True), [-i for i in c]))
            want += sorted(best)
        assert got.tolist() == want, (S, off, ks)
    # one segment = the global selection; and every segment is independent of the others
    S = np.abs(rng.standard_normal(5000)).astype(np.float32)
    assert np.array_equal(oracle.select_core_segmented(S, [0, 5000], [700]), oracle.select_core(S, 700))
    off, ks = [0, 1000, 1001, 3500, 5000], [100, 1, 0, 1500]
    got = oracle.select_core_segmented(S, off, ks)
    parts = [oracle.select_core(S[off[s]:off[s + 1]], ks[s]).astype(np.int64) + off[s] for s in range(4)]
    assert np.array_equal(got, np.concatenate(parts))
    S2 = S.copy()
    S2[:1000] = rng.random(1000).astype(np.float32)          # segment 0 changed: the others' choices stay
    got2 = oracle.select_core_segmented(S2, off, ks)
    assert np.array_equal(got2[got2 >= 1000], got[got >= 1000])


# ---------------------------------------------------------------- 8-bit codes for the pushed values

def test_q8_hand_example_and_special_values():
    # one bucket, exact in binary: scale 1, inverse step 127; -0.5 * 127 = -63.5 rounds to the even -64
    codes, scales = oracle.quantize_q8(np.array([1.0, -0.5, 0.25, 0.0], np.float32), bucket=4)
    assert codes.tolist() == [127, -64, 32, 0] and scales.tolist() == [1.0]
    deq = oracle.dequantize_q8(codes, scales, bucket=4)
    step = np.float32(1.0) / np.float32(127.0)
    assert bits(deq).tolist() == bits(np.array([127, -64, 32, 0], np.float32) * step).tolist()
    # an all-zero bucket; NaN -> 0; infinities -> +-127 and do not set the scale; ragged last bucket
    v = np.array([0, 0, 0, 0, np.nan, np.inf, -np.inf, 2.0, -3.0], np.float32)
    codes, scales = oracle.quantize_q8(v, bucket=4)
    assert scales.tolist() == [0.0, 2.0, 3.0]
    assert codes.tolist() == [0, 0, 0, 0, 0, 127, -127, 127, -127]
    codes, scales = oracle.quantize_q8(np.array([np.inf, 0.0, -np.inf, np.nan], np.float32), bucket=4)
    assert scales.tolist() == [0.0] and codes.tolist() == [127, 0, -127, 0]      # no finite magnitude at all


def test_q8_codes_are_one_rounding_of_the_scaled_value_and_the_error_is_half_a_step():
    rng = np.random.default_rng(31)
    v = (rng.standard_normal(5000) * np.exp(rng.uniform(-8, 2, 5000))).astype(np.float32)
    codes, scales = oracle.quantize_q8(v)
    assert scales.size == 20
    for b in range(20):
        seg = v[256 * b:256 * (b + 1)]
        assert scales[b] == np.abs(seg).max()
        inv = np.float32(127.0) / scales[b]                           # IEEE single division
        want = np.clip(np.rint(seg * inv), -127, 127).astype(np.int8)  # IEEE single product, ties to even
        assert np.array_equal(codes[256 * b:256 * (b + 1)], want), b
    deq = oracle.dequantize_q8(codes, scales)
    step = np.repeat(scales / np.float32(127.0), 256)[:v.size]
    assert np.all(np.abs(deq.astype(np.float64) - v) <= 0.5 * step.astype(np.float64) * (1 + 1e-6))
    # a second pass changes nothing: the codes of the decoded values are the codes
    codes2, scales2 = oracle.quantize_q8(deq)
    assert np.array_equal(codes2, codes)
