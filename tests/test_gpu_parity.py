"""GPU parity: every C-ABI call against the CPU oracle, element by element,
on the same seeded inputs.  Integer results (indices, bitmaps) and all fp32
results (scores, packed values, merged model, pulled values) must match bit
for bit: both sides use the same operation order (fp32 left-to-right worker
sum, one fused multiply-add), so the tolerance is 0 ULP.
"""
import numpy as np
import pytest
import torch

import oracle
from workloads import CONFIGS, all_inputs, scaled_config

pytestmark = pytest.mark.gpu

DIR_STRIDE = 64      # parameters per directory entry of core_aux (SLIMDP_DIR_STRIDE)


@pytest.fixture(scope="module")
def P():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    import paper_1709_09393_b200 as pkg
    return pkg


def dev(a: np.ndarray) -> torch.Tensor:
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint32:
        a = a.view(np.int32)
    return torch.from_numpy(a).cuda()


def host_u32(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy().view(np.uint32)


def host_bits(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy().view(np.uint32)


def bits(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)


def expected_aux(P, core: np.ndarray, n: int):
    """core_aux by its definition: bitmap of the core, non-core counts before each 64-parameter group."""
    nb = (n + 1023) // 1024
    member = np.zeros(nb * 1024, np.uint8)
    member[core] = 1
    words = np.packbits(member.reshape(-1, 8), axis=1, bitorder="little").reshape(-1).view(np.uint32)
    nd = nb * (1024 // DIR_STRIDE)
    per_group = member.reshape(nd, DIR_STRIDE).sum(axis=1, dtype=np.int64)
    directory = np.zeros(nd + 1, np.int64)
    directory[1:] = np.cumsum(DIR_STRIDE - per_group)       # 64 d minus the core members below 64 d
    directory[nd] = n - core.size
    return words, directory.astype(np.uint32)


def gpu_select(P, S: np.ndarray, k: int):
    n = S.size
    scores = dev(S.astype(np.float32, copy=False))
    core_idx = torch.empty(k, dtype=torch.int32, device="cuda")
    aux = torch.empty(P.core_aux_bytes(n), dtype=torch.uint8, device="cuda")
    ws = torch.empty(P.select_workspace_bytes(n), dtype=torch.uint8, device="cuda")
    P.slimdp_select_core(scores, k, core_idx, aux, ws)
    P.read_status(ws)
    return core_idx, aux


def check_aux(P, aux: torch.Tensor, core: np.ndarray, n: int):
    nb = (n + 1023) // 1024
    raw = aux.cpu().numpy()
    words, directory = expected_aux(P, core, n)
    assert np.array_equal(raw[:nb * 128].view(np.uint32), words)
    off = P.core_aux_dir_offset(n)
    assert np.array_equal(raw[off:off + 4 * directory.size].view(np.uint32), directory)


# --------------------------------------------------------------------- score

@pytest.mark.parametrize("n", [1, 3, 4, 5, 31, 1023, 1025, 100_007])
@pytest.mark.parametrize("K", [1, 2, 3, 4, 8, 16, 17, 64])
def test_score_parity(P, n, K):
    rng = np.random.default_rng(n * 131 + K)
    w = (rng.standard_normal(n) * 0.05).astype(np.float32)
    gs = [(rng.standard_normal(n) * 1e-3).astype(np.float32) for _ in range(K)]
    if n >= 31:
        w[:8] = [np.inf, -np.inf, np.nan, 0.0, -0.0, 1e-42, -1e-45, 3e38]
        gs[0][:8] = [0.0, 1.0, 0.0, np.nan, -0.0, 1e-44, 1e-45, 3e38]
    c = 0.73
    out = torch.empty(n, dtype=torch.float32, device="cuda")
    P.slimdp_score(dev(w), [dev(g) for g in gs], c, out)
    assert np.array_equal(host_bits(out), bits(oracle.score(w, gs, c)))


def test_score_unaligned_views(P):
    n, K = 10_001, 3
    rng = np.random.default_rng(5)
    w = rng.standard_normal(n + 3).astype(np.float32)
    gs = [rng.standard_normal(n + 3).astype(np.float32) for _ in range(K)]
    dw, dg = dev(w), [dev(g) for g in gs]
    out = torch.zeros(n + 3, dtype=torch.float32, device="cuda")
    # every buffer starts 4, 8 or 12 bytes past a 16-byte boundary
    P.slimdp_score(dw[1:n + 1], [dg[0][2:n + 2], dg[1][3:n + 3], dg[2][1:n + 1]], 1.0, out[3:n + 3])
    exp = oracle.score(w[1:n + 1], [gs[0][2:n + 2], gs[1][3:n + 3], gs[2][1:n + 1]], 1.0)
    got = out.cpu().numpy()
    assert np.array_equal(got[3:].view(np.uint32), bits(exp)) and np.all(got[:3] == 0)


@pytest.mark.parametrize("shift", [1, 2, 3])
def test_score_views_with_one_common_misalignment(P, shift):
    # slices of larger allocations that all start `shift` floats past a 16-byte boundary: the vectorised
    # kernel runs after the first 4 - shift parameters; the bytes around the outputs stay untouched
    n, K = 100_003, 4
    rng = np.random.default_rng(50 + shift)
    w = rng.standard_normal(n + 8).astype(np.float32)
    gs = [rng.standard_normal(n + 8).astype(np.float32) for _ in range(K)]
    dw, dg = dev(w), [dev(g) for g in gs]
    out = torch.zeros(n + 8, dtype=torch.float32, device="cuda")
    P.slimdp_score(dw[shift:shift + n], [g[shift:shift + n] for g in dg], 0.75, out[shift:shift + n])
    exp = oracle.score(w[shift:shift + n], [g[shift:shift + n] for g in gs], 0.75)
    got = out.cpu().numpy()
    assert np.array_equal(got[shift:shift + n].view(np.uint32), bits(exp))
    assert np.all(got[:shift] == 0) and np.all(got[shift + n:] == 0)


def test_index_buffers_need_only_four_byte_alignment(P):
    # core_idx / exp_idx that start 4 bytes past a 16-byte boundary go through select, explore and the exchange
    cfg = CONFIGS["tiny"]
    w, gs = all_inputs(cfg)
    ref = oracle.run_round(w, gs, cfg.c, cfg.k_core, cfg.k_exp, cfg.seed, 3, cfg.eta)
    n, K = cfg.N, cfg.K
    d_w, d_gs = dev(w), [dev(g) for g in gs]
    scores = torch.empty(n, dtype=torch.float32, device="cuda")
    core_store = torch.empty(cfg.k_core + 1, dtype=torch.int32, device="cuda")
    core_idx = core_store[1:]
    exp_store = [torch.empty(cfg.k_exp + 3, dtype=torch.int32, device="cuda") for _ in range(K)]
    exp_idx = [e[3:] for e in exp_store]
    assert core_idx.data_ptr() % 16 == 4 and exp_idx[0].data_ptr() % 16 == 12
    aux = torch.empty(P.core_aux_bytes(n), dtype=torch.uint8, device="cuda")
    ws = torch.empty(P.workspace_bytes(n, K, cfg.k_core, cfg.k_exp), dtype=torch.uint8, device="cuda")
    val = [torch.empty(cfg.m, dtype=torch.float32, device="cuda") for _ in range(K)]
    pulled = [torch.empty(cfg.m, dtype=torch.float32, device="cuda") for _ in range(K)]
    P.slimdp_score(d_w, d_gs, cfg.c, scores)
    P.slimdp_select_core(scores, cfg.k_core, core_idx, aux, ws)
    P.read_status(ws)
    P.slimdp_sample_explore_batched(aux, n, cfg.k_core, cfg.k_exp, cfg.seed, 0, 3, exp_idx, ws)
    P.read_status(ws)
    P.slimdp_exchange(d_w, d_gs, core_idx, exp_idx, cfg.eta, val, pulled)
    assert np.array_equal(host_u32(core_idx), ref["core_idx"])
    for k in range(K):
        assert np.array_equal(host_u32(exp_idx[k]), ref["exp_idx"][k])
        assert np.array_equal(host_bits(val[k]), bits(ref["val"][k]))
        assert np.array_equal(host_bits(pulled[k]), bits(ref["pulled"][k]))
    assert np.array_equal(host_bits(d_w), bits(ref["w"]))


# -------------------------------------------------------------------- select

def _score_patterns(n, rng):
    yield "random", np.abs(rng.standard_normal(n)).astype(np.float32)
    yield "all_equal", np.full(n, 0.25, np.float32)
    yield "increasing", np.arange(n, dtype=np.float32)
    yield "decreasing", np.arange(n, dtype=np.float32)[::-1].copy()
    yield "two_values", rng.integers(0, 2, n).astype(np.float32)
    yield "coarse_grid", (rng.integers(0, 37, n) * 2.0 ** -7).astype(np.float32)
    s = np.abs(rng.standard_normal(n)).astype(np.float32)
    s[rng.integers(0, n, max(1, n // 50))] = np.inf
    s[rng.integers(0, n, max(1, n // 70))] = np.uint32(0x7FC00000).view(np.float32)
    s[rng.integers(0, n, max(1, n // 30))] = 0.0
    s[rng.integers(0, n, max(1, n // 40))] = 1e-42
    yield "nonfinite_zero_denormal", s
    yield "arbitrary_bit_patterns", rng.integers(0, 2 ** 32, n, dtype=np.uint64).astype(np.uint32).view(np.float32)


@pytest.mark.parametrize("n", [1, 31, 32, 33, 1023, 1024, 1025, 4097, 100_007])
def test_select_parity_small_and_adversarial(P, n):
    rng = np.random.default_rng(n)
    for name, S in _score_patterns(n, rng):
        for k in sorted({0, 1, n // 10, n // 2, n - 1, n} - {-1}):
            if k < 0 or k > n:
                continue
            core_idx, aux = gpu_select(P, S, k)
            exp = oracle.select_core(S, k)
            assert np.array_equal(host_u32(core_idx), exp), (name, n, k)
            check_aux(P, aux, exp, n)


def test_select_large_tie_group_spanning_many_blocks(P):
    n, k = 3_000_000, 1_234_567
    rng = np.random.default_rng(77)
    S = (rng.integers(0, 5, n) * 0.125).astype(np.float32)     # 5 distinct scores, ~600k each
    core_idx, aux = gpu_select(P, S, k)
    exp = oracle.select_core(S, k)
    assert np.array_equal(host_u32(core_idx), exp)
    check_aux(P, aux, exp, n)


def test_select_tie_cut_at_every_offset_of_a_directory_group(P):
    # the emit step admits the first r equal keys in index order: r ends inside the first word of a
    # 64-parameter group, exactly between its two words, inside the second, and at a group's end,
    # in a sparse block (members written directly) and in a dense one (listed through shared memory);
    # 5 blocks: the last pair of blocks has one block only
    n = 5000
    rng = np.random.default_rng(5)
    sparse = np.zeros(n, np.float32)
    sparse[rng.choice(n, 400, replace=False)] = 0.5          # 400 equal keys above zeros
    dense = np.full(n, 0.5, np.float32)                      # every key equal
    tie_idx = np.flatnonzero(sparse)
    for S, ks in ((dense, range(2040, 2120)), (sparse, range(150, 230)), (dense, (n - 65, n - 64, n - 33, n - 32, n - 1, n))):
        for k in ks:
            core_idx, aux = gpu_select(P, S, k)
            exp = oracle.select_core(S, k)
            assert np.array_equal(host_u32(core_idx), exp), k
            check_aux(P, aux, exp, n)
    assert np.array_equal(oracle.select_core(sparse, 400), tie_idx.astype(np.uint32))


@pytest.mark.parametrize("case", ["random", "all_equal", "sampler_fooled", "two_values", "narrow_band"])
def test_select_bracketed_path_and_its_fallback(P, case):
    # n >= 2^21 takes the sampled-bracket path; inputs that defeat the sample or
    # overflow the candidate list must still give the exact core through the full path
    n = (1 << 22) + 77
    rng = np.random.default_rng(len(case))
    if case == "random":
        S = np.abs(rng.standard_normal(n)).astype(np.float32)
    elif case == "all_equal":
        S = np.full(n, 0.5, np.float32)
    elif case == "sampler_fooled":
        S = np.abs(rng.standard_normal(n)).astype(np.float32)
        S[::16] = 100.0                      # the evenly spaced sample sees (almost) only these
    elif case == "two_values":
        S = rng.integers(0, 2, n).astype(np.float32)
    else:
        S = (1.0 + rng.integers(0, 4000, n) * 2.0 ** -23).astype(np.float32)   # 4000 adjacent bit patterns
    for k in (1, 1000, n // 20, n // 3, n - 1, n):
        core_idx, aux = gpu_select(P, S, k)
        exp = oracle.select_core(S, k)
        assert np.array_equal(host_u32(core_idx), exp), (case, k)
        check_aux(P, aux, exp, n)


# ------------------------------------------------------------------- explore

def _gpu_core_aux(P, n, core: np.ndarray):
    """Build core_aux on the device from a chosen core: scores 1 on the core, 0 elsewhere."""
    S = np.zeros(n, np.float32)
    S[core] = 1.0
    core_idx, aux = gpu_select(P, S, core.size)
    assert np.array_equal(host_u32(core_idx), core)
    return aux


@pytest.mark.parametrize("n,k_core,k_exp", [
    (1, 0, 1), (2, 1, 1), (1000, 100, 45), (1000, 0, 1000), (1000, 1000, 0), (1000, 999, 1), (1024, 24, 1000),
    (4097, 1234, 2863), (50_000, 5000, 2250), (100_007, 20_000, 4000), (1_000_003, 300_000, 7000),
])
def test_explore_parity(P, n, k_core, k_exp):
    rng = np.random.default_rng(n + k_core)
    core = np.sort(rng.choice(n, size=k_core, replace=False)).astype(np.uint32)
    aux = _gpu_core_aux(P, n, core)
    ws = torch.empty(P.explore_workspace_bytes(n, k_exp, 1), dtype=torch.uint8, device="cuda")
    for seed, worker, rnd in [(0, 0, 0), (2 ** 40 + 17, 3, 9), (2 ** 64 - 1, 63, 2 ** 32 - 1)]:
        out = torch.empty(k_exp, dtype=torch.int32, device="cuda")
        P.slimdp_sample_explore(aux, n, k_core, k_exp, seed, worker, rnd, out, ws)
        P.read_status(ws)
        assert np.array_equal(host_u32(out), oracle.sample_explore(core, n, k_exp, seed, worker, rnd))


def test_explore_batched_equals_single_calls(P):
    n, k_core, k_exp, K = 300_000, 30_000, 13_500, 16
    rng = np.random.default_rng(3)
    core = np.sort(rng.choice(n, size=k_core, replace=False)).astype(np.uint32)
    aux = _gpu_core_aux(P, n, core)
    ws = torch.empty(P.explore_workspace_bytes(n, k_exp, K), dtype=torch.uint8, device="cuda")
    outs = [torch.empty(k_exp, dtype=torch.int32, device="cuda") for _ in range(K)]
    P.slimdp_sample_explore_batched(aux, n, k_core, k_exp, 9, 5, 2, outs, ws)
    P.read_status(ws)
    for k in range(K):
        assert np.array_equal(host_u32(outs[k]), oracle.sample_explore(core, n, k_exp, 9, 5 + k, 2))


# --------------------------------------------------------- pack / merge / pull

@pytest.mark.parametrize("n,k_core,k_exp,K", [(1, 1, 0, 1), (1, 0, 1, 2), (1000, 0, 0, 2), (1000, 100, 45, 4),
                                               (100_007, 20_000, 4000, 3), (100_007, 0, 100_007, 2),
                                               (100_007, 100_007, 0, 64), (300_001, 100_000, 200_001, 5)])
def test_pack_merge_pull_parity(P, n, k_core, k_exp, K):
    rng = np.random.default_rng(n + K)
    w = rng.standard_normal(n).astype(np.float32)
    ds = [(rng.standard_normal(n) * 0.1).astype(np.float32) for _ in range(K)]
    core = np.sort(rng.choice(n, size=k_core, replace=False)).astype(np.uint32)
    rest = np.setdiff1d(np.arange(n, dtype=np.uint32), core)
    exps = [np.sort(rng.choice(rest, size=k_exp, replace=False)).astype(np.uint32) for _ in range(K)]
    eta = 0.3
    d_core, d_exps, d_ds = dev(core), [dev(e) for e in exps], [dev(d) for d in ds]
    m = k_core + k_exp
    vals = [torch.empty(m, dtype=torch.float32, device="cuda") for _ in range(K)]
    # single-worker calls and the batched call must agree with the oracle
    for k in range(K):
        P.slimdp_pack(d_ds[k], d_core, d_exps[k], vals[k])
    exp_vals = [oracle.pack(ds[k], core, exps[k]) for k in range(K)]
    for k in range(K):
        assert np.array_equal(host_bits(vals[k]), bits(exp_vals[k]))
    vals_b = [torch.zeros(m, dtype=torch.float32, device="cuda") for _ in range(K)]
    P.slimdp_pack_batched(d_ds, d_core, d_exps, vals_b)
    for k in range(K):
        assert np.array_equal(host_bits(vals_b[k]), bits(exp_vals[k]))
    d_w = dev(w)
    P.slimdp_merge(d_w, d_core, d_exps, vals, eta)
    exp_w = oracle.merge(w, core, exps, exp_vals, eta)
    assert np.array_equal(host_bits(d_w), bits(exp_w))
    outs = [torch.empty(m, dtype=torch.float32, device="cuda") for _ in range(K)]
    P.slimdp_pull_batched(d_w, d_core, d_exps, outs)
    one = torch.empty(m, dtype=torch.float32, device="cuda")
    for k in range(K):
        exp_out = oracle.pull(exp_w, core, exps[k])
        assert np.array_equal(host_bits(outs[k]), bits(exp_out))
        P.slimdp_pull(d_w, d_core, d_exps[k], one)
        assert np.array_equal(host_bits(one), bits(exp_out))
    # the fused push + update + pull gives the same three results
    f_w = dev(w)
    f_vals = [torch.zeros(m, dtype=torch.float32, device="cuda") for _ in range(K)]
    f_outs = [torch.zeros(m, dtype=torch.float32, device="cuda") for _ in range(K)]
    P.slimdp_exchange(f_w, d_ds, d_core, d_exps, eta, f_vals, f_outs)
    assert np.array_equal(host_bits(f_w), bits(exp_w))
    for k in range(K):
        assert np.array_equal(host_bits(f_vals[k]), bits(exp_vals[k]))
        assert np.array_equal(host_bits(f_outs[k]), bits(oracle.pull(exp_w, core, exps[k])))


def test_merge_collisions_follow_worker_order(P):
    # every worker's explorer is the same set: each parameter receives K updates in ascending k
    n, K = 50_000, 7
    rng = np.random.default_rng(21)
    w = rng.standard_normal(n).astype(np.float32)
    exp = np.sort(rng.choice(n, size=20_000, replace=False)).astype(np.uint32)
    vals = [rng.standard_normal(exp.size).astype(np.float32) for _ in range(K)]
    none = np.zeros(0, np.uint32)
    d_w = dev(w)
    P.slimdp_merge(d_w, dev(none), [dev(exp)] * K, [dev(v) for v in vals], 1.0 / 3.0)
    fwd = oracle.merge(w, none, [exp] * K, vals, 1.0 / 3.0)
    rev = oracle.merge(w, none, [exp] * K, vals[::-1], 1.0 / 3.0)
    assert not np.array_equal(bits(fwd), bits(rev))        # the order matters for these values
    assert np.array_equal(host_bits(d_w), bits(fwd))
    # same through the fused call: worker k's update vector holds vals[k] on the shared explorer
    ds = []
    for k in range(K):
        d = np.zeros(n, np.float32)
        d[exp] = vals[k]
        ds.append(dev(d))
    f_w = dev(w)
    f_vals = [torch.empty(exp.size, dtype=torch.float32, device="cuda") for _ in range(K)]
    f_outs = [torch.empty(exp.size, dtype=torch.float32, device="cuda") for _ in range(K)]
    P.slimdp_exchange(f_w, ds, dev(none), [dev(exp)] * K, 1.0 / 3.0, f_vals, f_outs)
    assert np.array_equal(host_bits(f_w), bits(fwd))
    for k in range(K):
        assert np.array_equal(host_bits(f_outs[k]), bits(fwd[exp]))


# --------------------------------------------------------------- whole round

def gpu_round(P, w, gs, cfg_c, k_core, k_exp, seed, rnd, eta, fused=True, one_call=False, staging=False):
    n, K = w.size, len(gs)
    buf = P.RoundBuffers(n, K, k_core, k_exp, staging=staging)
    d_w, d_gs = dev(w), [dev(g) for g in gs]
    P.run_round(d_w, d_gs, cfg_c, seed, rnd, eta, buf, fused_exchange=fused, overlapped=one_call)
    P.read_status(buf.select_ws)
    P.read_status(buf.explore_ws)
    return d_w, buf


def assert_round_equal(P, d_w, buf, ref, n, scores=True):
    # bit equality throughout, NaNs included: a NaN result of an update is stored as 0x7FC00000 on both sides
    same = lambda got, want: np.array_equal(got, bits(want))
    if scores:      # slimdp_round keeps its scores in registers: the buffer is scratch there
        assert np.array_equal(host_bits(buf.scores), bits(ref["scores"])), "scores"
    assert np.array_equal(host_u32(buf.core_idx), ref["core_idx"]), "core_idx"
    check_aux(P, buf.core_aux, ref["core_idx"], n)
    for k in range(buf.K):
        assert np.array_equal(host_u32(buf.exp_idx[k]), ref["exp_idx"][k]), f"exp_idx[{k}]"
        assert np.array_equal(host_bits(buf.val[k]), bits(ref["val"][k])), f"val[{k}]"
        assert same(host_bits(buf.pulled[k]), ref["pulled"][k]), f"pulled[{k}]"
    assert same(host_bits(d_w), ref["w"]), "merged model"


def _round_case(P, cfg, rnd=0):
    w, gs = all_inputs(cfg)
    ref = oracle.run_round(w, gs, cfg.c, cfg.k_core, cfg.k_exp, cfg.seed, rnd, cfg.eta)
    # slimdp_exchange, the three separate calls, and the whole round as one call with and without its staging area
    for fused, one_call, staging in ((True, False, False), (False, False, False), (True, True, True), (True, True, False)):
        d_w, buf = gpu_round(P, w, gs, cfg.c, cfg.k_core, cfg.k_exp, cfg.seed, rnd, cfg.eta, fused, one_call, staging)
        assert_round_equal(P, d_w, buf, ref, cfg.N, scores=not one_call)
        del d_w, buf
    return w, gs, ref


@pytest.mark.parametrize("rnd", [0, 1, 2])
def test_round_tiny(P, rnd):
    _round_case(P, CONFIGS["tiny"], rnd)


def test_round_googlenet_shaped(P):
    _round_case(P, CONFIGS["googlenet"])


def test_round_resnet50_tie_stress(P):
    cfg = CONFIGS["resnet50_ties"]
    w, gs, ref = _round_case(P, cfg)
    # the recipe really does produce a large tie group at the threshold
    S = ref["scores"]
    thr = S[ref["core_idx"]].min()
    assert np.count_nonzero(S == thr) > 1000


def test_round_vgg16_shaped_full_size(P):
    _round_case(P, CONFIGS["vgg16"])


@pytest.mark.parametrize("case", ["beta_zero", "beta_equals_alpha", "everything_core", "everything_explored",
                                  "core_plus_rest"])
def test_round_degenerate_ratios(P, case):
    cfg = scaled_config(CONFIGS["googlenet"], 200_003)
    w, gs = all_inputs(cfg)
    n = cfg.N
    k_core, k_exp = {"beta_zero": (0, 30_000), "beta_equals_alpha": (30_000, 0), "everything_core": (n, 0),
                     "everything_explored": (0, n), "core_plus_rest": (12_345, n - 12_345)}[case]
    ref = oracle.run_round(w, gs, 1.0, k_core, k_exp, 5, 1, cfg.eta)
    for one_call in (False, True):
        d_w, buf = gpu_round(P, w, gs, 1.0, k_core, k_exp, 5, 1, cfg.eta, one_call=one_call)
        assert_round_equal(P, d_w, buf, ref, n, scores=not one_call)
        if k_core + k_exp == n:       # 100 % communication ratio: the dense Plump-DP merge
            assert np.array_equal(host_bits(d_w), bits(oracle.dense_merge(w, gs, cfg.eta)))


# slimdp_round folds scoring into the selection's pass over all parameters from n = 2^21 up.
FUSED_N = (1 << 21) + 1061      # several thousand bitmap blocks, a ragged last block, n % 4 == 1


@pytest.mark.parametrize("staging", [True, False])
@pytest.mark.parametrize("case", ["ragged", "k_core_one", "everything_core", "all_scores_equal", "two_values",
                                  "nan_and_inf", "half_core", "wide_bracket"])
def test_round_one_call_fused_cases(P, case, staging):
    cfg = scaled_config(CONFIGS["vgg16"], FUSED_N)
    w, gs = all_inputs(cfg)
    w, gs = w.copy(), [g.copy() for g in gs]
    n, k_core, k_exp = cfg.N, cfg.k_core, cfg.k_exp
    if case == "k_core_one":
        k_core = 1
    elif case == "everything_core":
        k_core, k_exp = n, 0
    elif case == "all_scores_equal":      # the bracket cannot hold: the full path scores into the scratch
        w[:] = 0.25
        for g in gs:
            g[:] = 0.0
    elif case == "two_values":            # threshold inside a tie group of about n / 2 parameters
        w[:] = np.where(np.arange(n) % 2 == 0, np.float32(0.5), np.float32(0.125))
        for g in gs:
            g[:] = 0.0
        k_core = n // 2 + 12_345
        k_exp = 1000
    elif case == "half_core":             # the largest core that is still staged
        k_core, k_exp = n // 2, n // 8
    elif case == "wide_bracket":          # a few huge scores: the bracket spans many octaves (three counting rounds)
        k_core, k_exp = 5, 1000
        w[::50_021] *= np.float32(1e30)
    elif case == "nan_and_inf":
        w[7::1001] = np.nan
        w.view(np.uint32)[9::5003] = 0xFFC12345          # a NaN with a sign and a payload
        gs[0].view(np.uint32)[13::7001] = 0x7F800001     # a signalling NaN in an update
        gs[1][3::2003] = np.inf
        gs[2][5::3001] = -np.inf
        w[11::4001] = np.float32(-0.0)
    ref = oracle.run_round(w, gs, cfg.c, k_core, k_exp, cfg.seed, 2, cfg.eta)
    d_w, buf = gpu_round(P, w, gs, cfg.c, k_core, k_exp, cfg.seed, 2, cfg.eta, one_call=True, staging=staging)
    assert_round_equal(P, d_w, buf, ref, n, scores=False)
    if case == "all_scores_equal":        # and there the scratch does hold the scores
        assert np.array_equal(host_bits(buf.scores), bits(ref["scores"]))


# The pass keeps its loads in a shared-memory ring whose depth follows the number of workers
# (8 stages for K <= 2 down to 2 for K = 12..17); from K = 18 a ring stage no longer fits and the
# register version of the pass runs.  One case per depth, and one on the other side of the limit.
@pytest.mark.parametrize("K", [1, 2, 3, 5, 7, 12, 17, 18, 33])
def test_round_one_call_any_worker_count(P, K):
    n = FUSED_N + 2 * K      # n % 4 in {1, 3}
    rng = np.random.default_rng(1000 + K)
    w = (rng.standard_normal(n) * 0.05).astype(np.float32)
    gs = [(rng.standard_normal(n) * 1e-2).astype(np.float32) for _ in range(K)]
    k_core, k_exp = n // 16, n // 200
    ref = oracle.run_round(w, gs, 1.0, k_core, k_exp, 9, 3, 1.0 / K)
    d_w, buf = gpu_round(P, w, gs, 1.0, k_core, k_exp, 9, 3, 1.0 / K, one_call=True)
    assert_round_equal(P, d_w, buf, ref, n, scores=False)


# In the one-call round the exchange's explorer warps compute the indices from the sorted ranks where
# a warp's parameter range is 1 to 32 groups of 64 parameters, i.e. for explorers of about 0.8 % to 50 % of
# the vector per worker; denser and thinner explorers take the separate index kernels.  One case per
# range size on either side of both limits.
@pytest.mark.parametrize("per_mille", [600, 300, 100, 30, 12, 6, 1])
def test_round_one_call_explorer_densities(P, per_mille):
    K, n = 3, FUSED_N
    rng = np.random.default_rng(per_mille)
    w = (rng.standard_normal(n) * 0.05).astype(np.float32)
    gs = [(rng.standard_normal(n) * 1e-2).astype(np.float32) for _ in range(K)]
    k_core = n // 33
    k_exp = (n - k_core) * per_mille // 1000
    ref = oracle.run_round(w, gs, 1.0, k_core, k_exp, 11, 5, 0.25)
    d_w, buf = gpu_round(P, w, gs, 1.0, k_core, k_exp, 11, 5, 0.25, one_call=True)
    assert_round_equal(P, d_w, buf, ref, n, scores=False)


# Short vectors through the one-call round: a single bitmap block or a few, the last directory groups
# partly or wholly beyond the end of the vector.
@pytest.mark.parametrize("n,k_core,k_exp", [(1, 0, 1), (1, 1, 0), (5, 2, 2), (63, 6, 3), (64, 6, 3), (65, 7, 58),
                                            (100, 10, 3), (1000, 100, 45), (1025, 1, 512), (4097, 400, 200),
                                            (70_001, 3000, 900)])
def test_round_one_call_short_vectors(P, n, k_core, k_exp):
    K = 2
    rng = np.random.default_rng(n)
    w = rng.standard_normal(n).astype(np.float32)
    gs = [(rng.standard_normal(n) * 0.1).astype(np.float32) for _ in range(K)]
    ref = oracle.run_round(w, gs, 0.5, k_core, k_exp, 3, 1, 0.5)
    d_w, buf = gpu_round(P, w, gs, 0.5, k_core, k_exp, 3, 1, 0.5, one_call=True)
    assert_round_equal(P, d_w, buf, ref, n, scores=True)      # below 2^21 parameters the scores are written


def test_round_one_call_any_alignment(P):
    # tensors that start 4 bytes off a 16-byte boundary: the round scores and selects in two steps
    cfg = scaled_config(CONFIGS["vgg16"], FUSED_N)
    w, gs = all_inputs(cfg)
    ref = oracle.run_round(w, gs, cfg.c, cfg.k_core, cfg.k_exp, cfg.seed, 0, cfg.eta)
    n, K = cfg.N, cfg.K
    buf = P.RoundBuffers(n, K, cfg.k_core, cfg.k_exp)
    off = lambda a: torch.cat([torch.zeros(1, dtype=torch.float32), torch.from_numpy(a)]).cuda()[1:]
    d_w, d_gs = off(w), [off(g) for g in gs]
    assert d_w.data_ptr() % 16 == 4
    P.run_round(d_w, d_gs, cfg.c, cfg.seed, 0, cfg.eta, buf, overlapped=True)
    P.read_status(buf.select_ws)
    P.read_status(buf.explore_ws)
    assert_round_equal(P, d_w, buf, ref, n, scores=True)      # unfused: the scores are there


def test_round_one_call_repeats_and_marks(P):
    cfg = scaled_config(CONFIGS["vgg16"], FUSED_N)
    w, gs = all_inputs(cfg)
    d_w, d_gs = dev(w), [dev(g) for g in gs]
    a_w = d_w.clone()
    buf = P.RoundBuffers(cfg.N, cfg.K, cfg.k_core, cfg.k_exp)
    ref_buf = P.RoundBuffers(cfg.N, cfg.K, cfg.k_core, cfg.k_exp)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(); e1.record()
    for rnd in range(3):      # successive rounds on the evolving model, buffers reused
        if rnd == 1:
            P.mark_dominant_kernel(e0, e1)
        P.run_round(d_w, d_gs, cfg.c, cfg.seed, rnd, cfg.eta, buf, overlapped=True)
        P.run_round(a_w, d_gs, cfg.c, cfg.seed, rnd, cfg.eta, ref_buf)
        torch.cuda.synchronize()
        assert torch.equal(d_w.view(torch.int32), a_w.view(torch.int32))
        assert torch.equal(buf.core_idx, ref_buf.core_idx)
        for k in range(cfg.K):
            assert torch.equal(buf.exp_idx[k], ref_buf.exp_idx[k])
            assert torch.equal(buf.pulled[k].view(torch.int32), ref_buf.pulled[k].view(torch.int32))
    assert 0.0 < e0.elapsed_time(e1) < 50.0      # ms: one pass over two million parameters


def test_round_one_call_rejects_overlapping_workspaces(P):
    cfg = CONFIGS["tiny"]
    w, gs = all_inputs(cfg)
    buf = P.RoundBuffers(cfg.N, cfg.K, cfg.k_core, cfg.k_exp)
    both = torch.empty(max(buf.select_ws.numel(), buf.explore_ws.numel()), dtype=torch.uint8, device="cuda")
    with pytest.raises(P.SlimDPError):
        P.slimdp_round(dev(w), [dev(g) for g in gs], cfg.c, cfg.seed, 0, cfg.eta, buf.scores, buf.core_idx,
                       buf.core_aux, buf.exp_idx, buf.val, buf.pulled, both, both)


def test_round_is_deterministic(P):
    cfg = CONFIGS["tiny"]
    w, gs = all_inputs(cfg)
    a_w, a = gpu_round(P, w, gs, cfg.c, cfg.k_core, cfg.k_exp, cfg.seed, 0, cfg.eta)
    b_w, b = gpu_round(P, w, gs, cfg.c, cfg.k_core, cfg.k_exp, cfg.seed, 0, cfg.eta)
    assert torch.equal(a_w, b_w) and torch.equal(a.core_idx, b.core_idx)
    nb = (cfg.N + 1023) // 1024
    off = P.core_aux_dir_offset(cfg.N)
    assert torch.equal(a.core_aux[:nb * 128], b.core_aux[:nb * 128])                      # bitmap
    nd = nb * (1024 // DIR_STRIDE)
    assert torch.equal(a.core_aux[off:off + 4 * (nd + 1)], b.core_aux[off:off + 4 * (nd + 1)])   # directory
    for k in range(cfg.K):
        assert torch.equal(a.exp_idx[k], b.exp_idx[k]) and torch.equal(a.pulled[k], b.pulled[k])


def test_round_on_host_buffers(P):
    cfg = scaled_config(CONFIGS["vgg16"], 3_000_017)
    w, gs = all_inputs(cfg)
    ref = oracle.run_round(w, gs, cfg.c, cfg.k_core, cfg.k_exp, cfg.seed, 0, cfg.eta)
    pin = lambda a: torch.from_numpy(a.view(np.int32) if a.dtype == np.uint32 else a).pin_memory()
    w_h = pin(w.copy())
    g_h = [pin(g) for g in gs]
    core_h = torch.empty(cfg.k_core, dtype=torch.int32).pin_memory()
    exp_h = [torch.empty(cfg.k_exp, dtype=torch.int32).pin_memory() for _ in range(cfg.K)]
    pulled_h = [torch.empty(cfg.m, dtype=torch.float32).pin_memory() for _ in range(cfg.K)]
    arena = torch.empty(P.round_arena_bytes(cfg.N, cfg.K, cfg.k_core, cfg.k_exp), dtype=torch.uint8, device="cuda")
    P.slimdp_round_host(w_h, g_h, cfg.c, cfg.k_core, cfg.k_exp, cfg.seed, 0, cfg.eta, core_h, exp_h, pulled_h, arena)
    assert np.array_equal(w_h.numpy().view(np.uint32), bits(ref["w"]))
    assert np.array_equal(core_h.numpy().view(np.uint32), ref["core_idx"])
    for k in range(cfg.K):
        assert np.array_equal(exp_h[k].numpy().view(np.uint32), ref["exp_idx"][k])
        assert np.array_equal(pulled_h[k].numpy().view(np.uint32), bits(ref["pulled"][k]))


def test_untouched_parameters_keep_their_bits(P):
    cfg = CONFIGS["tiny"]
    w, gs = all_inputs(cfg)
    d_w, buf = gpu_round(P, w, gs, cfg.c, cfg.k_core, cfg.k_exp, cfg.seed, 0, cfg.eta)
    touched = np.zeros(cfg.N, bool)
    touched[host_u32(buf.core_idx)] = True
    for k in range(cfg.K):
        e = host_u32(buf.exp_idx[k])
        assert np.intersect1d(e, host_u32(buf.core_idx)).size == 0
        touched[e] = True
    got = d_w.cpu().numpy()
    assert np.array_equal(got[~touched].view(np.uint32), w[~touched].view(np.uint32))


# ------------------------------------------------------------ key signature

@pytest.mark.parametrize("count", [0, 1, 31, 1000, 100_003, 3_000_001])
def test_core_signature_parity(P, count):
    rng = np.random.default_rng(count)
    keys = np.unique(rng.integers(0, 2 ** 32 - 1, count, dtype=np.uint64)).astype(np.uint32)   # ascending, distinct
    sig = torch.full((1,), -1, dtype=torch.int64, device="cuda")
    P.slimdp_core_signature(dev(keys), sig)
    assert int(sig.cpu().numpy().view(np.uint64)[0]) == oracle.core_signature(keys)
    assert P.wire_bytes(1000, 50) == 4 * 1000 + 8 * 50 + 8


# ---------------------------------------------------------------- wire message (Section 3.5)

def u64_dev(x: int) -> torch.Tensor:
    """A one-element int64 CUDA tensor holding the 64-bit pattern x."""
    return torch.from_numpy(np.array([x], np.uint64).view(np.int64)).cuda()


def u64_host(t: torch.Tensor) -> int:
    return int(t.cpu().numpy().view(np.uint64)[0])


@pytest.mark.parametrize("k_core,k_exp", [(0, 0), (1, 0), (0, 1), (7, 5), (700, 333), (100_003, 40_001)])
def test_wire_pack_and_unpack_match_the_oracle(P, k_core, k_exp):
    rng = np.random.default_rng(100 + k_core)
    n = 3 * (k_core + k_exp) + 10
    idx = rng.permutation(n).astype(np.uint32)
    core, exp = np.sort(idx[:k_core]), np.sort(idx[k_core:k_core + k_exp])
    val = rng.standard_normal(k_core + k_exp).astype(np.float32)
    if val.size:
        val.view(np.uint32)[0] = 0x7FC12345          # the message moves bits
    i32 = lambda a: torch.from_numpy(a.view(np.int32)).cuda()
    d_core, d_exp, d_val = i32(core), i32(exp), dev(val)
    d_sig = torch.zeros(1, dtype=torch.int64, device="cuda")
    P.slimdp_core_signature(d_core, d_sig)
    for with_keys in (False, True):
        want = oracle.wire_pack(core, exp, val, 3, 17, with_keys)
        msg = torch.zeros(P.wire_message_bytes(k_core, k_exp, with_keys), dtype=torch.uint8, device="cuda")
        assert msg.numel() == want.size
        P.slimdp_wire_pack(d_core, d_exp, d_val, d_sig, 3, 17, with_keys, msg)
        assert np.array_equal(msg.cpu().numpy(), want), f"message bytes, with_keys={with_keys}"
        # the receiver: cached keys current / stale
        for stale in (False, True):
            cached = u64_dev(oracle.core_signature(core) ^ (0x55 if stale else 0))
            o_core = torch.full((k_core,), -1, dtype=torch.int32, device="cuda")
            o_exp = torch.full((k_exp,), -1, dtype=torch.int32, device="cuda")
            o_val = torch.full((k_core + k_exp,), 7.0, dtype=torch.float32, device="cuda")
            o_sig = torch.full((1,), -1, dtype=torch.int64, device="cuda")
            status = torch.zeros(4, dtype=torch.int32, device="cuda")
            P.slimdp_wire_unpack(msg, cached, o_core, o_exp, o_val, o_sig, status)
            st = P.wire_read_status(status)
            ref_st, ref_core, ref_exp, ref_val, ref_sig = oracle.wire_unpack(want, u64_host(cached), k_core, k_exp)
            assert st == ref_st
            if st == 0:
                assert np.array_equal(host_u32(o_exp), ref_exp)
                assert np.array_equal(host_bits(o_val), bits(ref_val))
                assert u64_host(o_sig) == ref_sig
                if with_keys:
                    assert np.array_equal(host_u32(o_core), ref_core)
                else:
                    assert bool((o_core == -1).all())
            else:       # keys wanted: nothing was written
                assert st == P.WIRE_KEYS_WANTED and not with_keys and stale
                assert bool((o_exp == -1).all()) and bool((o_val == 7.0).all()) and int(o_sig.item()) == -1


def test_wire_malformed_messages_are_refused_on_the_device(P):
    core, exp = np.array([1, 4, 6], np.uint32), np.array([2, 3], np.uint32)
    val = np.arange(5, dtype=np.float32)
    good = oracle.wire_pack(core, exp, val, 0, 0, True)
    cached = u64_dev(oracle.core_signature(core))

    def verdict(msg_bytes, k_core=3, k_exp=2):
        msg = torch.from_numpy(msg_bytes.copy()).cuda()
        o_core = torch.zeros(k_core, dtype=torch.int32, device="cuda")
        o_exp = torch.zeros(k_exp, dtype=torch.int32, device="cuda")
        o_val = torch.zeros(k_core + k_exp, dtype=torch.float32, device="cuda")
        o_sig = torch.zeros(1, dtype=torch.int64, device="cuda")
        status = torch.zeros(4, dtype=torch.int32, device="cuda")
        P.slimdp_wire_unpack(msg, cached, o_core, o_exp, o_val, o_sig, status)
        return P.wire_read_status(status)

    assert verdict(good) == 0
    for mutate in (lambda m: m.__setitem__(0, m[0] ^ 1), lambda m: m.__setitem__(32, m[32] ^ 1),
                   lambda m: m.__setitem__(4, 2)):
        bad = good.copy()
        mutate(bad)
        with pytest.raises(P.SlimDPError):
            verdict(bad)
    with pytest.raises(P.SlimDPError):
        verdict(good[:-4])
    with pytest.raises(P.SlimDPError):
        verdict(good, k_core=2, k_exp=2)


def test_wire_unpack_feeds_the_merge(P):
    cfg = CONFIGS["tiny"]
    w, gs = all_inputs(cfg)
    ref = oracle.run_round(w, gs, cfg.c, cfg.k_core, cfg.k_exp, cfg.seed, 0, cfg.eta)
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.int32)).cuda()
    d_core = i32(ref["core_idx"])
    d_sig = torch.zeros(1, dtype=torch.int64, device="cuda")
    P.slimdp_core_signature(d_core, d_sig)
    exps, vals = [], []
    for k in range(cfg.K):      # every worker's push goes through a message and is taken apart again
        msg = torch.empty(P.wire_message_bytes(cfg.k_core, cfg.k_exp, False), dtype=torch.uint8, device="cuda")
        P.slimdp_wire_pack(d_core, i32(ref["exp_idx"][k]), dev(ref["val"][k]), d_sig, k, 0, False, msg)
        o_core = torch.empty(cfg.k_core, dtype=torch.int32, device="cuda")
        o_exp = torch.empty(cfg.k_exp, dtype=torch.int32, device="cuda")
        o_val = torch.empty(cfg.m, dtype=torch.float32, device="cuda")
        status = torch.zeros(4, dtype=torch.int32, device="cuda")
        P.slimdp_wire_unpack(msg, d_sig, o_core, o_exp, o_val, d_sig.clone(), status)
        assert P.wire_read_status(status) == 0
        exps.append(o_exp)
        vals.append(o_val)
    d_w = dev(w)
    P.slimdp_merge(d_w, d_core, exps, vals, cfg.eta)
    assert np.array_equal(host_bits(d_w), bits(ref["w"]))


# ------------------------------------------------------------- 8-bit pushed values (Section 2.2, last remark)

@pytest.mark.parametrize("n,k_core,k_exp,K", [(1000, 100, 37, 1), (100_003, 20_000, 5_001, 3), (5000, 0, 700, 2),
                                               (5000, 256, 0, 2), (300_000, 65_536, 30_000, 8)])
def test_q8_pack_and_merge_match_the_oracle(P, n, k_core, k_exp, K):
    rng = np.random.default_rng(n + K)
    idx = rng.permutation(n).astype(np.uint32)
    core = np.sort(idx[:k_core])
    exps = [np.sort(rng.permutation(np.setdiff1d(np.arange(n, dtype=np.uint32), core))[:k_exp]) for _ in range(K)]
    w = rng.standard_normal(n).astype(np.float32)
    ds = [(rng.standard_normal(n) * np.exp(rng.uniform(-6, 1, n))).astype(np.float32) for _ in range(K)]
    ds[0][::97] = 0.0
    if k_core:                                   # non-finite values, and a bucket with nothing but zeros
        ds[0][core[:3]] = [np.nan, np.inf, -np.inf]
        ds[-1][core[:min(256, k_core)]] = 0.0
    m = k_core + k_exp
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.int32)).cuda()
    d_core, d_exps = i32(core), [i32(e) for e in exps]
    codes = [torch.zeros(m, dtype=torch.int8, device="cuda") for _ in range(K)]
    scales = [torch.zeros((m + 255) // 256, dtype=torch.float32, device="cuda") for _ in range(K)]
    P.slimdp_pack_q8_batched([dev(d) for d in ds], d_core, d_exps, codes, scales)
    deq = []
    for k in range(K):
        ref_codes, ref_scales = oracle.quantize_q8(oracle.pack(ds[k], core, exps[k]))
        assert np.array_equal(codes[k].cpu().numpy(), ref_codes), f"codes of worker {k}"
        assert np.array_equal(host_bits(scales[k]), bits(ref_scales)), f"scales of worker {k}"
        deq.append(oracle.dequantize_q8(ref_codes, ref_scales))
    d_w = dev(w)
    P.slimdp_merge_q8(d_w, d_core, d_exps, codes, scales, 1.0 / K)
    assert np.array_equal(host_bits(d_w), bits(oracle.merge(w, core, exps, deq, 1.0 / K)))


# ------------------------------------------------------------- per-layer selection (Section 5)

def _segmented_case(P, S, off, ks):
    n = S.size
    k = int(sum(ks))
    core_idx = torch.empty(k, dtype=torch.int32, device="cuda")
    aux = torch.empty(P.core_aux_bytes(n), dtype=torch.uint8, device="cuda")
    ws = torch.empty(P.select_segmented_workspace_bytes(n, len(ks)), dtype=torch.uint8, device="cuda")
    P.slimdp_select_core_segmented(dev(S), off, ks, core_idx, aux, ws)
    P.read_status(ws)
    ref = oracle.select_core_segmented(S, off, ks)
    assert np.array_equal(host_u32(core_idx), ref)
    check_aux(P, aux, ref, n)


@pytest.mark.parametrize("name", ["googlenet", "resnet50_ties", "vgg16"])
def test_segmented_select_on_the_layer_tables(P, name):
    # the layers of the shaped workloads (biases and batch-norm vectors are segments of their own);
    # every layer keeps the workload's core ratio of its own parameters
    cfg = CONFIGS[name] if name != "vgg16" else scaled_config(CONFIGS["vgg16"], 20_000_003)
    w, gs = all_inputs(cfg)
    S = oracle.score(w, gs, cfg.c)
    off = [0]
    for seg in cfg.segments:
        off.append(off[-1] + seg.size)
    ks = [(off[i + 1] - off[i]) * cfg.core_pct // 100 for i in range(len(off) - 1)]
    _segmented_case(P, S, off, ks)


@pytest.mark.parametrize("case", ["ties", "edges", "one_segment", "bits"])
def test_segmented_select_adversarial(P, case):
    rng = np.random.default_rng(77)
    if case == "ties":            # few distinct scores: thresholds sit in tie groups that cross block and CTA boundaries
        n = 700_001
        S = (rng.integers(0, 8, n) / 8.0).astype(np.float32)
        off = [0, 1, 33, 1024, 1025, 100_000, 100_000, 350_011, n]
        ks = [1, 7, 500, 0, 33_333, 0, 125_000, 200_000]
    elif case == "edges":         # nothing / everything of a segment, empty segments, segments of one parameter
        n = 50_000
        S = np.abs(rng.standard_normal(n)).astype(np.float32)
        off = [0, 0, 10, 11, 2048, 2048, 30_000, n]
        ks = [0, 10, 0, 2037, 0, 1, n - 30_000]
    elif case == "one_segment":   # reduces to the selection over the whole vector
        n = 300_007
        S = np.abs(rng.standard_normal(n)).astype(np.float32)
        off, ks = [0, n], [n // 7]
    else:                          # arbitrary bit patterns
        n = 200_003
        S = rng.integers(0, 2 ** 32, n, dtype=np.uint64).astype(np.uint32).view(np.float32)
        off = [0, 50_000, 50_064, n]
        ks = [25_000, 64, 1]
    _segmented_case(P, S, off, ks)
    if case == "one_segment":
        assert np.array_equal(oracle.select_core_segmented(S, off, ks), oracle.select_core(S, ks[0]))



# ------------------------------------------------------------- round contexts

def test_two_host_threads_run_rounds_on_one_device_at_once(P):
    """Two host threads, each with its own stream, round context and buffers, enqueue rounds on one
    device at the same time; both must leave the oracle's bytes.  A third pair of rounds shares the
    library's default context from two threads (serialised by its lock)."""
    import threading
    cfg = scaled_config(CONFIGS["vgg16"], FUSED_N)
    w, gs = all_inputs(cfg)
    refs, w_ref = [], w
    for t in range(3):                       # three successive rounds on the evolving model
        r = oracle.run_round(w_ref, gs, cfg.c, cfg.k_core, cfg.k_exp, cfg.seed, t, cfg.eta)
        refs.append(r)
        w_ref = r["w"]

    def worker(own_ctx, errors, slot):
        try:
            torch.cuda.set_device(0)
            stream = torch.cuda.Stream()
            ctx = P.RoundContext() if own_ctx else None
            with torch.cuda.stream(stream):
                d_w, d_gs = dev(w), [dev(g) for g in gs]
                buf = P.RoundBuffers(cfg.N, cfg.K, cfg.k_core, cfg.k_exp)
                for t in range(3):
                    P.slimdp_round(d_w, d_gs, cfg.c, cfg.seed, t, cfg.eta, buf.scores, buf.core_idx, buf.core_aux,
                                   buf.exp_idx, buf.val, buf.pulled, buf.select_ws, buf.explore_ws, None, ctx, stream)
                stream.synchronize()
                P.read_status(buf.select_ws, stream)
                P.read_status(buf.explore_ws, stream)
                ok = np.array_equal(host_bits(d_w), bits(refs[2]["w"])) and \
                    np.array_equal(host_u32(buf.core_idx), refs[2]["core_idx"])
                for k in range(cfg.K):
                    ok = ok and np.array_equal(host_u32(buf.exp_idx[k]), refs[2]["exp_idx"][k]) and \
                        np.array_equal(host_bits(buf.pulled[k]), bits(refs[2]["pulled"][k]))
                if not ok:
                    errors.append(f"thread {slot}: results differ from the oracle")
            if ctx is not None:
                ctx.close()
        except Exception as e:          # noqa: BLE001  (reported to the main thread)
            errors.append(f"thread {slot}: {e!r}")

    for own_ctx in (True, False):
        errors = []
        threads = [threading.Thread(target=worker, args=(own_ctx, errors, i)) for i in range(2)]
        for th in threads:
            th.start()
        for th in threads:
            th.join()
        assert not errors, errors
    P.release_default_round_ctx()            # and the default context can be given back and made again
    d_w, buf = gpu_round(P, w, gs, cfg.c, cfg.k_core, cfg.k_exp, cfg.seed, 0, cfg.eta, one_call=True)
    assert np.array_equal(host_bits(d_w), bits(refs[0]["w"]))


def test_rounds_back_to_back_on_a_vector_with_several_tiles_per_cta(P):
    """Six one-call rounds enqueued without a synchronisation in between, on a vector long enough that the
    persistent CTAs of the selection's last kernel walk several tiles each; the model after the last round and
    that round's outputs must be the oracle's."""
    cfg = scaled_config(CONFIGS["vgg16"], 24_000_007)
    w, gs = all_inputs(cfg)
    rounds = 6
    w_ref = w
    for t in range(rounds):
        ref = oracle.run_round(w_ref, gs, cfg.c, cfg.k_core, cfg.k_exp, cfg.seed, t, cfg.eta)
        w_ref = ref["w"]
    d_w, d_gs = dev(w), [dev(g) for g in gs]
    buf = P.RoundBuffers(cfg.N, cfg.K, cfg.k_core, cfg.k_exp)
    for rep in range(3):                 # the whole sequence three times over: races show up as flakiness
        d_w.copy_(torch.from_numpy(w))
        for t in range(rounds):
            P.slimdp_round(d_w, d_gs, cfg.c, cfg.seed, t, cfg.eta, buf.scores, buf.core_idx, buf.core_aux, buf.exp_idx,
                           buf.val, buf.pulled, buf.select_ws, buf.explore_ws)
        P.read_status(buf.select_ws)
        P.read_status(buf.explore_ws)
        assert_round_equal(P, d_w, buf, ref, cfg.N, scores=False)
