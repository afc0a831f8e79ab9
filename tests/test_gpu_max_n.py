"""The largest supported vector: n = 2^32 - 1 parameters (indices are uint32).

Checks the 64-bit offset arithmetic of every call at the top of the index range.  The inputs
are mostly zero with a few hundred distinct non-zero values at chosen positions (the very
first and very last indices among them), so the expected core, packed values, merged model
and pulled values follow from the definitions without sorting 4.3 G keys; the explorer is
checked against the CPU oracle.  The one-call round then runs on a model without zeros (so that
its bracketed selection, not the fallback, is what runs): its outputs are compared with the separate
calls on the same inputs and, on the host, with the definitions (threshold by np.partition plus the
tie rule, the oracle's explorers, the oracle's merge and pull on the touched places).
Needs about 110 GB on the device and 70 GB of host memory.
"""
import os

import numpy as np
import pytest
import torch

import oracle

pytestmark = [pytest.mark.gpu, pytest.mark.slow]

N = 2 ** 32 - 1


def _enough_memory() -> bool:
    import psutil
    if psutil.virtual_memory().available < 70 << 30:
        return False
    return torch.cuda.is_available() and torch.cuda.mem_get_info()[0] > (130 << 30)


def test_maximum_vector_length():
    if os.environ.get("SLIMDP_SKIP_LARGE") == "1":
        pytest.skip("SLIMDP_SKIP_LARGE=1")
    if not _enough_memory():
        pytest.skip("needs 70 GB of free host memory and 130 GB of free device memory")
    import paper_1709_09393_b200 as P
    rng = np.random.default_rng(2 ** 32 - 1)
    # 600 marked parameters: both ends of the vector, block / directory boundaries, random places
    special = np.unique(np.concatenate([
        np.array([0, 1, 31, 32, 63, 64, 1023, 1024, N - 1, N - 2, N - 32, N - 33, N - 64, N - 65, N - 1024,
                  2 ** 31 - 1, 2 ** 31, 2 ** 31 + 1], dtype=np.int64),
        rng.integers(0, N, 582, dtype=np.int64)]))
    w_vals = (1.0 + rng.random(special.size)).astype(np.float32)          # distinct with probability ~1
    g_vals = (rng.standard_normal(special.size) * 0.25).astype(np.float32)
    idx_t = torch.from_numpy(special).cuda()

    w = torch.zeros(N, dtype=torch.float32, device="cuda")
    g = torch.zeros(N, dtype=torch.float32, device="cuda")
    w[idx_t] = torch.from_numpy(w_vals).cuda()
    g[idx_t] = torch.from_numpy(g_vals).cuda()

    # score (K = 1): S = |w| + c |g| at the marked places, 0 elsewhere
    scores = torch.empty(N, dtype=torch.float32, device="cuda")
    c = 0.5
    P.slimdp_score(w, [g], c, scores)
    S_special = oracle.score(w_vals, [g_vals], c)
    assert np.array_equal(scores[idx_t].cpu().numpy().view(np.uint32), S_special.view(np.uint32))
    assert int(torch.count_nonzero(scores).item()) == special.size

    # select: the k_core largest of the marked places (all other scores are 0)
    k_core = 400
    order = np.lexsort((special, -S_special.astype(np.float64)))          # score descending, index ascending
    core = np.sort(special[order[:k_core]]).astype(np.uint32)
    core_idx = torch.empty(k_core, dtype=torch.int32, device="cuda")
    aux = torch.empty(P.core_aux_bytes(N), dtype=torch.uint8, device="cuda")
    ws = torch.empty(P.select_workspace_bytes(N), dtype=torch.uint8, device="cuda")
    P.slimdp_select_core(scores, k_core, core_idx, aux, ws)
    P.read_status(ws)
    assert np.array_equal(core_idx.cpu().numpy().view(np.uint32), core)
    # more core members than non-zero scores: ties among the zeros go to the smallest indices
    k_big = special.size + 1000
    big_idx = torch.empty(k_big, dtype=torch.int32, device="cuda")
    P.slimdp_select_core(scores, k_big, big_idx, aux, ws)
    P.read_status(ws)
    zeros_first = np.setdiff1d(np.arange(0, 3000, dtype=np.int64), special)[:1000]
    assert np.array_equal(big_idx.cpu().numpy().view(np.uint32),
                          np.sort(np.concatenate([special, zeros_first])).astype(np.uint32))
    del big_idx, scores, ws
    torch.cuda.empty_cache()

    # explore on the 400-member core (core_aux must be rebuilt for it)
    scores = torch.zeros(N, dtype=torch.float32, device="cuda")
    scores[torch.from_numpy(core.astype(np.int64)).cuda()] = 1.0
    ws = torch.empty(P.select_workspace_bytes(N), dtype=torch.uint8, device="cuda")
    P.slimdp_select_core(scores, k_core, core_idx, aux, ws)
    P.read_status(ws)
    assert np.array_equal(core_idx.cpu().numpy().view(np.uint32), core)
    del scores, ws
    torch.cuda.empty_cache()
    k_exp, K = 100_003, 2
    ews = torch.empty(P.explore_workspace_bytes(N, k_exp, K), dtype=torch.uint8, device="cuda")
    exp_idx = [torch.empty(k_exp, dtype=torch.int32, device="cuda") for _ in range(K)]
    P.slimdp_sample_explore_batched(aux, N, k_core, k_exp, 77, 5, 3, exp_idx, ews)
    P.read_status(ews)
    exps = [oracle.sample_explore(core, N, k_exp, 77, 5 + k, 3) for k in range(K)]
    for k in range(K):
        assert np.array_equal(exp_idx[k].cpu().numpy().view(np.uint32), exps[k])
        assert int(exps[k].max()) > 2 ** 32 - 2 ** 20          # the sample reaches the top of the range

    # exchange with K = 2 workers; worker k's update vector is g scaled by (k + 1) at its own communication set
    eta = 0.5
    deltas, vals_ref = [], []
    for k in range(K):
        d = torch.zeros(N, dtype=torch.float32, device="cuda")
        both = np.concatenate([core, exps[k]]).astype(np.int64)
        dv = ((k + 1) * rng.standard_normal(both.size)).astype(np.float32)
        d[torch.from_numpy(both).cuda()] = torch.from_numpy(dv).cuda()
        deltas.append(d)
        vals_ref.append(dv)                                    # = pack by definition (core first, explorer second)
    m = k_core + k_exp
    val = [torch.empty(m, dtype=torch.float32, device="cuda") for _ in range(K)]
    pulled = [torch.empty(m, dtype=torch.float32, device="cuda") for _ in range(K)]
    P.slimdp_exchange(w, deltas, core_idx, exp_idx, eta, val, pulled)
    # expected merge on the touched places only: a compact copy of the model restricted to them
    touched = np.unique(np.concatenate([core] + exps).astype(np.int64))
    w_small = np.zeros(touched.size, np.float32)
    in_touched = np.isin(special, touched)
    w_small[np.searchsorted(touched, special[in_touched])] = w_vals[in_touched]
    pos = lambda a: np.searchsorted(touched, a.astype(np.int64)).astype(np.uint32)
    merged_small = oracle.merge(w_small, pos(core), [pos(e) for e in exps], vals_ref, eta)
    got_small = w[torch.from_numpy(touched).cuda()].cpu().numpy()
    assert np.array_equal(got_small.view(np.uint32), merged_small.view(np.uint32))
    # nothing else was written: the only other non-zero entries are the marked places outside every set
    assert int(torch.count_nonzero(w).item()) == int(np.count_nonzero(merged_small)) + int((~in_touched).sum())
    for k in range(K):
        assert np.array_equal(val[k].cpu().numpy().view(np.uint32), vals_ref[k].view(np.uint32))
        ref_pull = oracle.pull(merged_small, pos(core), pos(exps[k]))
        assert np.array_equal(pulled[k].cpu().numpy().view(np.uint32), ref_pull.view(np.uint32))

    # the whole round as one call at this length: same bytes as the separate calls on the same inputs
    del val, pulled, exp_idx, ews, aux, core_idx, g
    torch.cuda.empty_cache()
    w.uniform_(-1.0, 1.0)      # a model without the zeros, so that the selection's bracket holds at this length too
    k_core, k_exp = 30_000_001, 40_000_003      # 0.7 % core, ~1 % explorers
    m = k_core + k_exp

    def buffers():
        return dict(core=torch.empty(k_core, dtype=torch.int32, device="cuda"),
                    aux=torch.empty(P.core_aux_bytes(N), dtype=torch.uint8, device="cuda"),
                    exp=[torch.empty(k_exp, dtype=torch.int32, device="cuda") for _ in range(K)],
                    val=[torch.empty(m, dtype=torch.float32, device="cuda") for _ in range(K)],
                    pulled=[torch.empty(m, dtype=torch.float32, device="cuda") for _ in range(K)])

    sel_ws = torch.empty(P.select_workspace_bytes(N), dtype=torch.uint8, device="cuda")
    exp_ws = torch.empty(P.explore_workspace_bytes(N, k_exp, K), dtype=torch.uint8, device="cuda")
    scores = torch.empty(N, dtype=torch.float32, device="cuda")
    a, b = buffers(), buffers()
    w0 = w.cpu().numpy()                                           # the model before the round (host copy)
    w_a = w.clone()
    P.slimdp_score(w_a, deltas, c, scores)
    P.slimdp_select_core(scores, k_core, a["core"], a["aux"], sel_ws)
    P.slimdp_sample_explore_batched(a["aux"], N, k_core, k_exp, 78, 0, 4, a["exp"], exp_ws)
    P.slimdp_exchange(w_a, deltas, a["core"], a["exp"], eta, a["val"], a["pulled"])
    P.read_status(sel_ws)
    P.read_status(exp_ws)
    stage = torch.empty(P.round_stage_bytes(N, K, k_core), dtype=torch.uint8, device="cuda")
    assert stage.numel() > 0
    P.slimdp_round(w, deltas, c, 78, 4, eta, scores, b["core"], b["aux"], b["exp"], b["val"], b["pulled"], sel_ws,
                   exp_ws, stage)
    P.read_status(sel_ws)
    P.read_status(exp_ws)
    assert torch.equal(a["core"], b["core"])
    assert torch.equal(w_a.view(torch.int32), w.view(torch.int32))
    for k in range(K):
        assert torch.equal(a["exp"][k], b["exp"][k])
        assert torch.equal(a["val"][k].view(torch.int32), b["val"][k].view(torch.int32))
        assert torch.equal(a["pulled"][k].view(torch.int32), b["pulled"][k].view(torch.int32))
    del a, w_a, scores, sel_ws, exp_ws, stage
    torch.cuda.empty_cache()

    # ... and the one-call round against the definitions, evaluated on the host without the library:
    # the updates are zero outside a few hundred thousand places, so S = |w| there (Eq. 1 with g = 0) and
    # the oracle scores the rest; the core is the threshold (k-th largest key) plus the tie rule.
    nz = np.unique(np.concatenate([np.concatenate([core, e]).astype(np.int64) for e in exps]))
    nz_t = torch.from_numpy(nz).cuda()
    d_nz = [d[nz_t].cpu().numpy() for d in deltas]                 # the updates where they are not zero
    assert all(int(torch.count_nonzero(d).item()) <= nz.size for d in deltas)
    S = np.abs(w0)
    S[nz] = oracle.score(w0[nz], d_nz, c)
    keys = S.view(np.uint32)
    part = keys.copy()
    part.partition(N - k_core)
    T = part[N - k_core]                                           # the k_core-th largest key
    del part
    greater = np.flatnonzero(keys > T)
    equal = np.flatnonzero(keys == T)
    del S, keys
    core_ref = np.sort(np.concatenate([greater, equal[:k_core - greater.size]])).astype(np.uint32)
    del greater, equal
    assert core_ref.size == k_core
    assert np.array_equal(b["core"].cpu().numpy().view(np.uint32), core_ref)
    exps_ref = [oracle.sample_explore(core_ref, N, k_exp, 78, k, 4) for k in range(K)]
    for k in range(K):
        assert np.array_equal(b["exp"][k].cpu().numpy().view(np.uint32), exps_ref[k]), k
    # pack by definition: the update's value where it has one, zero elsewhere
    vals_ref = []
    for k in range(K):
        both = np.concatenate([core_ref, exps_ref[k]]).astype(np.int64)
        at = np.minimum(np.searchsorted(nz, both), nz.size - 1)
        vals_ref.append(np.where(nz[at] == both, d_nz[k][at], np.float32(0.0)).astype(np.float32))
        assert np.array_equal(b["val"][k].cpu().numpy().view(np.uint32), vals_ref[k].view(np.uint32)), k
    # merge and pull on the touched places (a compact copy of the model restricted to them) ...
    touched = np.unique(np.concatenate([core_ref] + exps_ref).astype(np.int64))
    pos = lambda x: np.searchsorted(touched, x.astype(np.int64)).astype(np.uint32)
    merged_small = oracle.merge(w0[touched], pos(core_ref), [pos(e) for e in exps_ref], vals_ref, eta)
    w1 = w.cpu().numpy()
    assert np.array_equal(w1[touched].view(np.uint32), merged_small.view(np.uint32))
    for k in range(K):
        ref_pull = oracle.pull(merged_small, pos(core_ref), pos(exps_ref[k]))
        assert np.array_equal(b["pulled"][k].cpu().numpy().view(np.uint32), ref_pull.view(np.uint32)), k
    # ... and nothing else was written
    changed = np.flatnonzero(w1.view(np.uint32) != w0.view(np.uint32))
    assert np.isin(changed, touched, assume_unique=True).all()
