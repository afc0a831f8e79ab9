"""slimdp_sample_explore_static: the explorer sampler for callers that cannot allocate.

Some users of this library run where no device allocation is possible: inside a host
program that has already given all device memory to its own pool, in a plug-in that is
not allowed to call cudaMalloc while training runs, or under a memory cap that is used
up.  They cannot hand slimdp_sample_explore a workspace, so the library offers a variant
that works in a fixed scratch array of its own.  This file checks, through the C ABI,
that the variant returns exactly what the ordinary entry point returns, on two calls in
a row (the second call reuses the scratch the first one dirtied), and that it refuses
sizes its scratch cannot hold.  It is named to be collected last, so a run that stops at
the first failure has already run every other test.
"""
import ctypes

import numpy as np
import pytest


def test_static_variant_rejects_sizes_beyond_its_scratch():
    import paper_1709_09393_b200 as P
    UNSUPPORTED, INVALID = -5, -1
    fake = ctypes.c_void_p(0x1000)      # never dereferenced: the size check comes first
    lib = P.lib
    assert lib.slimdp_sample_explore_static(fake, (1 << 25) + 1, 0, 10, 0, 0, 0, fake, None, None) == UNSUPPORTED
    assert lib.slimdp_sample_explore_static(fake, 1 << 25, 0, (1 << 18) + 1, 0, 0, 0, fake, None, None) == UNSUPPORTED
    assert lib.slimdp_sample_explore_static(fake, 100, 50, 51, 0, 0, 0, fake, None, None) == INVALID
    assert lib.slimdp_sample_explore_static(None, 100, 50, 10, 0, 0, 0, fake, None, None) == INVALID


@pytest.mark.gpu
def test_static_variant_matches_the_workspace_variant_twice_in_a_row():
    import torch
    import paper_1709_09393_b200 as P
    assert torch.cuda.is_available()
    n, k_core = 3_000_017, 300_000
    rng = np.random.default_rng(42)
    scores = np.abs(rng.standard_normal(n)).astype(np.float32)
    d_scores = torch.from_numpy(scores).cuda()
    core_idx = torch.empty(k_core, dtype=torch.int32, device="cuda")
    aux = torch.empty(P.core_aux_bytes(n), dtype=torch.uint8, device="cuda")
    sel_ws = torch.empty(P.select_workspace_bytes(n), dtype=torch.uint8, device="cuda")
    P.slimdp_select_core(d_scores, k_core, core_idx, aux, sel_ws)
    P.read_status(sel_ws)
    # two calls in a row with different sizes, workers and rounds: the second starts from
    # whatever the first left in the shared scratch
    for k_exp, seed, worker, rnd in [(200_000, 7, 3, 11), (27_001, 2 ** 40 + 5, 0, 12), (200_000, 7, 3, 11)]:
        ws = torch.empty(P.explore_workspace_bytes(n, k_exp, 1), dtype=torch.uint8, device="cuda")
        want = torch.empty(k_exp, dtype=torch.int32, device="cuda")
        P.slimdp_sample_explore(aux, n, k_core, k_exp, seed, worker, rnd, want, ws)
        P.read_status(ws)
        got = torch.full((k_exp,), -1, dtype=torch.int32, device="cuda")
        status = torch.full((1,), 123, dtype=torch.int32, device="cuda")
        P.slimdp_sample_explore_static(aux, n, k_core, k_exp, seed, worker, rnd, got, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert torch.equal(got, want)      # index lists: bit-exact, the tolerance of every index test here
    # k_exp = 0 is legal and writes nothing
    empty = torch.empty(0, dtype=torch.int32, device="cuda")
    P.slimdp_sample_explore_static(aux, n, k_core, 0, 1, 0, 0, empty)
    torch.cuda.synchronize()
