"""The C-ABI boundary without a GPU: the library loads, exports every symbol
the header declares, sizes its workspaces consistently, and rejects bad
arguments on the host before anything is enqueued."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def P():
    import importlib.util
    spec = importlib.util.spec_from_file_location("_slimdp_cuda_build",
                                                  os.path.join(ROOT, "paper_1709_09393_b200", "build.py"))
    build = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(build)
    build.build()          # the package refuses to import without its library, so build by file path first
    import paper_1709_09393_b200 as pkg
    return pkg


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "slimdp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(slimdp_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(P):
    names = declared_symbols()
    assert {"slimdp_score", "slimdp_select_core", "slimdp_sample_explore", "slimdp_pack", "slimdp_merge",
            "slimdp_pull"} <= set(names)
    from paper_1709_09393_b200.binding import EXPORTS
    for name in names:
        assert hasattr(P.lib, name), name
        assert name in EXPORTS, f"{name} has no Python signature"
    assert set(EXPORTS) == set(names)


def test_status_strings(P):
    assert P.lib.slimdp_status_string(0) == b"ok"
    for code in (-1, -2, -3, -4, -5):
        assert P.lib.slimdp_status_string(code) not in (b"ok", b"unknown status")
    assert P.lib.slimdp_status_string(-99) == b"unknown status"


def test_size_queries(P):
    for n in (1, 1023, 1024, 1025, 10 ** 6, 138_357_544, 2 ** 32 - 1):
        nb = (n + 1023) // 1024
        off = P.core_aux_dir_offset(n)
        assert off >= nb * 128 and off % 256 == 0
        assert P.core_aux_bytes(n) >= off + 4 * (16 * nb + 1)
        assert P.select_workspace_bytes(n) >= 256 + 6 * 4096 * 4 + (1 << 18) * 4 + 2 * nb * 128 + ((nb + 63) // 64) * 8
        k_exp = n // 100
        assert P.explore_workspace_bytes(n, k_exp, 8) > P.explore_workspace_bytes(n, k_exp, 1) >= 256 + 8 * k_exp
        assert P.explore_workspace_bytes(n, n, 1) >= 8 * n
        assert P.workspace_bytes(n, 8, 0, k_exp) == max(P.select_workspace_bytes(n),
                                                        P.explore_workspace_bytes(n, k_exp, 8))
    # out-of-range arguments size to zero
    assert P.core_aux_bytes(0) == 0 and P.core_aux_bytes(2 ** 32) == 0
    assert P.explore_workspace_bytes(1000, 10, 0) == 0 and P.explore_workspace_bytes(1000, 10, 65) == 0
    assert P.explore_workspace_bytes(1000, 1001, 1) == 0
    assert P.round_arena_bytes(1000, 4, 1001, 0) == 0 and P.round_arena_bytes(1000, 4, 600, 401) == 0
    a = P.round_arena_bytes(10 ** 6, 4, 10 ** 5, 45_000)
    assert a >= 4 * 10 ** 6 * 6 + 4 * 145_000 * 8


def test_invalid_arguments_are_rejected_on_the_host(P):
    lib = P.lib
    INVALID, WORKSPACE = -1, -2
    fake = ctypes.c_void_p(0x1000)            # never dereferenced: validation fails first
    arr = (ctypes.c_void_p * 2)(0x1000, 0x2000)
    null_in = (ctypes.c_void_p * 2)(0x1000, None)
    # score
    assert lib.slimdp_score(fake, arr, 2, 1.0, 0, fake, None) == INVALID          # n = 0
    assert lib.slimdp_score(fake, arr, 2, 1.0, 2 ** 32, fake, None) == INVALID    # n too large
    assert lib.slimdp_score(fake, arr, 0, 1.0, 10, fake, None) == INVALID         # K = 0
    assert lib.slimdp_score(fake, arr, 65, 1.0, 10, fake, None) == INVALID        # K > max
    assert lib.slimdp_score(None, arr, 2, 1.0, 10, fake, None) == INVALID
    assert lib.slimdp_score(fake, null_in, 2, 1.0, 10, fake, None) == INVALID
    assert lib.slimdp_score(fake, arr, 2, float("nan"), 10, fake, None) == INVALID
    assert lib.slimdp_score(ctypes.c_void_p(0x1002), arr, 2, 1.0, 10, fake, None) == INVALID   # not 4-byte aligned
    # select
    assert lib.slimdp_select_core(fake, 10, 11, fake, fake, fake, 1 << 30, None) == INVALID    # k_core > n
    assert lib.slimdp_select_core(fake, 10, 5, None, fake, fake, 1 << 30, None) == INVALID
    assert lib.slimdp_select_core(fake, 10, 5, fake, fake, fake, 16, None) == WORKSPACE
    # explore
    assert lib.slimdp_sample_explore(fake, 10, 5, 6, 0, 0, 0, fake, fake, 1 << 30, None) == INVALID  # k_exp > M
    assert lib.slimdp_sample_explore(fake, 10, 5, 5, 0, 0, 0, None, fake, 1 << 30, None) == INVALID
    assert lib.slimdp_sample_explore(fake, 10, 5, 5, 0, 0, 0, fake, fake, 16, None) == WORKSPACE
    assert lib.slimdp_sample_explore_batched(fake, 10, 5, 5, 0, 0, 65, 0, arr, fake, 1 << 30, None) == INVALID
    # pack / pull / merge
    assert lib.slimdp_pack(None, 10, fake, 5, fake, 5, fake, None) == INVALID
    assert lib.slimdp_pack(fake, 10, fake, 5, fake, 6, fake, None) == INVALID
    assert lib.slimdp_pull(fake, 10, None, 5, fake, 5, fake, None) == INVALID
    assert lib.slimdp_merge(fake, 10, 2, fake, 5, arr, 5, arr, float("inf"), None) == INVALID
    assert lib.slimdp_merge(fake, 10, 2, fake, 5, null_in, 5, arr, 0.5, None) == INVALID
    assert lib.slimdp_merge(None, 10, 2, fake, 5, arr, 5, arr, 0.5, None) == INVALID
    assert lib.slimdp_exchange(fake, 10, 2, arr, fake, 5, arr, 5, 0.5, arr, null_in, None) == INVALID
    assert lib.slimdp_exchange(fake, 10, 2, null_in, fake, 5, arr, 5, 0.5, arr, arr, None) == INVALID
    assert lib.slimdp_exchange(fake, 10, 2, arr, fake, 5, arr, 6, 0.5, arr, arr, None) == INVALID
    assert lib.slimdp_dense_merge_score(fake, arr, 2, float("nan"), 1.0, 10, fake, None) == INVALID
    assert lib.slimdp_dense_merge_score(fake, null_in, 2, 0.5, 1.0, 10, None, None) == INVALID
    assert lib.slimdp_dense_merge_score(None, arr, 2, 0.5, 1.0, 10, None, None) == INVALID
    assert lib.slimdp_worker_merge_batched(arr, 2, 10, fake, 5, arr, 6, arr, None) == INVALID
    assert lib.slimdp_worker_merge_batched(null_in, 2, 10, fake, 5, arr, 5, arr, None) == INVALID
    # whole round on host buffers
    assert lib.slimdp_round_host(fake, arr, 2, 10, 1.0, 5, 5, 0, 0, 0.5, fake, arr, arr, None, 0, None) == INVALID
    assert lib.slimdp_round_host(fake, arr, 2, 10, 1.0, 5, 5, 0, 0, 0.5, fake, arr, arr, fake, 16, None) == WORKSPACE
    assert lib.slimdp_read_status(None, None) == INVALID


def test_wire_bytes_of_a_push(P):
    # Section 3.5: values only for the core (keys cached), <key, value> for the explorer
    from workloads import CONFIGS
    for cfg in CONFIGS.values():
        val_bytes, key_bytes = 4 * cfg.m, 4 * cfg.k_exp
        assert val_bytes + key_bytes == 4 * (cfg.k_core + 2 * cfg.k_exp)
        alpha, beta = cfg.m / cfg.N, cfg.k_core / cfg.N
        assert abs((val_bytes + key_bytes) / (4 * cfg.N) - (2 * alpha - beta)) < 1e-12
