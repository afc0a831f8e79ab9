"""Python face of the CPU oracle (test infrastructure, not the product).

Thin numpy wrappers around oracle/slimdp_oracle.cpp, one per step of the
Slim-DP communication round, plus `run_round`, which calls them in the
order of the round.  Only the tests, the smoke check and the benchmark's CPU
baseline leg import this package; the CUDA library never does.
"""
from __future__ import annotations

import ctypes
from typing import Dict, List, Sequence

import numpy as np

from .build import build as _build

_lib = ctypes.CDLL(_build())

_u32p = ctypes.POINTER(ctypes.c_uint32)
_f32p = ctypes.POINTER(ctypes.c_float)
_pp = ctypes.POINTER(ctypes.c_void_p)


def _sig(name, restype, *argtypes):
    fn = getattr(_lib, name)
    fn.restype = restype
    fn.argtypes = list(argtypes)
    return fn


_philox = _sig("oracle_philox4x32_10", None, _u32p, _u32p, _u32p)
_round_keys = _sig("oracle_round_keys", None, ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint32, _u32p)
_feistel = _sig("oracle_feistel_perm", ctypes.c_uint64, ctypes.c_uint64, ctypes.c_uint64, _u32p)
_score = _sig("oracle_score", None, _f32p, _pp, ctypes.c_uint32, ctypes.c_float, ctypes.c_uint64, _f32p)
_select = _sig("oracle_select_core", None, _f32p, ctypes.c_uint64, ctypes.c_uint64, _u32p)
_explore = _sig("oracle_sample_explore", None, _u32p, ctypes.c_uint64, ctypes.c_uint64, ctypes.c_uint64,
                ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint32, _u32p)
_pack = _sig("oracle_pack", None, _f32p, _u32p, ctypes.c_uint64, _u32p, ctypes.c_uint64, _f32p)
_merge = _sig("oracle_merge", None, _f32p, ctypes.c_uint32, _u32p, ctypes.c_uint64, _pp, ctypes.c_uint64,
              _pp, ctypes.c_float)
_pull = _sig("oracle_pull", None, _f32p, _u32p, ctypes.c_uint64, _u32p, ctypes.c_uint64, _f32p)
_dense = _sig("oracle_dense_merge", None, _f32p, ctypes.c_uint64, ctypes.c_uint32, _pp, ctypes.c_float)
_signature = _sig("oracle_core_signature", ctypes.c_uint64, _u32p, ctypes.c_uint64)
_u8p = ctypes.POINTER(ctypes.c_uint8)
_wire_bytes = _sig("oracle_wire_message_bytes", ctypes.c_uint64, ctypes.c_uint64, ctypes.c_uint64, ctypes.c_int)
_wire_pack = _sig("oracle_wire_pack", None, _u32p, ctypes.c_uint64, _u32p, ctypes.c_uint64, _f32p, ctypes.c_uint32,
                  ctypes.c_uint32, ctypes.c_int, _u8p)
_wire_unpack = _sig("oracle_wire_unpack", ctypes.c_int32, _u8p, ctypes.c_uint64, ctypes.c_uint64, ctypes.c_uint64,
                    ctypes.c_uint64, _u32p, _u32p, _f32p, ctypes.POINTER(ctypes.c_uint64))
_u64p = ctypes.POINTER(ctypes.c_uint64)
_i8p = ctypes.POINTER(ctypes.c_int8)
_select_seg = _sig("oracle_select_core_segmented", None, _f32p, ctypes.c_uint64, _u64p, _u64p, ctypes.c_uint32, _u32p)
_quant = _sig("oracle_quantize_q8", None, _f32p, ctypes.c_uint64, ctypes.c_uint32, _i8p, _f32p)
_dequant = _sig("oracle_dequantize_q8", None, _i8p, _f32p, ctypes.c_uint64, ctypes.c_uint32, _f32p)
_wmerge = _sig("oracle_worker_merge", None, _f32p, _u32p, ctypes.c_uint64, _u32p, ctypes.c_uint64, _f32p)


def _f32(a) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a


def _u32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.uint32)


def _ptr(a: np.ndarray, typ):
    return a.ctypes.data_as(typ)


def _ptr_array(arrs: Sequence[np.ndarray]):
    return (ctypes.c_void_p * len(arrs))(*[a.ctypes.data for a in arrs])


def philox4x32_10(key: Sequence[int], ctr: Sequence[int]) -> List[int]:
    k, c, o = _u32(key), _u32(ctr), np.zeros(4, np.uint32)
    _philox(_ptr(k, _u32p), _ptr(c, _u32p), _ptr(o, _u32p))
    return [int(x) for x in o]


def round_keys(seed: int, worker: int, rnd: int) -> np.ndarray:
    rk = np.zeros(12, np.uint32)
    _round_keys(seed, worker, rnd, _ptr(rk, _u32p))
    return rk


def feistel_perm(j: int, M: int, rk: np.ndarray) -> int:
    rk = _u32(rk)
    return int(_feistel(j, M, _ptr(rk, _u32p)))


def score(w, grads: Sequence[np.ndarray], c: float) -> np.ndarray:
    w = _f32(w)
    gs = [_f32(g) for g in grads]
    assert len(gs) >= 1 and all(g.shape == w.shape for g in gs)
    out = np.empty_like(w)
    _score(_ptr(w, _f32p), _ptr_array(gs), len(gs), c, w.size, _ptr(out, _f32p))
    return out


def select_core(scores, k_core: int) -> np.ndarray:
    s = _f32(scores)
    assert 0 <= k_core <= s.size
    out = np.empty(k_core, np.uint32)
    _select(_ptr(s, _f32p), s.size, k_core, _ptr(out, _u32p))
    return out


def sample_explore(core_idx, n: int, k_exp: int, seed: int, worker: int, rnd: int) -> np.ndarray:
    core = _u32(core_idx)
    assert 0 <= k_exp <= n - core.size
    out = np.empty(k_exp, np.uint32)
    _explore(_ptr(core, _u32p), n, core.size, k_exp, seed, worker, rnd, _ptr(out, _u32p))
    return out


def pack(delta, core_idx, exp_idx) -> np.ndarray:
    d, c, e = _f32(delta), _u32(core_idx), _u32(exp_idx)
    out = np.empty(c.size + e.size, np.float32)
    _pack(_ptr(d, _f32p), _ptr(c, _u32p), c.size, _ptr(e, _u32p), e.size, _ptr(out, _f32p))
    return out


def merge(w, core_idx, exp_idx: Sequence[np.ndarray], val: Sequence[np.ndarray], eta: float) -> np.ndarray:
    """Returns the merged copy of w (the input is left untouched)."""
    out = _f32(w).copy()
    c = _u32(core_idx)
    es = [_u32(e) for e in exp_idx]
    vs = [_f32(v) for v in val]
    K = len(vs)
    assert len(es) == K and all(e.size == es[0].size for e in es)
    k_exp = es[0].size if K else 0
    assert all(v.size == c.size + k_exp for v in vs)
    _merge(_ptr(out, _f32p), K, _ptr(c, _u32p), c.size, _ptr_array(es), k_exp, _ptr_array(vs), eta)
    return out


def pull(w, core_idx, exp_idx) -> np.ndarray:
    w, c, e = _f32(w), _u32(core_idx), _u32(exp_idx)
    out = np.empty(c.size + e.size, np.float32)
    _pull(_ptr(w, _f32p), _ptr(c, _u32p), c.size, _ptr(e, _u32p), e.size, _ptr(out, _f32p))
    return out


def dense_merge(w, grads: Sequence[np.ndarray], eta: float) -> np.ndarray:
    out = _f32(w).copy()
    gs = [_f32(g) for g in grads]
    _dense(_ptr(out, _f32p), out.size, len(gs), _ptr_array(gs), eta)
    return out


def worker_merge(w_local, core_idx, exp_idx, pulled) -> np.ndarray:
    """Returns the merged copy of the local model (the input is left untouched)."""
    out = _f32(w_local).copy()
    c, e, p = _u32(core_idx), _u32(exp_idx), _f32(pulled)
    assert p.size == c.size + e.size
    _wmerge(_ptr(out, _f32p), _ptr(c, _u32p), c.size, _ptr(e, _u32p), e.size, _ptr(p, _f32p))
    return out


def core_signature(keys) -> int:
    k = _u32(keys)
    return int(_signature(_ptr(k, _u32p), k.size))


def select_core_segmented(scores, seg_off: Sequence[int], seg_k: Sequence[int]) -> np.ndarray:
    """Per-segment top-k: segment s = [seg_off[s], seg_off[s+1]) contributes its seg_k[s] largest scores."""
    s = _f32(scores)
    off = np.ascontiguousarray(seg_off, dtype=np.uint64)
    ks = np.ascontiguousarray(seg_k, dtype=np.uint64)
    assert off.size == ks.size + 1 and off[0] == 0 and off[-1] == s.size
    assert all(int(ks[i]) <= int(off[i + 1]) - int(off[i]) for i in range(ks.size))
    out = np.empty(int(ks.sum()), np.uint32)
    _select_seg(_ptr(s, _f32p), s.size, _ptr(off, _u64p), _ptr(ks, _u64p), ks.size, _ptr(out, _u32p))
    return out


Q8_BUCKET = 256


def quantize_q8(val, bucket: int = Q8_BUCKET):
    """(codes int8[m], scales float32[ceil(m / bucket)]) of the packed values."""
    v = _f32(val)
    codes = np.zeros(v.size, np.int8)
    scales = np.zeros((v.size + bucket - 1) // bucket, np.float32)
    _quant(_ptr(v, _f32p), v.size, bucket, _ptr(codes, _i8p), _ptr(scales, _f32p))
    return codes, scales


def dequantize_q8(codes, scales, bucket: int = Q8_BUCKET) -> np.ndarray:
    c = np.ascontiguousarray(codes, dtype=np.int8)
    s = _f32(scales)
    out = np.zeros(c.size, np.float32)
    _dequant(_ptr(c, _i8p), _ptr(s, _f32p), c.size, bucket, _ptr(out, _f32p))
    return out


def wire_message_bytes(k_core: int, k_exp: int, with_keys: bool) -> int:
    return int(_wire_bytes(k_core, k_exp, int(with_keys)))


def wire_pack(core_idx, exp_idx, val, worker: int, rnd: int, with_keys: bool) -> np.ndarray:
    """One worker's push as a byte message (Section 3.5)."""
    c, e, v = _u32(core_idx), _u32(exp_idx), _f32(val)
    assert v.size == c.size + e.size
    msg = np.zeros(wire_message_bytes(c.size, e.size, with_keys), np.uint8)
    _wire_pack(_ptr(c, _u32p), c.size, _ptr(e, _u32p), e.size, _ptr(v, _f32p), worker, rnd, int(with_keys),
               _ptr(msg, _u8p))
    return msg


def wire_unpack(msg, cached_signature: int, k_core: int, k_exp: int):
    """Takes a push message apart on the receiver's side.  Returns (status, core_idx or None, exp_idx, val,
    signature): status 0 = taken, 1 = keys wanted (nothing else is meaningful), -1 = malformed."""
    m = np.ascontiguousarray(msg, dtype=np.uint8)
    core = np.zeros(k_core, np.uint32)
    exp = np.zeros(k_exp, np.uint32)
    val = np.zeros(k_core + k_exp, np.float32)
    sig = ctypes.c_uint64(cached_signature)
    st = int(_wire_unpack(_ptr(m, _u8p), m.size, cached_signature, k_core, k_exp, _ptr(core, _u32p), _ptr(exp, _u32p),
                          _ptr(val, _f32p), ctypes.byref(sig)))
    carried_keys = st == 0 and m.size >= 8 and (int(m[4]) & 1) == 1
    return st, (core if carried_keys else None), exp, val, int(sig.value)


def run_round(w, grads: Sequence[np.ndarray], c: float, k_core: int, k_exp: int,
              seed: int, rnd: int, eta: float) -> Dict[str, object]:
    """One whole communication round in the order
    score -> select -> K x explore -> K x pack -> merge -> K x pull."""
    K = len(grads)
    n = int(np.asarray(w).size)
    S = score(w, grads, c)
    core = select_core(S, k_core)
    exp = [sample_explore(core, n, k_exp, seed, k, rnd) for k in range(K)]
    val = [pack(grads[k], core, exp[k]) for k in range(K)]
    merged = merge(w, core, exp, val, eta)
    pulled = [pull(merged, core, exp[k]) for k in range(K)]
    return {"scores": S, "core_idx": core, "exp_idx": exp, "val": val, "w": merged, "pulled": pulled}
