"""ctypes binding of libslimdp.so.  Argument marshalling only.

The shared library must have been built in-tree (python -m
paper_1709_09393_b200.build); importing this module without it raises.
There is no fallback path of any kind.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libslimdp.so")

if not os.path.exists(_LIB_PATH):
    raise ImportError(
        f"{_LIB_PATH} is missing: build the CUDA library first (python -m paper_1709_09393_b200.build)")

lib = ctypes.CDLL(_LIB_PATH)

_vp = ctypes.c_void_p
_u64 = ctypes.c_uint64
_u32 = ctypes.c_uint32
_f32 = ctypes.c_float
_sz = ctypes.c_size_t
_pp = ctypes.POINTER(ctypes.c_void_p)

EXPORTS = {
    "slimdp_status_string": (ctypes.c_char_p, [ctypes.c_int32]),
    "slimdp_core_aux_bytes": (_sz, [_u64]),
    "slimdp_core_aux_dir_offset": (_sz, [_u64]),
    "slimdp_select_workspace_bytes": (_sz, [_u64]),
    "slimdp_explore_workspace_bytes": (_sz, [_u64, _u64, _u32]),
    "slimdp_workspace_bytes": (_sz, [_u64, _u32, _u64, _u64]),
    "slimdp_score": (ctypes.c_int32, [_vp, _pp, _u32, _f32, _u64, _vp, _vp]),
    "slimdp_select_core": (ctypes.c_int32, [_vp, _u64, _u64, _vp, _vp, _vp, _sz, _vp]),
    "slimdp_sample_explore": (ctypes.c_int32, [_vp, _u64, _u64, _u64, _u64, _u32, _u32, _vp, _vp, _sz, _vp]),
    "slimdp_sample_explore_batched": (ctypes.c_int32,
                                      [_vp, _u64, _u64, _u64, _u64, _u32, _u32, _u32, _pp, _vp, _sz, _vp]),
    "slimdp_sample_explore_static": (ctypes.c_int32, [_vp, _u64, _u64, _u64, _u64, _u32, _u32, _vp, _vp, _vp]),
    "slimdp_pack": (ctypes.c_int32, [_vp, _u64, _vp, _u64, _vp, _u64, _vp, _vp]),
    "slimdp_pack_batched": (ctypes.c_int32, [_pp, _u32, _u64, _vp, _u64, _pp, _u64, _pp, _vp]),
    "slimdp_merge": (ctypes.c_int32, [_vp, _u64, _u32, _vp, _u64, _pp, _u64, _pp, _f32, _vp]),
    "slimdp_pull": (ctypes.c_int32, [_vp, _u64, _vp, _u64, _vp, _u64, _vp, _vp]),
    "slimdp_pull_batched": (ctypes.c_int32, [_vp, _u32, _u64, _vp, _u64, _pp, _u64, _pp, _vp]),
    "slimdp_exchange": (ctypes.c_int32, [_vp, _u64, _u32, _pp, _vp, _u64, _pp, _u64, _f32, _pp, _pp, _vp]),
    "slimdp_dense_merge_score": (ctypes.c_int32, [_vp, _pp, _u32, _f32, _f32, _u64, _vp, _vp]),
    "slimdp_worker_merge_batched": (ctypes.c_int32, [_pp, _u32, _u64, _vp, _u64, _pp, _u64, _pp, _vp]),
    "slimdp_core_signature": (ctypes.c_int32, [_vp, _u64, _vp, _vp]),
    "slimdp_wire_bytes": (_sz, [_u64, _u64]),
    "slimdp_select_segmented_workspace_bytes": (_sz, [_u64, _u32]),
    "slimdp_select_core_segmented": (ctypes.c_int32, [_vp, _u64, _vp, _vp, _u32, _vp, _vp, _vp, _sz, _vp]),
    "slimdp_pack_q8_batched": (ctypes.c_int32, [_pp, _u32, _u64, _vp, _u64, _pp, _u64, _pp, _pp, _vp]),
    "slimdp_merge_q8": (ctypes.c_int32, [_vp, _u64, _u32, _vp, _u64, _pp, _u64, _pp, _pp, _f32, _vp]),
    "slimdp_explore_shard_workspace_bytes": (_sz, [_u64, _u64, _u64]),
    "slimdp_sample_explore_shard": (ctypes.c_int32, [_vp, _u64, _u64, _u64, _u64, _u64, _u64, _u32, _u32, _vp, _u64, _vp,
                                                     _vp, _sz, _vp]),
    "slimdp_select_shard_begin": (ctypes.c_int32, [_u64, _vp, _vp]),
    "slimdp_select_hist": (ctypes.c_int32, [_vp, _u64, _u32, _vp, _vp, _vp]),
    "slimdp_select_resolve": (ctypes.c_int32, [_vp, _u32, _vp, _vp]),
    "slimdp_select_count": (ctypes.c_int32, [_vp, _u64, _vp, _vp, _vp]),
    "slimdp_select_emit": (ctypes.c_int32, [_vp, _u64, _u32, _u64, _u64, _vp, _vp, _vp, _sz, _vp]),
    "slimdp_wire_message_bytes": (_sz, [_u64, _u64, ctypes.c_int]),
    "slimdp_wire_pack": (ctypes.c_int32, [_vp, _u64, _vp, _u64, _vp, _vp, _u32, _u32, ctypes.c_int, _vp, _vp]),
    "slimdp_wire_unpack": (ctypes.c_int32, [_vp, _sz, _vp, _u64, _u64, _vp, _vp, _vp, _vp, _vp, _vp]),
    "slimdp_wire_read_status": (ctypes.c_int32, [_vp, _vp]),
    "slimdp_read_status": (ctypes.c_int32, [_vp, _vp]),
    "slimdp_launch_count": (_u64, []),
    "slimdp_round_arena_bytes": (_sz, [_u64, _u32, _u64, _u64]),
    "slimdp_round": (ctypes.c_int32, [_vp, _pp, _u32, _u64, _f32, _u64, _u64, _u64, _u32, _f32, _vp, _vp, _vp, _pp, _pp,
                                      _pp, _vp, _sz, _vp, _sz, _vp, _sz, _vp, _vp]),
    "slimdp_round_ctx_create": (ctypes.c_int32, [_pp]),
    "slimdp_round_ctx_destroy": (ctypes.c_int32, [_vp]),
    "slimdp_round_release_default_ctx": (ctypes.c_int32, []),
    "slimdp_round_stage_bytes": (_sz, [_u64, _u32, _u64]),
    "slimdp_mark_dominant_kernel": (None, [_vp, _vp]),
    "slimdp_round_host": (ctypes.c_int32, [_vp, _pp, _u32, _u64, _f32, _u64, _u64, _u64, _u32, _f32, _vp, _pp, _pp,
                                           _vp, _sz, _vp]),
}

for _name, (_res, _args) in EXPORTS.items():
    _fn = getattr(lib, _name)
    _fn.restype = _res
    _fn.argtypes = _args


class SlimDPError(RuntimeError):
    def __init__(self, call: str, status: int):
        self.status = status
        msg = lib.slimdp_status_string(status).decode()
        super().__init__(f"{call} failed: {msg} ({status})")


def _check(call: str, status: int) -> None:
    if status != 0:
        raise SlimDPError(call, status)


def _stream(stream: Optional[torch.cuda.Stream] = None) -> int:
    return (stream or torch.cuda.current_stream()).cuda_stream


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    """Device/host address, or NULL for a missing or empty tensor."""
    if t is None:
        return None
    return t.data_ptr() or None


def _dev(t: torch.Tensor, dtype, name: str) -> torch.Tensor:
    if not t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise TypeError(f"{name}: expected a contiguous CUDA tensor of {dtype}")
    return t


def _ptr_array(ts: Sequence[torch.Tensor]):
    return (ctypes.c_void_p * len(ts))(*[t.data_ptr() for t in ts])


# int32 carries uint32 indices (torch has no full uint32 support); values are reinterpreted, not converted
IDX = torch.int32


def core_aux_bytes(n: int) -> int:
    return lib.slimdp_core_aux_bytes(n)


def core_aux_dir_offset(n: int) -> int:
    return lib.slimdp_core_aux_dir_offset(n)


def select_workspace_bytes(n: int) -> int:
    return lib.slimdp_select_workspace_bytes(n)


def explore_workspace_bytes(n: int, k_exp: int, num_workers: int) -> int:
    return lib.slimdp_explore_workspace_bytes(n, k_exp, num_workers)


def workspace_bytes(n: int, K: int, k_core: int, k_exp: int) -> int:
    return lib.slimdp_workspace_bytes(n, K, k_core, k_exp)


def round_arena_bytes(n: int, K: int, k_core: int, k_exp: int) -> int:
    return lib.slimdp_round_arena_bytes(n, K, k_core, k_exp)


def launch_count() -> int:
    """Kernels launched by the library in this process so far."""
    return lib.slimdp_launch_count()


def read_status(ws: torch.Tensor, stream=None) -> None:
    _check("slimdp_read_status", lib.slimdp_read_status(ws.data_ptr(), _stream(stream)))


def slimdp_score(w: torch.Tensor, grads: Sequence[torch.Tensor], c: float, scores: torch.Tensor, stream=None):
    n = w.numel()
    _dev(w, torch.float32, "w")
    _dev(scores, torch.float32, "scores")
    for g in grads:
        if _dev(g, torch.float32, "grads").numel() != n:
            raise ValueError("grads: length differs from w")
    if scores.numel() != n:
        raise ValueError("scores: length differs from w")
    _check("slimdp_score", lib.slimdp_score(w.data_ptr(), _ptr_array(grads), len(grads), c, n, scores.data_ptr(),
                                            _stream(stream)))


def slimdp_select_core(scores: torch.Tensor, k_core: int, core_idx: torch.Tensor, core_aux: torch.Tensor,
                       ws: torch.Tensor, stream=None):
    _dev(scores, torch.float32, "scores")
    _dev(core_idx, IDX, "core_idx")
    if core_idx.numel() != k_core:
        raise ValueError("core_idx: length differs from k_core")
    _check("slimdp_select_core",
           lib.slimdp_select_core(scores.data_ptr(), scores.numel(), k_core, _ptr(core_idx), core_aux.data_ptr(),
                                  ws.data_ptr(), ws.numel() * ws.element_size(), _stream(stream)))


def slimdp_sample_explore(core_aux: torch.Tensor, n: int, k_core: int, k_exp: int, seed: int, worker: int,
                          rnd: int, exp_idx: torch.Tensor, ws: torch.Tensor, stream=None):
    _dev(exp_idx, IDX, "exp_idx")
    if exp_idx.numel() != k_exp:
        raise ValueError("exp_idx: length differs from k_exp")
    _check("slimdp_sample_explore",
           lib.slimdp_sample_explore(core_aux.data_ptr(), n, k_core, k_exp, seed, worker, rnd, _ptr(exp_idx),
                                     ws.data_ptr(), ws.numel() * ws.element_size(), _stream(stream)))


def slimdp_sample_explore_batched(core_aux: torch.Tensor, n: int, k_core: int, k_exp: int, seed: int,
                                  first_worker: int, rnd: int, exp_idx: Sequence[torch.Tensor], ws: torch.Tensor,
                                  stream=None):
    for e in exp_idx:
        if _dev(e, IDX, "exp_idx").numel() != k_exp:
            raise ValueError("exp_idx: length differs from k_exp")
    _check("slimdp_sample_explore_batched",
           lib.slimdp_sample_explore_batched(core_aux.data_ptr(), n, k_core, k_exp, seed, first_worker,
                                             len(exp_idx), rnd, _ptr_array(exp_idx), ws.data_ptr(),
                                             ws.numel() * ws.element_size(), _stream(stream)))


def slimdp_sample_explore_static(core_aux: torch.Tensor, n: int, k_core: int, k_exp: int, seed: int, worker: int,
                                 rnd: int, exp_idx: torch.Tensor, status: Optional[torch.Tensor] = None,
                                 stream=None):
    """slimdp_sample_explore for callers that cannot allocate a workspace: the library's own
    static scratch is used (n <= 2^25, k_exp <= 2^18).  `status`, if given, is a one-element
    int32 CUDA tensor that receives the device-side consistency status in stream order."""
    _dev(exp_idx, IDX, "exp_idx")
    if exp_idx.numel() != k_exp:
        raise ValueError("exp_idx: length differs from k_exp")
    if status is not None:
        _dev(status, torch.int32, "status")
    _check("slimdp_sample_explore_static",
           lib.slimdp_sample_explore_static(core_aux.data_ptr(), n, k_core, k_exp, seed, worker, rnd, _ptr(exp_idx),
                                            _ptr(status), _stream(stream)))


def _check_sets(core_idx, exp_idx, out, what):
    _dev(core_idx, IDX, "core_idx")
    _dev(exp_idx, IDX, "exp_idx")
    _dev(out, torch.float32, what)
    if out.numel() != core_idx.numel() + exp_idx.numel():
        raise ValueError(f"{what}: length differs from k_core + k_exp")


def slimdp_pack(delta: torch.Tensor, core_idx: torch.Tensor, exp_idx: torch.Tensor, val: torch.Tensor, stream=None):
    _dev(delta, torch.float32, "delta")
    _check_sets(core_idx, exp_idx, val, "val")
    _check("slimdp_pack", lib.slimdp_pack(delta.data_ptr(), delta.numel(), _ptr(core_idx), core_idx.numel(),
                                          _ptr(exp_idx), exp_idx.numel(), _ptr(val), _stream(stream)))


def slimdp_pack_batched(deltas: Sequence[torch.Tensor], core_idx: torch.Tensor, exp_idx: Sequence[torch.Tensor],
                        val: Sequence[torch.Tensor], stream=None):
    K = len(deltas)
    if len(exp_idx) != K or len(val) != K:
        raise ValueError("deltas, exp_idx and val must have K entries each")
    for d, e, v in zip(deltas, exp_idx, val):
        _dev(d, torch.float32, "deltas")
        _check_sets(core_idx, e, v, "val")
    _check("slimdp_pack_batched",
           lib.slimdp_pack_batched(_ptr_array(deltas), K, deltas[0].numel(), _ptr(core_idx), core_idx.numel(),
                                   _ptr_array(exp_idx), exp_idx[0].numel(), _ptr_array(val), _stream(stream)))


def slimdp_merge(w_global: torch.Tensor, core_idx: torch.Tensor, exp_idx: Sequence[torch.Tensor],
                 val: Sequence[torch.Tensor], eta: float, stream=None):
    _dev(w_global, torch.float32, "w_global")
    K = len(val)
    if len(exp_idx) != K:
        raise ValueError("exp_idx and val must have K entries each")
    for e, v in zip(exp_idx, val):
        _check_sets(core_idx, e, v, "val")
    _check("slimdp_merge",
           lib.slimdp_merge(w_global.data_ptr(), w_global.numel(), K, _ptr(core_idx), core_idx.numel(),
                            _ptr_array(exp_idx), exp_idx[0].numel(), _ptr_array(val), eta, _stream(stream)))


def slimdp_pull(w_global: torch.Tensor, core_idx: torch.Tensor, exp_idx: torch.Tensor, out: torch.Tensor,
                stream=None):
    _dev(w_global, torch.float32, "w_global")
    _check_sets(core_idx, exp_idx, out, "out")
    _check("slimdp_pull", lib.slimdp_pull(w_global.data_ptr(), w_global.numel(), _ptr(core_idx), core_idx.numel(),
                                          _ptr(exp_idx), exp_idx.numel(), _ptr(out), _stream(stream)))


def slimdp_pull_batched(w_global: torch.Tensor, core_idx: torch.Tensor, exp_idx: Sequence[torch.Tensor],
                        out: Sequence[torch.Tensor], stream=None):
    _dev(w_global, torch.float32, "w_global")
    K = len(out)
    if len(exp_idx) != K:
        raise ValueError("exp_idx and out must have K entries each")
    for e, o in zip(exp_idx, out):
        _check_sets(core_idx, e, o, "out")
    _check("slimdp_pull_batched",
           lib.slimdp_pull_batched(w_global.data_ptr(), K, w_global.numel(), _ptr(core_idx), core_idx.numel(),
                                   _ptr_array(exp_idx), exp_idx[0].numel(), _ptr_array(out), _stream(stream)))


def slimdp_exchange(w_global: torch.Tensor, deltas: Sequence[torch.Tensor], core_idx: torch.Tensor,
                    exp_idx: Sequence[torch.Tensor], eta: float, val: Sequence[torch.Tensor],
                    pulled: Sequence[torch.Tensor], stream=None):
    """Push + update + pull for all workers; same results as pack_batched, merge, pull_batched."""
    _dev(w_global, torch.float32, "w_global")
    K = len(deltas)
    if len(exp_idx) != K or len(val) != K or len(pulled) != K:
        raise ValueError("deltas, exp_idx, val and pulled must have K entries each")
    for d, e, v, o in zip(deltas, exp_idx, val, pulled):
        if _dev(d, torch.float32, "deltas").numel() != w_global.numel():
            raise ValueError("deltas: length differs from w_global")
        _check_sets(core_idx, e, v, "val")
        _check_sets(core_idx, e, o, "pulled")
    _check("slimdp_exchange",
           lib.slimdp_exchange(w_global.data_ptr(), w_global.numel(), K, _ptr_array(deltas), _ptr(core_idx),
                               core_idx.numel(), _ptr_array(exp_idx), exp_idx[0].numel(), eta, _ptr_array(val),
                               _ptr_array(pulled), _stream(stream)))


def slimdp_round(w_global: torch.Tensor, grads: Sequence[torch.Tensor], c: float, seed: int, rnd: int, eta: float,
                 scores: torch.Tensor, core_idx: torch.Tensor, core_aux: torch.Tensor,
                 exp_idx: Sequence[torch.Tensor], val: Sequence[torch.Tensor], pulled: Sequence[torch.Tensor],
                 select_ws: torch.Tensor, explore_ws: torch.Tensor, stage: Optional[torch.Tensor] = None,
                 ctx: Optional["RoundContext"] = None, stream=None):
    """One whole round on device buffers; same results as score, select_core, sample_explore_batched,
    exchange, except that `scores` is scratch (written only if the selection falls back to its full path).
    `stage` (uint8, round_stage_bytes long) lets the round set the core's update values aside during its
    pass; `ctx` is the round context whose streams the round runs on (None: the library's default one)."""
    n = w_global.numel()
    _dev(w_global, torch.float32, "w_global")
    K = len(grads)
    if len(exp_idx) != K or len(val) != K or len(pulled) != K:
        raise ValueError("grads, exp_idx, val and pulled must have K entries each")
    if _dev(scores, torch.float32, "scores").numel() != n:
        raise ValueError("scores: length differs from w_global")
    for g, e, v, o in zip(grads, exp_idx, val, pulled):
        if _dev(g, torch.float32, "grads").numel() != n:
            raise ValueError("grads: length differs from w_global")
        _check_sets(core_idx, e, v, "val")
        _check_sets(core_idx, e, o, "pulled")
    for t, name in ((core_aux, "core_aux"), (select_ws, "select_ws"), (explore_ws, "explore_ws")):
        _dev(t, torch.uint8, name)
    if stage is not None:
        _dev(stage, torch.uint8, "stage")
    _check("slimdp_round",
           lib.slimdp_round(w_global.data_ptr(), _ptr_array(grads), K, n, c, core_idx.numel(), exp_idx[0].numel(),
                            seed, rnd, eta, _ptr(scores), _ptr(core_idx), _ptr(core_aux), _ptr_array(exp_idx),
                            _ptr_array(val), _ptr_array(pulled), _ptr(select_ws), select_ws.numel(),
                            _ptr(explore_ws), explore_ws.numel(), _ptr(stage), stage.numel() if stage is not None else 0,
                            ctx.handle if ctx is not None else None, _stream(stream)))


def round_stage_bytes(n: int, K: int, k_core: int) -> int:
    """Bytes of staging area for slimdp_round on the current device (0: staging does not apply)."""
    return lib.slimdp_round_stage_bytes(n, K, k_core)


class RoundContext:
    """A round context on the current device (two streams, four events), owned by the caller."""

    def __init__(self):
        h = ctypes.c_void_p()
        _check("slimdp_round_ctx_create", lib.slimdp_round_ctx_create(ctypes.byref(h)))
        self.handle = h

    def close(self) -> None:
        if self.handle is not None:
            _check("slimdp_round_ctx_destroy", lib.slimdp_round_ctx_destroy(self.handle))
            self.handle = None

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()


def release_default_round_ctx() -> None:
    _check("slimdp_round_release_default_ctx", lib.slimdp_round_release_default_ctx())


def mark_dominant_kernel(begin: Optional[torch.cuda.Event], end: Optional[torch.cuda.Event]) -> None:
    """The next slimdp_round records the two events around its pass over all parameters.  Both
    events must have been recorded once already (torch creates the CUDA event lazily)."""
    lib.slimdp_mark_dominant_kernel(begin.cuda_event if begin is not None else None,
                                    end.cuda_event if end is not None else None)


def slimdp_dense_merge_score(w_global: torch.Tensor, grads: Sequence[torch.Tensor], eta: float, c: float,
                             scores: Optional[torch.Tensor] = None, stream=None):
    """Dense push of all workers at a reselection boundary; optionally scores the updated model."""
    n = w_global.numel()
    _dev(w_global, torch.float32, "w_global")
    for g in grads:
        if _dev(g, torch.float32, "grads").numel() != n:
            raise ValueError("grads: length differs from w_global")
    if scores is not None and _dev(scores, torch.float32, "scores").numel() != n:
        raise ValueError("scores: length differs from w_global")
    _check("slimdp_dense_merge_score",
           lib.slimdp_dense_merge_score(w_global.data_ptr(), _ptr_array(grads), len(grads), eta, c, n, _ptr(scores),
                                        _stream(stream)))


def slimdp_worker_merge_batched(w_local: Sequence[torch.Tensor], core_idx: torch.Tensor,
                                exp_idx: Sequence[torch.Tensor], pulled: Sequence[torch.Tensor], stream=None):
    """Worker-side Merge: pulled values overwrite each local model on its communication set."""
    K = len(w_local)
    if len(exp_idx) != K or len(pulled) != K:
        raise ValueError("w_local, exp_idx and pulled must have K entries each")
    n = w_local[0].numel()
    for wl, e, p in zip(w_local, exp_idx, pulled):
        if _dev(wl, torch.float32, "w_local").numel() != n:
            raise ValueError("w_local: lengths differ")
        _check_sets(core_idx, e, p, "pulled")
    _check("slimdp_worker_merge_batched",
           lib.slimdp_worker_merge_batched(_ptr_array(w_local), K, n, _ptr(core_idx), core_idx.numel(),
                                           _ptr_array(exp_idx), exp_idx[0].numel(), _ptr_array(pulled),
                                           _stream(stream)))


def slimdp_core_signature(keys: torch.Tensor, signature: torch.Tensor, stream=None):
    """64-bit signature of a key list (key caching, Section 3.5) into a one-element int64 CUDA tensor."""
    _dev(keys, IDX, "keys")
    _dev(signature, torch.int64, "signature")
    _check("slimdp_core_signature",
           lib.slimdp_core_signature(_ptr(keys), keys.numel(), signature.data_ptr(), _stream(stream)))


def wire_bytes(k_core: int, k_exp: int) -> int:
    return lib.slimdp_wire_bytes(k_core, k_exp)


def select_segmented_workspace_bytes(n: int, segments: int) -> int:
    return lib.slimdp_select_segmented_workspace_bytes(n, segments)


def slimdp_select_core_segmented(scores: torch.Tensor, seg_off: Sequence[int], seg_k: Sequence[int],
                                 core_idx: torch.Tensor, core_aux: torch.Tensor, ws: torch.Tensor, stream=None):
    """Per-layer selection: segment s = [seg_off[s], seg_off[s+1]) contributes its seg_k[s] largest scores."""
    _dev(scores, torch.float32, "scores")
    _dev(core_idx, IDX, "core_idx")
    S = len(seg_k)
    if len(seg_off) != S + 1:
        raise ValueError("seg_off must have one entry more than seg_k")
    if core_idx.numel() != sum(int(k) for k in seg_k):
        raise ValueError("core_idx: length differs from the sum of seg_k")
    off = (ctypes.c_uint64 * (S + 1))(*[int(x) for x in seg_off])
    ks = (ctypes.c_uint64 * S)(*[int(x) for x in seg_k])
    _check("slimdp_select_core_segmented",
           lib.slimdp_select_core_segmented(scores.data_ptr(), scores.numel(), off, ks, S, _ptr(core_idx),
                                            core_aux.data_ptr(), ws.data_ptr(), ws.numel(), _stream(stream)))


Q8_BUCKET = 256


def slimdp_pack_q8_batched(deltas: Sequence[torch.Tensor], core_idx: torch.Tensor, exp_idx: Sequence[torch.Tensor],
                           codes: Sequence[torch.Tensor], scales: Sequence[torch.Tensor], stream=None):
    """Extraction with the 8-bit quantiser folded in: codes[k] int8[m], scales[k] float32[ceil(m / 256)]."""
    K, n = len(deltas), deltas[0].numel()
    m = core_idx.numel() + exp_idx[0].numel()
    for d, e, c, s in zip(deltas, exp_idx, codes, scales):
        _dev(d, torch.float32, "deltas")
        _dev(e, IDX, "exp_idx")
        if _dev(c, torch.int8, "codes").numel() != m or _dev(s, torch.float32, "scales").numel() != (m + 255) // 256:
            raise ValueError("codes / scales: wrong length")
    _check("slimdp_pack_q8_batched",
           lib.slimdp_pack_q8_batched(_ptr_array(deltas), K, n, _ptr(core_idx), core_idx.numel(), _ptr_array(exp_idx),
                                      exp_idx[0].numel(), _ptr_array(codes), _ptr_array(scales), _stream(stream)))


def slimdp_merge_q8(w_global: torch.Tensor, core_idx: torch.Tensor, exp_idx: Sequence[torch.Tensor],
                    codes: Sequence[torch.Tensor], scales: Sequence[torch.Tensor], eta: float, stream=None):
    """Server update reading the pushed values through their 8-bit codes."""
    _dev(w_global, torch.float32, "w_global")
    K = len(codes)
    for e, c, s in zip(exp_idx, codes, scales):
        _dev(e, IDX, "exp_idx")
        _dev(c, torch.int8, "codes")
        _dev(s, torch.float32, "scales")
    _check("slimdp_merge_q8",
           lib.slimdp_merge_q8(w_global.data_ptr(), w_global.numel(), K, _ptr(core_idx), core_idx.numel(),
                               _ptr_array(exp_idx), exp_idx[0].numel(), _ptr_array(codes), _ptr_array(scales), eta,
                               _stream(stream)))


def explore_shard_workspace_bytes(n_shard: int, noncore_total: int, k_exp: int) -> int:
    return lib.slimdp_explore_shard_workspace_bytes(n_shard, noncore_total, k_exp)


def slimdp_sample_explore_shard(core_aux: torch.Tensor, n_shard: int, k_core_shard: int, noncore_total: int,
                                noncore_below: int, k_exp: int, seed: int, worker: int, rnd: int,
                                exp_idx: torch.Tensor, count: torch.Tensor, ws: torch.Tensor, stream=None):
    """One shard's share of a worker's explorer: count[0] shard-local indices into exp_idx (its length is the cap)."""
    _dev(exp_idx, IDX, "exp_idx")
    _dev(count, torch.int32, "count")
    _check("slimdp_sample_explore_shard",
           lib.slimdp_sample_explore_shard(core_aux.data_ptr(), n_shard, k_core_shard, noncore_total, noncore_below,
                                           k_exp, seed, worker, rnd, _ptr(exp_idx), exp_idx.numel(), count.data_ptr(),
                                           ws.data_ptr(), ws.numel(), _stream(stream)))


def slimdp_select_shard_begin(k_total: int, state: torch.Tensor, stream=None):
    """state (int64[2] CUDA tensor) <- (prefix 0, rank k_total): start of a selection over a sharded model."""
    _dev(state, torch.int64, "state")
    _check("slimdp_select_shard_begin", lib.slimdp_select_shard_begin(k_total, state.data_ptr(), _stream(stream)))


def slimdp_select_hist(scores: torch.Tensor, rnd: int, state: torch.Tensor, hist: torch.Tensor, stream=None):
    """hist (int64[4096]) += this shard's keys by their digit of round rnd."""
    _dev(scores, torch.float32, "scores")
    if _dev(hist, torch.int64, "hist").numel() < 4096:
        raise ValueError("hist: 4096 counters are needed")
    _check("slimdp_select_hist", lib.slimdp_select_hist(_ptr(scores), scores.numel(), rnd, state.data_ptr(),
                                                        hist.data_ptr(), _stream(stream)))


def slimdp_select_resolve(hist: torch.Tensor, rnd: int, state: torch.Tensor, stream=None):
    _dev(hist, torch.int64, "hist")
    _check("slimdp_select_resolve", lib.slimdp_select_resolve(hist.data_ptr(), rnd, state.data_ptr(), _stream(stream)))


def slimdp_select_count(scores: torch.Tensor, state: torch.Tensor, counts: torch.Tensor, stream=None):
    """counts (int64[2]) += (keys above the threshold, keys equal to it) in this shard."""
    _dev(scores, torch.float32, "scores")
    _dev(counts, torch.int64, "counts")
    _check("slimdp_select_count", lib.slimdp_select_count(_ptr(scores), scores.numel(), state.data_ptr(),
                                                          counts.data_ptr(), _stream(stream)))


def slimdp_select_emit(scores: torch.Tensor, threshold_bits: int, tie_quota: int, core_idx: torch.Tensor,
                       core_aux: torch.Tensor, ws: torch.Tensor, stream=None):
    """This shard's part of the core (shard-local indices) for a global threshold and the shard's tie quota."""
    _dev(scores, torch.float32, "scores")
    _dev(core_idx, IDX, "core_idx")
    _check("slimdp_select_emit",
           lib.slimdp_select_emit(scores.data_ptr(), scores.numel(), threshold_bits, tie_quota, core_idx.numel(),
                                  _ptr(core_idx), core_aux.data_ptr(), ws.data_ptr(), ws.numel(), _stream(stream)))


WIRE_KEYS_WANTED = 1


def wire_message_bytes(k_core: int, k_exp: int, with_keys: bool) -> int:
    return lib.slimdp_wire_message_bytes(k_core, k_exp, int(with_keys))


def slimdp_wire_pack(core_idx: torch.Tensor, exp_idx: torch.Tensor, val: torch.Tensor, signature: torch.Tensor,
                     worker: int, rnd: int, with_keys: bool, msg: torch.Tensor, stream=None):
    """One worker's push as a message (Section 3.5) into the uint8 CUDA tensor `msg`."""
    _dev(core_idx, IDX, "core_idx")
    _dev(exp_idx, IDX, "exp_idx")
    _dev(val, torch.float32, "val")
    _dev(signature, torch.int64, "signature")
    _dev(msg, torch.uint8, "msg")
    if val.numel() != core_idx.numel() + exp_idx.numel():
        raise ValueError("val: length differs from k_core + k_exp")
    if msg.numel() != wire_message_bytes(core_idx.numel(), exp_idx.numel(), with_keys):
        raise ValueError("msg: length differs from wire_message_bytes")
    _check("slimdp_wire_pack",
           lib.slimdp_wire_pack(_ptr(core_idx), core_idx.numel(), _ptr(exp_idx), exp_idx.numel(), _ptr(val),
                                signature.data_ptr(), worker, rnd, int(with_keys), msg.data_ptr(), _stream(stream)))


def slimdp_wire_unpack(msg: torch.Tensor, cached_signature: torch.Tensor, core_idx: torch.Tensor,
                       exp_idx: torch.Tensor, val: torch.Tensor, signature_out: torch.Tensor, status: torch.Tensor,
                       stream=None):
    """Takes a push message apart; the verdict lands in status[0] (read it with wire_read_status)."""
    _dev(msg, torch.uint8, "msg")
    _dev(cached_signature, torch.int64, "cached_signature")
    _dev(signature_out, torch.int64, "signature_out")
    _dev(core_idx, IDX, "core_idx")
    _dev(exp_idx, IDX, "exp_idx")
    _dev(val, torch.float32, "val")
    if _dev(status, torch.int32, "status").numel() < 4:
        raise ValueError("status: four int32 words are needed")
    if val.numel() != core_idx.numel() + exp_idx.numel():
        raise ValueError("val: length differs from k_core + k_exp")
    _check("slimdp_wire_unpack",
           lib.slimdp_wire_unpack(msg.data_ptr(), msg.numel(), cached_signature.data_ptr(), core_idx.numel(),
                                  exp_idx.numel(), _ptr(core_idx), _ptr(exp_idx), _ptr(val),
                                  signature_out.data_ptr(), status.data_ptr(), _stream(stream)))


def wire_read_status(status: torch.Tensor, stream=None) -> int:
    """0 = taken apart, WIRE_KEYS_WANTED = the sender has to send its keys; malformed messages raise."""
    st = lib.slimdp_wire_read_status(status.data_ptr(), _stream(stream))
    if st not in (0, WIRE_KEYS_WANTED):
        raise SlimDPError("slimdp_wire_unpack", st)
    return st


def _host(t: torch.Tensor, dtype, name: str) -> torch.Tensor:
    if t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise TypeError(f"{name}: expected a contiguous host tensor of {dtype}")
    return t


def slimdp_round_host(w_host: torch.Tensor, grads_host: Sequence[torch.Tensor], c: float, k_core: int, k_exp: int,
                      seed: int, rnd: int, eta: float, core_idx_host: torch.Tensor,
                      exp_idx_host: Sequence[torch.Tensor], pulled_host: Sequence[torch.Tensor],
                      arena: torch.Tensor, stream=None):
    """One whole round on host tensors (pinned for speed); w_host is replaced by the merged model."""
    n, K = w_host.numel(), len(grads_host)
    _host(w_host, torch.float32, "w_host")
    _host(core_idx_host, IDX, "core_idx_host")
    for g, e, p in zip(grads_host, exp_idx_host, pulled_host):
        if _host(g, torch.float32, "grads_host").numel() != n:
            raise ValueError("grads_host: length differs from w_host")
        if _host(e, IDX, "exp_idx_host").numel() != k_exp:
            raise ValueError("exp_idx_host: length differs from k_exp")
        if _host(p, torch.float32, "pulled_host").numel() != k_core + k_exp:
            raise ValueError("pulled_host: length differs from k_core + k_exp")
    if core_idx_host.numel() != k_core or len(exp_idx_host) != K or len(pulled_host) != K:
        raise ValueError("output buffers do not match k_core / K")
    if not arena.is_cuda:
        raise TypeError("arena: expected a CUDA tensor")
    _check("slimdp_round_host",
           lib.slimdp_round_host(w_host.data_ptr(), _ptr_array(grads_host), K, n, c, k_core, k_exp, seed, rnd, eta,
                                 _ptr(core_idx_host), _ptr_array(exp_idx_host), _ptr_array(pulled_host),
                                 arena.data_ptr(), arena.numel() * arena.element_size(), _stream(stream)))
