"""Seeded generation of the global weights and the per-worker updates.

Every tensor is produced in fixed chunks of CHUNK elements, each chunk from
its own numpy Generator seeded with (config seed, tensor id, worker, chunk
index), so any slice [start, stop) can be regenerated on its own and the
values do not depend on how the caller splits the work.
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
import os
from typing import List, Optional

import numpy as np

from .configs import Config

CHUNK = 1 << 22
_TENSOR_W = 0
_TENSOR_G = 1


def _scale_by_segment(cfg: Config, x: np.ndarray, a: int, b: int, mult: float, for_weights: bool) -> None:
    """x holds standard-normal draws for parameters [a, b); scale in place."""
    for lo, hi, seg in cfg.bounds():
        if hi <= a or lo >= b:
            continue
        s, e = max(lo, a) - a, min(hi, b) - a
        if for_weights:
            if seg.kind == "weight":
                x[s:e] *= np.float32(seg.sigma)
            elif seg.kind == "one":
                x[s:e] = 1.0
            else:
                x[s:e] = 0.0
        else:
            x[s:e] *= np.float32(seg.sigma * mult)


def _chunk(cfg: Config, tensor: int, worker: int, ci: int) -> np.ndarray:
    a = ci * CHUNK
    b = min(a + CHUNK, cfg.N)
    rng = np.random.default_rng([cfg.seed, tensor, worker, ci])
    n = CHUNK      # always a whole chunk, so a prefix of a config sees the same draws
    if tensor == _TENSOR_W:
        x = rng.standard_normal(n, dtype=np.float32)[:b - a]
        _scale_by_segment(cfg, x, a, b, 1.0, True)
        if cfg.quantise:
            x = (np.clip(np.rint(x * np.float32(512.0)), -128, 127) * np.float32(2.0 ** -9)).astype(np.float32)
        return x
    if cfg.grad_dist == "normal":
        x = rng.standard_normal(n, dtype=np.float32)[:b - a]
        x *= np.float32(cfg.grad_scale)
    elif cfg.grad_dist == "normal_layer":
        x = rng.standard_normal(n, dtype=np.float32)[:b - a]
        _scale_by_segment(cfg, x, a, b, cfg.grad_scale, False)
    elif cfg.grad_dist == "laplace":
        # Laplace(0, b) as b * (E1 - E2), E1 and E2 independent Exp(1)
        x = rng.standard_exponential(n, dtype=np.float32)
        x -= rng.standard_exponential(n, dtype=np.float32)
        x = x[:b - a]
        x *= np.float32(cfg.grad_scale)
    else:
        raise ValueError(cfg.grad_dist)
    if cfg.quantise:
        x = (np.clip(np.rint(x * np.float32(65536.0)), -128, 127) * np.float32(2.0 ** -16)).astype(np.float32)
    return x


def _tensor(cfg: Config, tensor: int, worker: int, start: int, stop: Optional[int],
            out: Optional[np.ndarray] = None, pool: Optional[ThreadPoolExecutor] = None) -> np.ndarray:
    stop = cfg.N if stop is None else stop
    if not (0 <= start <= stop <= cfg.N):
        raise ValueError("slice out of range")
    if out is None:
        out = np.empty(stop - start, dtype=np.float32)
    if stop == start:
        return out

    def job(ci: int) -> None:
        a = ci * CHUNK
        x = _chunk(cfg, tensor, worker, ci)
        lo, hi = max(a, start), min(a + x.size, stop)
        out[lo - start:hi - start] = x[lo - a:hi - a]

    cis = range(start // CHUNK, (stop - 1) // CHUNK + 1)
    if pool is None:
        for ci in cis:
            job(ci)
    else:
        list(pool.map(job, cis))
    return out


def weights(cfg: Config, start: int = 0, stop: Optional[int] = None, out=None, pool=None) -> np.ndarray:
    """Global model w-bar[start:stop] as float32."""
    return _tensor(cfg, _TENSOR_W, 0, start, stop, out, pool)


def grads(cfg: Config, worker: int, start: int = 0, stop: Optional[int] = None, out=None, pool=None) -> np.ndarray:
    """Worker `worker`'s accumulated update delta_k[start:stop] as float32."""
    if not (0 <= worker < cfg.K):
        raise ValueError("worker out of range")
    return _tensor(cfg, _TENSOR_G, worker, start, stop, out, pool)


def all_inputs(cfg: Config, threads: Optional[int] = None):
    """(w, [delta_0 .. delta_{K-1}]) for the whole config, generated with a thread pool."""
    threads = threads or min(16, os.cpu_count() or 1)
    with ThreadPoolExecutor(threads) as pool:
        w = weights(cfg, pool=pool)
        g: List[np.ndarray] = [grads(cfg, k, pool=pool) for k in range(cfg.K)]
    return w, g
