"""Algorithm 1's communication schedule on the device: which C-ABI call runs in which round.

The object holds the global model, the K workers' local models and the buffers of a round;
`round(deltas)` takes the K accumulated updates of one communication (local training is the
caller's business) and enqueues, on the current stream:
  exploration for round t; the dense push + update + scoring if (t + 1) % q == 0, else the
  fused push / update / pull on the communication set; the pull (after a dense push); the
  worker-side merge; and after a dense push the reselection of the core for the rounds to come.
Before the first reselection the core is chosen from the initial model's magnitudes alone.
Call order and buffer ownership only; every step is one library call.
"""
from __future__ import annotations

from typing import List, Sequence

import torch

from . import binding as B
from .round import RoundBuffers


class SlimDPDriver:
    def __init__(self, w0: torch.Tensor, K: int, k_core: int, k_exp: int, q: int, c: float, eta: float, seed: int):
        if q < 1:
            raise ValueError("q must be at least 1")
        self.w = w0.clone()
        self.n, self.K, self.k_core, self.k_exp, self.q = w0.numel(), K, k_core, k_exp, q
        self.c, self.eta, self.seed, self.t = c, eta, seed, 0
        self.local: List[torch.Tensor] = [w0.clone() for _ in range(K)]
        self.buf = RoundBuffers(self.n, K, k_core, k_exp, w0.device)
        zero = torch.zeros_like(w0)
        B.slimdp_score(self.w, [zero], c, self.buf.scores)
        self._reselect()

    def _reselect(self) -> None:
        b = self.buf
        B.slimdp_select_core(b.scores, self.k_core, b.core_idx, b.core_aux, b.select_ws)

    def round(self, deltas: Sequence[torch.Tensor]) -> None:
        b, t = self.buf, self.t
        B.slimdp_sample_explore_batched(b.core_aux, self.n, self.k_core, self.k_exp, self.seed, 0, t, b.exp_idx,
                                        b.explore_ws)
        boundary = (t + 1) % self.q == 0
        if boundary:
            B.slimdp_dense_merge_score(self.w, deltas, self.eta, self.c, b.scores)
            B.slimdp_pull_batched(self.w, b.core_idx, b.exp_idx, b.pulled)
        else:
            B.slimdp_exchange(self.w, deltas, b.core_idx, b.exp_idx, self.eta, b.val, b.pulled)
        B.slimdp_worker_merge_batched(self.local, b.core_idx, b.exp_idx, b.pulled)
        self.t = t + 1
        if boundary:
            self._reselect()

    def check(self) -> None:
        """Synchronises and raises if a device-side consistency check failed."""
        B.read_status(self.buf.select_ws)
        B.read_status(self.buf.explore_ws)
