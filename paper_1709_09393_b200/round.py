"""Buffers for one communication round and the call sequence of the round
(score, select, K x explore, K x pack, merge, K x pull).  Allocation and
call order only; each step is one C-ABI call."""
from __future__ import annotations

from typing import List, Sequence

import torch

from . import binding as B


class RoundBuffers:
    """Device buffers one round needs for n parameters, K workers and the
    integer set sizes k_core, k_exp.  Allocated once, reused every round."""

    def __init__(self, n: int, K: int, k_core: int, k_exp: int, device="cuda", staging: bool = False):
        self.n, self.K, self.k_core, self.k_exp = n, K, k_core, k_exp
        m = k_core + k_exp
        dev = torch.device(device)
        self.scores = torch.empty(n, dtype=torch.float32, device=dev)
        self.core_idx = torch.empty(k_core, dtype=B.IDX, device=dev)
        self.core_aux = torch.empty(B.core_aux_bytes(n), dtype=torch.uint8, device=dev)
        self.select_ws = torch.empty(B.select_workspace_bytes(n), dtype=torch.uint8, device=dev)
        self.explore_ws = torch.empty(B.explore_workspace_bytes(n, k_exp, K), dtype=torch.uint8, device=dev)
        # the one-call round's optional staging area (off by default: on the measured workloads the pass
        # loses more by filling it than the exchange gains by streaming it)
        stage_bytes = B.round_stage_bytes(n, K, k_core) if staging else 0
        self.stage = torch.empty(stage_bytes, dtype=torch.uint8, device=dev) if stage_bytes else None
        self.exp_idx: List[torch.Tensor] = [torch.empty(k_exp, dtype=B.IDX, device=dev) for _ in range(K)]
        self.val: List[torch.Tensor] = [torch.empty(m, dtype=torch.float32, device=dev) for _ in range(K)]
        self.pulled: List[torch.Tensor] = [torch.empty(m, dtype=torch.float32, device=dev) for _ in range(K)]


def run_round(w: torch.Tensor, grads: Sequence[torch.Tensor], c: float, seed: int, rnd: int, eta: float,
              buf: RoundBuffers, with_score: bool = True, fused_exchange: bool = True,
              overlapped: bool = False) -> None:
    """Enqueue one round on the current stream; w is merged in place.  fused_exchange selects
    slimdp_exchange over the three separate calls, overlapped the single slimdp_round call
    over the sequence of calls (identical results in every case)."""
    n, k_core, k_exp = buf.n, buf.k_core, buf.k_exp
    if overlapped:
        if not with_score:
            raise ValueError("slimdp_round always scores")
        B.slimdp_round(w, grads, c, seed, rnd, eta, buf.scores, buf.core_idx, buf.core_aux, buf.exp_idx, buf.val,
                       buf.pulled, buf.select_ws, buf.explore_ws, buf.stage)
        return
    if with_score:
        B.slimdp_score(w, grads, c, buf.scores)
    B.slimdp_select_core(buf.scores, k_core, buf.core_idx, buf.core_aux, buf.select_ws)
    B.slimdp_sample_explore_batched(buf.core_aux, n, k_core, k_exp, seed, 0, rnd, buf.exp_idx, buf.explore_ws)
    if fused_exchange:
        B.slimdp_exchange(w, grads, buf.core_idx, buf.exp_idx, eta, buf.val, buf.pulled)
        return
    B.slimdp_pack_batched(grads, buf.core_idx, buf.exp_idx, buf.val)
    B.slimdp_merge(w, buf.core_idx, buf.exp_idx, buf.val, eta)
    B.slimdp_pull_batched(w, buf.core_idx, buf.exp_idx, buf.pulled)
