"""Core selection over a range-sharded model (Section 2.1's parameter server with the global model
cut into contiguous shards, one per GPU): the call order and the two small reductions between the
selection's steps.  Host logic only; every step on the data is a call of the `backend`.

One process per shard under torch.distributed: the histograms are summed with all_reduce, the
per-shard counts collected with all_gather (NCCL on device tensors, gloo on host tensors).
Without a process group the same code walks a list of shards in one process.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import torch


def shard_bounds(n: int, shards: int) -> List[Tuple[int, int]]:
    """Contiguous index ranges [begin, end) of the shards; the first n % shards shards hold one more."""
    q, r = divmod(n, shards)
    out, at = [], 0
    for g in range(shards):
        size = q + (1 if g < r else 0)
        out.append((at, at + size))
        at += size
    return out


def tie_quotas(greater: Sequence[int], equal: Sequence[int], k_total: int) -> List[int]:
    """How many of its keys equal to the threshold each shard admits: ties go to the smaller global
    index and shards are ascending index ranges, so the r = k_total - sum(greater) admitted ties are
    handed out to the shards in order."""
    r = k_total - sum(greater)
    if r < 0 or r > sum(equal):
        raise ValueError("counts do not match the threshold")
    out = []
    for e in equal:
        take = min(e, r)
        out.append(take)
        r -= take
    return out


class CudaBackend:
    """The steps on one shard's scores as calls of the CUDA library."""

    def __init__(self):
        from . import binding as B
        self.B = B

    def new_state(self, device):
        return torch.zeros(2, dtype=torch.int64, device=device)

    def begin(self, k_total, state):
        self.B.slimdp_select_shard_begin(k_total, state)

    def hist(self, scores, rnd, state, hist):
        self.B.slimdp_select_hist(scores, rnd, state, hist)

    def resolve(self, hist, rnd, state):
        self.B.slimdp_select_resolve(hist, rnd, state)

    def count(self, scores, state, counts):
        self.B.slimdp_select_count(scores, state, counts)

    def read_state(self, state):
        """(threshold bits, tie rank r, status) after the last round."""
        host = state.cpu().numpy()
        return int(host.view("uint32")[0]), int(host.view("uint64")[1]), int(host.view("int32")[1])

    def emit(self, scores, threshold_bits, quota, k_shard):
        B = self.B
        n = scores.numel()
        core_idx = torch.empty(k_shard, dtype=B.IDX, device=scores.device)
        core_aux = torch.empty(B.core_aux_bytes(n), dtype=torch.uint8, device=scores.device)
        ws = torch.empty(B.select_workspace_bytes(n), dtype=torch.uint8, device=scores.device)
        B.slimdp_select_emit(scores, threshold_bits, quota, core_idx, core_aux, ws)
        B.read_status(ws)
        return core_idx, core_aux


def select_core_sharded(local_scores: Sequence[torch.Tensor], k_total: int, backend, group=None):
    """Exact global top-k_total over the concatenation of all shards' scores.

    local_scores: the scores of the shards THIS process holds, in ascending shard order (one per
    process under torch.distributed; all of them in a single process).  Returns, per local shard,
    (core_idx with shard-local indices, core_aux, k_shard)."""
    import torch.distributed as dist
    distributed = dist.is_available() and dist.is_initialized()
    device = local_scores[0].device
    state = backend.new_state(device)
    backend.begin(k_total, state)
    for rnd in range(3):
        hist = torch.zeros(4096, dtype=torch.int64, device=device)
        for s in local_scores:
            backend.hist(s, rnd, state, hist)
        if distributed:
            dist.all_reduce(hist, op=dist.ReduceOp.SUM, group=group)
        backend.resolve(hist, rnd, state)
    threshold, r, status = backend.read_state(state)
    if status != 0:
        raise RuntimeError("sharded selection: the summed histograms hold fewer keys than k_total")
    local_counts = []
    for s in local_scores:
        c = torch.zeros(2, dtype=torch.int64, device=device)
        backend.count(s, state, c)
        local_counts.append(c)
    mine = torch.stack(local_counts)                                    # [local shards, 2]
    if distributed:
        world = dist.get_world_size(group)
        gathered = [torch.zeros_like(mine) for _ in range(world)]
        dist.all_gather(gathered, mine, group=group)
        all_counts = torch.cat(gathered).cpu().tolist()
        first = dist.get_rank(group) * len(local_scores)
    else:
        all_counts = mine.cpu().tolist()
        first = 0
    greater = [int(c[0]) for c in all_counts]
    equal = [int(c[1]) for c in all_counts]
    if k_total - sum(greater) != r:
        raise RuntimeError("sharded selection: counts disagree with the resolved rank")
    quotas = tie_quotas(greater, equal, k_total)
    out = []
    for j, s in enumerate(local_scores):
        g = first + j
        k_shard = greater[g] + quotas[g]
        core_idx, core_aux = backend.emit(s, threshold, quotas[g], k_shard)
        out.append((core_idx, core_aux, k_shard))
    return out
