"""A host stand-in for the CUDA steps of the sharded selection (test infrastructure): the same five
calls on CPU tensors, written with numpy from the definition of the radix rounds (digits of 12, 10
and 10 bits of the keys' bit patterns, most significant first).  Lets the host logic of
paper_1709_09393_b200/sharded.py run under gloo without a GPU."""
import numpy as np
import torch

SHIFT = (20, 10, 0)
BINS = (4096, 1024, 1024)


class NumpyBackend:
    def new_state(self, device):
        return torch.zeros(2, dtype=torch.int64)

    def begin(self, k_total, state):
        state[0] = 0            # low word: prefix, high word: status
        state[1] = k_total

    def _keys(self, scores):
        return scores.numpy().view(np.uint32)

    def hist(self, scores, rnd, state, hist):
        keys = self._keys(scores)
        prefix = int(state[0]) & 0xFFFFFFFF
        if rnd > 0:
            above = 32 - (12 if rnd == 1 else 22)              # bits already fixed: 12 after round 0, 22 after round 1
            keys = keys[(keys >> above) == (prefix >> above)]
        digit = (keys >> SHIFT[rnd]) & (BINS[rnd] - 1)
        hist[:BINS[rnd]] += torch.from_numpy(np.bincount(digit, minlength=BINS[rnd]).astype(np.int64))

    def resolve(self, hist, rnd, state):
        h = hist[:BINS[rnd]].numpy()
        want = int(state[1])
        from_top = np.cumsum(h[::-1])
        pos = int(np.searchsorted(from_top, want))            # first bin (from the top) where the count reaches `want`
        if pos >= BINS[rnd]:
            state[0] = int(state[0]) | (0xFFFFFFFC << 32)      # status -4 in the high word
            return
        b = BINS[rnd] - 1 - pos
        state[0] = (int(state[0]) & 0xFFFFFFFF) | (b << SHIFT[rnd])
        state[1] = want - (int(from_top[pos - 1]) if pos else 0)

    def count(self, scores, state, counts):
        keys = self._keys(scores)
        T = int(state[0]) & 0xFFFFFFFF
        counts[0] += int((keys > T).sum())
        counts[1] += int((keys == T).sum())

    def read_state(self, state):
        raw = int(state[0]) & 0xFFFFFFFFFFFFFFFF
        status = (raw >> 32) & 0xFFFFFFFF
        return raw & 0xFFFFFFFF, int(state[1]), (status - (1 << 32)) if status >> 31 else status

    def emit(self, scores, threshold_bits, quota, k_shard):
        keys = self._keys(scores)
        core = np.sort(np.concatenate([np.flatnonzero(keys > threshold_bits),
                                       np.flatnonzero(keys == threshold_bits)[:quota]])).astype(np.uint32)
        assert core.size == k_shard
        return torch.from_numpy(core.view(np.int32)), None
