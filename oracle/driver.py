"""Algorithm 1 of the paper as a plain loop over the oracle's steps (test infrastructure).

One object plays the parameter server and the K workers' communication side; local training is
outside (the caller supplies each round's accumulated updates delta_k).  Readings, in the
paper's order:
  * before the first reselection the core comes from the initial model alone (scores with a
    zero gradient, i.e. pure magnitude): Algorithm 1 uses T_S from round 0 on but only defines
    it at t % q == 0;
  * worker, round t: Exploration, then Push(delta) if (t + 1) % q == 0 else Push(T_C(delta)),
    then Pull(T_C(w-bar)) with the communication set formed BEFORE the push, then Merge;
  * server: Update with what was pushed, t <- t + 1, and if t % q == 0 Core-Selection on the
    UPDATED model with the updates just pushed densely (Section 3.3 step 6).
"""
from __future__ import annotations

from typing import List, Sequence

import numpy as np

import oracle


class Driver:
    def __init__(self, w0: np.ndarray, K: int, k_core: int, k_exp: int, q: int, c: float, eta: float, seed: int):
        self.w = np.ascontiguousarray(w0, dtype=np.float32).copy()
        self.n, self.K, self.k_core, self.k_exp, self.q = self.w.size, K, k_core, k_exp, q
        self.c, self.eta, self.seed, self.t = c, eta, seed, 0
        self.local = [self.w.copy() for _ in range(K)]          # w_k^0 <- Pull(w-bar^0)
        zero = np.zeros(self.n, np.float32)
        self.core = oracle.select_core(oracle.score(self.w, [zero], c), k_core)
        self.exp: List[np.ndarray] = []
        self.pulled: List[np.ndarray] = []

    def round(self, deltas: Sequence[np.ndarray]) -> None:
        K, t = self.K, self.t
        self.exp = [oracle.sample_explore(self.core, self.n, self.k_exp, self.seed, k, t) for k in range(K)]
        boundary = (t + 1) % self.q == 0
        if boundary:
            self.w = oracle.dense_merge(self.w, deltas, self.eta)
        else:
            val = [oracle.pack(deltas[k], self.core, self.exp[k]) for k in range(K)]
            self.w = oracle.merge(self.w, self.core, self.exp, val, self.eta)
        self.pulled = [oracle.pull(self.w, self.core, self.exp[k]) for k in range(K)]
        self.local = [oracle.worker_merge(self.local[k], self.core, self.exp[k], self.pulled[k]) for k in range(K)]
        self.t = t + 1
        if boundary:
            self.core = oracle.select_core(oracle.score(self.w, deltas, self.c), self.k_core)
