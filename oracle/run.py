"""Replay of a whole parallel-decoding run on the CPU checker.  TEST INFRASTRUCTURE ONLY.

Holds, per scene, the Algorithm 1 pass list and a float32 copy of the scene's KV cache
(exact widening of the bf16/fp32 inputs); a pass appends the new K/V rows of every
active field at their slot rows, then attends (append-then-attend, so a token sees
itself).  Small cases only: the cache lives in host memory."""
from __future__ import annotations

from typing import List, Sequence, Tuple

import numpy as np

from . import attention as _att
from . import schedule as _sch


class OracleRun:
    def __init__(self, n: int, edges: Sequence[Tuple[int, int]], slot_cap: Sequence[int],
                 n_fixed: Sequence[int], prefix_len: int, lens: np.ndarray, layers: int,
                 hq: int, hkv: int, head_dim: int, scale: float, max_active: int):
        self.n, self.edges = n, list(edges)
        self.slot_cap, self.n_fixed = list(slot_cap), list(n_fixed)
        self.P = prefix_len
        self.lens = np.asarray(lens)
        self.batch = self.lens.shape[0]
        self.L, self.hq, self.hkv, self.D = layers, hq, hkv, head_dim
        self.scale, self.max_active = scale, max_active
        self.base = _sch.slot_base(slot_cap)
        self.R = prefix_len + self.base[n]
        self.passes: List[List[List[Tuple[int, int]]]] = [
            _sch.simulate(n, edges, self.lens[s].tolist(), n_fixed) for s in range(self.batch)]
        self.n_steps = max(len(p) for p in self.passes)
        self.K = np.full((self.batch, layers, hkv, self.R, head_dim), np.nan, dtype=np.float32)
        self.V = np.full_like(self.K, np.nan)   # rows never written stay NaN: reading one shows up

    def active(self, s: int, step: int) -> List[Tuple[int, int]]:
        return self.passes[s][step] if step < len(self.passes[s]) else []

    def tables(self, s: int, step: int):
        return _sch.pass_tables(self.n, self.edges, self.slot_cap, self.lens[s].tolist(), self.n_fixed,
                                self.P, self.active(s, step))

    def write_prefix(self, layer: int, K: np.ndarray, V: np.ndarray) -> None:
        """K, V: [batch][hkv][P][D]"""
        self.K[:, layer, :, :self.P] = K
        self.V[:, layer, :, :self.P] = V

    def write_fixed(self, layer: int, K: np.ndarray, V: np.ndarray) -> None:
        """K, V: [batch][hkv][sum n_fixed][D], ordered by node then token."""
        i = 0
        for v in range(self.n):
            for j in range(self.n_fixed[v]):
                r = _sch.kv_row(self.P, self.base, v, j)
                self.K[:, layer, :, r] = K[:, :, i]
                self.V[:, layer, :, r] = V[:, :, i]
                i += 1

    def append(self, step: int, layer: int, k_new: np.ndarray, v_new: np.ndarray) -> None:
        """k_new, v_new: [batch][max_active][hkv][D]; branch b of scene s goes to its slot row."""
        for s in range(self.batch):
            for b, (v, t) in enumerate(self.active(s, step)):
                r = _sch.kv_row(self.P, self.base, v, t)
                self.K[s, layer, :, r] = k_new[s, b]
                self.V[s, layer, :, r] = v_new[s, b]

    def attend(self, step: int, layer: int, q: np.ndarray, nthreads: int = 0) -> np.ndarray:
        """q [batch][max_active][hq][D] -> float64 same shape (rows of idle branch slots = 0)."""
        out = np.zeros((self.batch, self.max_active, self.hq, self.D), dtype=np.float64)
        for s in range(self.batch):
            tab = self.tables(s, step)
            A = len(tab["node"])
            if A:
                out[s, :A] = _att.attention(q[s, :A], self.K[s, layer], self.V[s, layer], tab["vis"],
                                            self.scale, nthreads)
        return out
