"""Seeded synthetic workloads: template graphs, slot tables, field lengths, Q/K/V values.

This module only *describes inputs*.  It holds none of the method's arithmetic (no
scheduling, no closure, no masks, no attention): the CUDA path and the CPU checker
each compute those on their own from what is generated here.

The shapes follow the paper's setting: a fixed template of fields with dependencies
(Sec. 3.1-3.2), every field padded to a fixed slot (Sec. 3.3), a chain of thought of
a few hundred tokens, and a shared vision+prompt prefix whose KV all fields read.
The paper's dataset and fine-tuned models are not available, so values are i.i.d.
Gaussian from a seed.
"""
from __future__ import annotations

import dataclasses
import zlib
from typing import List, Optional, Tuple

import numpy as np
import torch

BASE_SEED = 260202864


@dataclasses.dataclass
class Workload:
    """One synthetic problem instance (template + shapes + per-scene field lengths)."""

    name: str
    dtype: str                 # "f32" | "bf16"
    layers: int
    hq: int
    hkv: int
    head_dim: int
    batch: int                 # independent scenes
    prefix_len: int            # P: shared vision+prompt rows at the head of every cache
    n_nodes: int
    edges: List[Tuple[int, int]]   # (src, dst): dst needs src complete
    slot_cap: List[int]        # C[v]: fixed slot length of field v
    n_fixed: List[int]         # pre-filled field-name tokens at the head of slot v
    max_active: int            # widest frontier the template can produce
    lens: np.ndarray           # int32 [batch][n_nodes]: valid rows of field v in scene s
    seed: int
    kv_scale: float = 1.0      # K, V = kv_scale * N(0,1); Q = N(0,1)

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    @property
    def esize(self) -> int:
        return 4 if self.dtype == "f32" else 2

    @property
    def cot_rows(self) -> int:
        return int(sum(self.slot_cap))

    @property
    def rows(self) -> int:
        return self.prefix_len + self.cot_rows

    @property
    def group(self) -> int:
        return self.hq // self.hkv

    @property
    def softmax_scale(self) -> float:
        return 1.0 / float(np.sqrt(self.head_dim))


def _fan_graph(n_par: int) -> Tuple[int, List[Tuple[int, int]]]:
    """n_par independent fields -> one summary field -> one final field."""
    edges = [(i, n_par) for i in range(n_par)] + [(n_par, n_par + 1)]
    return n_par + 2, edges


def cfg0_tiny() -> Workload:
    """Tiny fp32: root -> 4 independent children -> summary; 16-token slots; prefix 256."""
    edges = [(0, 1), (0, 2), (0, 3), (0, 4), (1, 5), (2, 5), (3, 5), (4, 5)]
    n = 6
    return Workload("cfg0_tiny_f32", "f32", 1, 4, 2, 64, 1, 256, n, edges, [16] * n, [0] * n, 4,
                    np.full((1, n), 16, np.int32), BASE_SEED + 0, 1.0)


def cfg1_7b(layers: int = 28) -> Workload:
    """7B-class bf16: 6 perception fields -> meta-action -> final; slots 64, lengths U{32..64}."""
    n, edges = _fan_graph(6)
    seed = BASE_SEED + 1
    rng = np.random.default_rng(seed)
    lens = rng.integers(32, 65, size=(1, n)).astype(np.int32)
    return Workload("cfg1_7b_bf16", "bf16", layers, 28, 4, 128, 1, 2048, n, edges, [64] * n, [0] * n, 6,
                    lens, seed, 0.5)


def cfg2_batched(layers: int = 32, batch: int = 16) -> Workload:
    """Batched scenes bf16: same template, slots 96, lengths U{16..96} drawn per scene."""
    n, edges = _fan_graph(6)
    seed = BASE_SEED + 2
    rng = np.random.default_rng(seed)
    lens = rng.integers(16, 97, size=(batch, n)).astype(np.int32)
    return Workload("cfg2_batched_bf16", "bf16", layers, 32, 8, 128, batch, 4096, n, edges, [96] * n,
                    [0] * n, 6, lens, seed, 0.5)


def cfg2_dual_response(layers: int = 32, batch: int = 16, response_len: int = 24) -> Workload:
    """The batched configuration with one more source field, decoded beside the chain of thought
    (Sec. 4.3, future work: a fast response produced concurrently with the comprehensive CoT).
    The field depends on nothing and nothing depends on it: as long as it is no longer than the
    critical path it adds width to the first passes and no pass to the schedule."""
    w = cfg2_batched(layers, batch)
    n = w.n_nodes
    lens = np.concatenate([w.lens, np.full((batch, 1), response_len, np.int32)], axis=1)
    return Workload("cfg2_dual_response_bf16", w.dtype, layers, w.hq, w.hkv, w.head_dim, batch, w.prefix_len, n + 1,
                    list(w.edges), list(w.slot_cap) + [32], list(w.n_fixed) + [0], w.max_active + 1, lens, w.seed, w.kv_scale)


def cfg3_wide(layers: int = 32, batch: int = 8) -> Workload:
    """Wide graph bf16: 16 leaves -> 2 aggregators (seeded 8-subsets) -> final; 48-token slots."""
    seed = BASE_SEED + 3
    rng = np.random.default_rng(seed)
    edges: List[Tuple[int, int]] = []
    for agg in (16, 17):
        for leaf in sorted(rng.choice(16, size=8, replace=False).tolist()):
            edges.append((int(leaf), agg))
    edges += [(16, 18), (17, 18)]
    n = 19
    return Workload("cfg3_wide_bf16", "bf16", layers, 32, 8, 128, batch, 8192, n, edges, [48] * n,
                    [0] * n, 16, np.full((batch, n), 48, np.int32), seed, 1.0)


def cfg4_sweep(prefix_len: int, branches: int, batch: int, chain: bool = False,
               point: int = 0) -> Workload:
    """Sweep point bf16: `branches` fields of 64-token slots, all independent
    (parallel schedule) or in a chain (the sequential-decode comparator)."""
    n = branches
    edges = [(i, i + 1) for i in range(n - 1)] if chain else []
    kind = "chain" if chain else "par"
    return Workload(f"cfg4_P{prefix_len}_B{branches}_Bt{batch}_{kind}", "bf16", 1, 32, 8, 128, batch,
                    prefix_len, n, edges, [64] * n, [0] * n, 1 if chain else branches,
                    np.full((batch, n), 64, np.int32), BASE_SEED + 4 + point, 0.5)


def random_template(seed: int, n_nodes: int, edge_prob: float = 0.3, cap_lo: int = 2, cap_hi: int = 9,
                    batch: int = 1, prefix_len: int = 5, fixed_hi: int = 0, hq: int = 4, hkv: int = 2,
                    head_dim: int = 64, dtype: str = "f32") -> Workload:
    """Small random template for randomized tests: edges only from lower to higher ids."""
    rng = np.random.default_rng(seed)
    edges = [(u, v) for v in range(n_nodes) for u in range(v) if rng.random() < edge_prob]
    cap = rng.integers(cap_lo, cap_hi + 1, size=n_nodes).astype(int).tolist()
    fixed = [int(rng.integers(0, min(fixed_hi, c - 1) + 1)) if fixed_hi > 0 else 0 for c in cap]
    lens = np.stack([[int(rng.integers(f + 1, c + 1)) for f, c in zip(fixed, cap)]
                     for _ in range(batch)]).astype(np.int32)
    return Workload(f"rand_{seed}", dtype, 1, hq, hkv, head_dim, batch, prefix_len, n_nodes, edges, cap,
                    fixed, n_nodes, lens, seed, 1.0)


# ----------------------------------------------------------------------------------
# values
# ----------------------------------------------------------------------------------

def _gen(seed: int, tag: str, device: str, *idx: int) -> torch.Generator:
    """A generator whose stream depends only on (seed, tag, idx, device type)."""
    h = zlib.crc32(repr((tag,) + tuple(int(i) for i in idx)).encode())
    g = torch.Generator(device=device)
    g.manual_seed((int(seed) * 1000003 + h) % (2 ** 63 - 1))
    return g


def prefix_kv(w: Workload, layer: int, device: str = "cpu",
              scenes: Optional[range] = None) -> Tuple[torch.Tensor, torch.Tensor]:
    """K and V of the shared prefix rows: two tensors [n_scenes][hkv][P][D] in w's dtype."""
    scenes = range(w.batch) if scenes is None else scenes
    ks, vs = [], []
    for s in scenes:
        g = _gen(w.seed, "prefix", device, s, layer)
        shape = (2, w.hkv, w.prefix_len, w.head_dim)
        kv = (torch.randn(shape, generator=g, device=device, dtype=torch.float32) * w.kv_scale)
        kv = kv.to(w.torch_dtype)
        ks.append(kv[0])
        vs.append(kv[1])
    return torch.stack(ks), torch.stack(vs)


def step_qkv(w: Workload, step: int, layer: int, device: str = "cpu"
             ) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    """This step's packed inputs for one layer, one row per branch slot of every scene:
    q [batch][max_active][hq][D], k_new and v_new [batch][max_active][hkv][D].
    Rows beyond a scene's active count are drawn too and must be ignored by consumers."""
    g = _gen(w.seed, "step", device, step, layer)
    q = torch.randn((w.batch, w.max_active, w.hq, w.head_dim), generator=g, device=device,
                    dtype=torch.float32).to(w.torch_dtype)
    kv = (torch.randn((2, w.batch, w.max_active, w.hkv, w.head_dim), generator=g, device=device,
                      dtype=torch.float32) * w.kv_scale).to(w.torch_dtype)
    return q, kv[0], kv[1]


def fixed_kv(w: Workload, layer: int, device: str = "cpu") -> Tuple[torch.Tensor, torch.Tensor]:
    """K and V of the pre-filled field-name rows: [batch][hkv][sum(n_fixed)][D] each, ordered
    by node id then token (empty when the template has no fixed tokens)."""
    nf = int(sum(w.n_fixed))
    g = _gen(w.seed, "fixed", device, layer)
    kv = (torch.randn((2, w.batch, w.hkv, nf, w.head_dim), generator=g, device=device,
                      dtype=torch.float32) * w.kv_scale).to(w.torch_dtype)
    return kv[0], kv[1]
