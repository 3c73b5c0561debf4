"""Exact-integer checker: field DAG, Algorithm 1 schedule, slots, visibility, bitmaps.

TEST INFRASTRUCTURE ONLY (see the package docstring).  Notation follows the paper:
G = (V, E); the ready set S of Algorithm 1 is, in every pass, the set of unfinished fields whose
prerequisites have all finished.

Readings taken where the paper is silent (Sec. 3.2 - 3.3 leave these open):
  * a newly ready field first decodes in the NEXT forward pass (Alg. 1: decoding is the
    first statement of the next loop iteration);
  * within a pass fields are packed in ascending node id;
  * a field is finished when it has produced len[v] rows (len[v] <= slot C[v], truncation,
    Sec. 3.3); rows len[v]..C[v]-1 of its slot are padding;
  * the KV row and position id of token t of field v is P + base[v] + t with
    base[v] = sum of C[u] for u < v (fixed slots make later positions known, Sec. 3.3);
  * a token attends to itself (append, then attend), so a chain template is ordinary
    causal decoding;
  * the first n_fixed[v] rows of a slot are the pre-filled field-name tokens: visible to
    every query at a higher row whatever the dependencies (Sec. 3.3, Fig. 3 caption);
    the generated tokens of v start at t = n_fixed[v].
"""
from __future__ import annotations

from typing import Dict, List, Sequence, Set, Tuple

import numpy as np

TILE_ROWS = 64  # rows per KV tile of the visited-tile list (an interface constant)


class GraphError(ValueError):
    pass


def validate(n: int, edges: Sequence[Tuple[int, int]]) -> None:
    """Node ids in range, no self loops, no directed cycle (Sec. 3.2: the graph is a DAG)."""
    for (a, b) in edges:
        if not (0 <= a < n and 0 <= b < n):
            raise GraphError("node id out of range")
        if a == b:
            raise GraphError("cycle")
    # colour-marking depth-first search
    succ: Dict[int, List[int]] = {v: [] for v in range(n)}
    for (a, b) in edges:
        succ[a].append(b)
    colour = [0] * n

    def visit(v: int) -> None:
        colour[v] = 1
        for u in succ[v]:
            if colour[u] == 1:
                raise GraphError("cycle")
            if colour[u] == 0:
                visit(u)
        colour[v] = 2

    for v in range(n):
        if colour[v] == 0:
            visit(v)


def ancestors(n: int, edges: Sequence[Tuple[int, int]]) -> List[Set[int]]:
    """Eq. 1: A is an ancestor of B iff a directed path A -> ... -> B exists.
    Found by walking parent links backwards from each node (depth-first)."""
    validate(n, edges)
    parents: List[List[int]] = [[] for _ in range(n)]
    for (a, b) in edges:
        parents[b].append(a)
    out: List[Set[int]] = []
    for v in range(n):
        seen: Set[int] = set()
        stack = list(parents[v])
        while stack:
            u = stack.pop()
            if u not in seen:
                seen.add(u)
                stack.extend(parents[u])
        out.append(seen)
    return out


def slot_base(slot_cap: Sequence[int]) -> List[int]:
    """base[v] = sum_{u<v} C[u]; base[n] = T, the rows the whole template reserves."""
    base = [0]
    for c in slot_cap:
        base.append(base[-1] + int(c))
    return base


def simulate(n: int, edges: Sequence[Tuple[int, int]], lens: Sequence[int],
             n_fixed: Sequence[int] | None = None) -> List[List[Tuple[int, int]]]:
    """The schedule Algorithm 1 (Sec. 3.2) produces, written as its defining property instead of
    the listing's bookkeeping: in every forward pass exactly those fields decode one token that
    are unfinished and whose prerequisites had all finished BEFORE the pass; a field is finished
    once it holds lens[v] rows.  Returns, per forward pass, the packed list of (v, t): field v
    decodes its token t in that pass (ascending v)."""
    validate(n, edges)
    n_fixed = [0] * n if n_fixed is None else list(n_fixed)
    for v in range(n):
        if not (n_fixed[v] + 1 <= lens[v]):
            raise GraphError("every field must generate at least one token")
    parents: List[List[int]] = [[a for (a, b) in edges if b == v] for v in range(n)]
    rows = [n_fixed[v] for v in range(n)]         # rows of v already in the cache
    passes: List[List[Tuple[int, int]]] = []
    while True:
        finished = [rows[v] == lens[v] for v in range(n)]          # state before this pass
        ready = [v for v in range(n) if not finished[v] and all(finished[u] for u in parents[v])]
        if not ready:
            break
        passes.append([(v, rows[v]) for v in ready])
        for v in ready:
            rows[v] += 1
    if any(rows[v] != lens[v] for v in range(n)):
        raise GraphError("schedule did not complete")
    return passes


def critical_path(n: int, edges: Sequence[Tuple[int, int]], weight: Sequence[int]) -> Tuple[int, List[int]]:
    """Sec. 3.2: the minimum number of forward passes equals the largest cumulative
    number of tokens along any dependency chain.  finish[v] = weight[v] + max over parents."""
    validate(n, edges)
    parents: List[List[int]] = [[] for _ in range(n)]
    for (a, b) in edges:
        parents[b].append(a)
    finish: Dict[int, int] = {}

    def f(v: int) -> int:
        if v not in finish:
            finish[v] = int(weight[v]) + max([f(p) for p in parents[v]], default=0)
        return finish[v]

    return max(f(v) for v in range(n)), [f(v) for v in range(n)]


def kv_row(prefix_len: int, base: Sequence[int], v: int, t: int) -> int:
    """Cache row (= position id) of token t of field v (Sec. 3.3: fixed slots)."""
    return prefix_len + base[v] + t


def visible_rows(n: int, anc: Sequence[Set[int]], slot_cap: Sequence[int], lens: Sequence[int],
                 n_fixed: Sequence[int], prefix_len: int, v: int, t: int) -> np.ndarray:
    """bool[R]: which cache rows the query (field v, token t) may attend.

    prefix: always.  Field u's row j: visible iff u is an ancestor of v and j is a real
    (non-padding) token of u (Eq. 1 + invisible padding), or u == v and j <= t (causal
    within the field), or j is a fixed field-name token at a lower row than the query."""
    base = slot_base(slot_cap)
    R = prefix_len + base[n]
    vis = np.zeros(R, dtype=bool)
    vis[:prefix_len] = True
    q_row = kv_row(prefix_len, base, v, t)
    for u in range(n):
        r0 = kv_row(prefix_len, base, u, 0)
        if u in anc[v]:
            vis[r0:r0 + lens[u]] = True          # real tokens of an ancestor, never its padding
        if u == v:
            vis[r0:r0 + t + 1] = True            # own tokens up to and including this one
        for j in range(n_fixed[u]):              # pre-filled field-name tokens at lower rows
            if r0 + j < q_row:
                vis[r0 + j] = True
    return vis


def pack_bits(vis_cot: np.ndarray) -> np.ndarray:
    """bool[T] -> uint64[ceil(T/64)], bit i of word w <-> template row 64*w + i."""
    T = vis_cot.shape[0]
    W = (T + 63) // 64
    padded = np.zeros(W * 64, dtype=np.uint8)
    padded[:T] = vis_cot
    return np.packbits(padded, bitorder="little").view("<u8").astype(np.uint64)


def pass_tables(n: int, edges: Sequence[Tuple[int, int]], slot_cap: Sequence[int], lens: Sequence[int],
                n_fixed: Sequence[int], prefix_len: int, this_pass: Sequence[Tuple[int, int]]):
    """Everything the path derives for one scene in one forward pass:
    node, tok_idx, kv_row (= pos_id), per-branch visibility bool[A][R], per-branch bitmap
    words uint64[A][W], union bitmap uint64[W] and the ascending list of visited tiles."""
    anc = ancestors(n, edges)
    base = slot_base(slot_cap)
    T = base[n]
    R = prefix_len + T
    W = (T + 63) // 64
    A = len(this_pass)
    node = np.array([v for (v, _) in this_pass], dtype=np.int32)
    tok_idx = np.array([t for (_, t) in this_pass], dtype=np.int32)
    rows = np.array([kv_row(prefix_len, base, v, t) for (v, t) in this_pass], dtype=np.int32)
    vis = np.zeros((A, R), dtype=bool)
    mask = np.zeros((A, W), dtype=np.uint64)
    for b, (v, t) in enumerate(this_pass):
        vis[b] = visible_rows(n, anc, slot_cap, lens, n_fixed, prefix_len, v, t)
        mask[b] = pack_bits(vis[b, prefix_len:])
    union = vis.any(axis=0) if A else np.zeros(R, dtype=bool)
    umask = pack_bits(union[prefix_len:])
    ntile = (R + TILE_ROWS - 1) // TILE_ROWS
    tiles = np.array([i for i in range(ntile) if union[i * TILE_ROWS:(i + 1) * TILE_ROWS].any()],
                     dtype=np.int32)
    return dict(node=node, tok_idx=tok_idx, kv_row=rows, pos_id=rows.copy(), vis=vis, mask=mask,
                umask=umask, tiles=tiles)


def average_parallel_degree(passes: Sequence[Sequence[Tuple[int, int]]]) -> float:
    """Sec. 4.3: tokens processed per forward pass, averaged over the run."""
    return sum(len(p) for p in passes) / float(len(passes))
