"""Pins of the integer checker (oracle/schedule.py) against things other than itself:
brute-force path enumeration, boolean matrix powers, the closed-form critical path
(Sec. 3.2), hand-derived fixtures, and structural invariants."""
import itertools
import os

import numpy as np
import pytest

from oracle import schedule as sch
from paper_2602_02864_b200 import workloads as wl

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _paths_exist_bruteforce(n, edges, a, b):
    """Is there a directed path a -> ... -> b?  Enumerate node sequences explicitly."""
    E = set(edges)
    for k in range(2, n + 1):
        for mid in itertools.permutations([x for x in range(n) if x not in (a, b)], k - 2):
            seq = (a,) + mid + (b,)
            if all((seq[i], seq[i + 1]) in E for i in range(len(seq) - 1)):
                return True
    return False


def _all_small_dags(n):
    pairs = [(u, v) for v in range(n) for u in range(v)]
    for bits in range(1 << len(pairs)):
        yield [pairs[i] for i in range(len(pairs)) if bits >> i & 1]


@pytest.mark.parametrize("n", [1, 2, 3, 4, 5])
def test_closure_bruteforce_all_small_dags(n):
    perm = list(range(n))[::-1]  # also exercise edges that go from higher to lower ids
    for edges in _all_small_dags(n):
        for relabel in (False, True):
            e = [(perm[a], perm[b]) for a, b in edges] if relabel else edges
            anc = sch.ancestors(n, e)
            for a in range(n):
                for b in range(n):
                    want = a != b and _paths_exist_bruteforce(n, e, a, b)
                    assert (a in anc[b]) == want, (e, a, b)


def test_closure_matrix_power_random():
    for seed in range(300):
        w = wl.random_template(seed, n_nodes=2 + seed % 11, edge_prob=0.25)
        n = w.n_nodes
        adj = np.zeros((n, n), dtype=np.int64)
        for a, b in w.edges:
            adj[a, b] = 1
        reach = np.zeros_like(adj)
        power = np.eye(n, dtype=np.int64)
        for _ in range(n):
            power = (power @ adj > 0).astype(np.int64)
            reach |= power
        anc = sch.ancestors(n, w.edges)
        for b in range(n):
            assert anc[b] == {a for a in range(n) if reach[a, b]}
            assert b not in anc[b]                       # irreflexive
            for a in anc[b]:                             # transitive
                assert anc[a] <= anc[b]


def test_validate_rejects_cycles_and_ranges():
    with pytest.raises(sch.GraphError):
        sch.validate(3, [(0, 1), (1, 2), (2, 0)])
    with pytest.raises(sch.GraphError):
        sch.validate(2, [(0, 0)])
    with pytest.raises(sch.GraphError):
        sch.validate(2, [(0, 2)])
    with pytest.raises(sch.GraphError):
        sch.validate(4, [(0, 1), (1, 2), (2, 3), (3, 1)])
    sch.validate(4, [(0, 1), (0, 2), (1, 3), (2, 3)])


def _longest_chain_bruteforce(n, edges, weight):
    """max over every directed path of the summed weights (explicit enumeration)."""
    succ = {v: [b for a, b in edges if a == v] for v in range(n)}
    best = 0

    def walk(v, acc):
        nonlocal best
        acc += weight[v]
        best = max(best, acc)
        for u in succ[v]:
            walk(u, acc)

    for v in range(n):
        walk(v, 0)
    return best


def test_step_count_is_critical_path_random():
    """Sec. 3.2: #forward passes == largest cumulative token count along a chain."""
    for seed in range(200):
        w = wl.random_template(1000 + seed, n_nodes=1 + seed % 9, edge_prob=0.35, fixed_hi=seed % 3)
        lens = w.lens[0].tolist()
        weight = [l - f for l, f in zip(lens, w.n_fixed)]
        passes = sch.simulate(w.n_nodes, w.edges, lens, w.n_fixed)
        steps, finish = sch.critical_path(w.n_nodes, w.edges, weight)
        assert len(passes) == steps == _longest_chain_bruteforce(w.n_nodes, w.edges, weight)
        # field v is active exactly on passes finish[v]-weight[v]+1 .. finish[v] (1-based)
        for v in range(w.n_nodes):
            on = [k + 1 for k, p in enumerate(passes) if any(x == v for x, _ in p)]
            assert on == list(range(finish[v] - weight[v] + 1, finish[v] + 1))
        # a field never runs in the same pass as one of its ancestors
        anc = sch.ancestors(w.n_nodes, w.edges)
        for p in passes:
            act = [v for v, _ in p]
            assert act == sorted(act)
            for v in act:
                assert not (anc[v] & set(act))


def test_every_token_emitted_once_in_order():
    for seed in range(50):
        w = wl.random_template(5000 + seed, n_nodes=7, fixed_hi=2)
        lens = w.lens[0].tolist()
        passes = sch.simulate(w.n_nodes, w.edges, lens, w.n_fixed)
        seen = [vt for p in passes for vt in p]
        assert len(seen) == len(set(seen)) == sum(l - f for l, f in zip(lens, w.n_fixed))
        for v in range(w.n_nodes):
            assert [t for (x, t) in seen if x == v] == list(range(w.n_fixed[v], lens[v]))


def test_chain_and_edgeless_special_cases():
    lens = [3, 5, 2, 7]
    chain = sch.simulate(4, [(0, 1), (1, 2), (2, 3)], lens)
    assert len(chain) == sum(lens) and all(len(p) == 1 for p in chain)
    free = sch.simulate(4, [], lens)
    assert len(free) == max(lens) and len(free[0]) == 4
    assert sch.average_parallel_degree(free) == pytest.approx(sum(lens) / max(lens))


def test_cfg0_golden():
    gold = {}
    for line in open(os.path.join(GOLD, "cfg0_schedule.txt")):
        if line.strip() and not line.startswith("#"):
            k, *v = line.split()
            gold[k] = v
    w = wl.cfg0_tiny()
    passes = sch.simulate(w.n_nodes, w.edges, w.lens[0].tolist(), w.n_fixed)
    assert sum(len(p) for p in passes) == int(gold["tokens"][0])
    assert len(passes) == int(gold["steps"][0])
    assert sch.average_parallel_degree(passes) == float(gold["avg_parallel_degree"][0])
    widths = [int(x) for x in gold["widths"]]
    assert [len(passes[i]) for i in (0, 16, 32)] == widths
    assert max(len(p) for p in passes) == w.max_active


def test_rows_positions_and_write_counts():
    for seed in range(40):
        w = wl.random_template(7000 + seed, n_nodes=6, fixed_hi=2, prefix_len=seed % 70)
        lens = w.lens[0].tolist()
        base = sch.slot_base(w.slot_cap)
        T = base[-1]
        passes = sch.simulate(w.n_nodes, w.edges, lens, w.n_fixed)
        writes = np.zeros(w.prefix_len + T, dtype=int)
        for p in passes:
            for v, t in p:
                writes[sch.kv_row(w.prefix_len, base, v, t)] += 1
        # each generated row written exactly once; prefix, fixed rows and padding never
        for v in range(w.n_nodes):
            for j in range(w.slot_cap[v]):
                want = 1 if w.n_fixed[v] <= j < lens[v] else 0
                assert writes[w.prefix_len + base[v] + j] == want
        assert writes[:w.prefix_len].sum() == 0
        rows = [sch.kv_row(w.prefix_len, base, v, t) for v in range(w.n_nodes) for t in range(lens[v])]
        assert rows == sorted(rows) and len(set(rows)) == len(rows) and rows[-1] < w.prefix_len + T


def test_eq1_hand_example():
    """Token-level visibility of a hand-worked template (fixture derived by hand from Eq. 1)."""
    names = {"A": 0, "B": 1, "C": 2, "D": 3}
    edges = [(0, 2), (2, 3)]
    cap, lens, fixed, P = [3, 3, 3, 3], [2, 3, 2, 2], [1, 0, 0, 1], 1
    anc = sch.ancestors(4, edges)
    n_checked = 0
    for line in open(os.path.join(GOLD, "eq1_example_mask.txt")):
        if not line.strip() or line.startswith("#"):
            continue
        left, right = line.split(":")
        f, t = left.split()
        want = sorted(int(x) for x in right.split())
        vis = sch.visible_rows(4, anc, cap, lens, fixed, P, names[f], int(t))
        assert np.flatnonzero(vis).tolist() == want, line
        n_checked += 1
    assert n_checked == 7


def test_tile_list_and_union_bitmap_hand_example():
    """pass_tables' tile list, union bitmap and branch bitmaps against a hand-worked case: a prefix
    that is no tile multiple, a tile that holds nothing but padding, a partial last tile."""
    n, edges, cap, lens, P = 3, [(0, 2)], [140, 70, 30], [5, 8, 2], 70
    passes = sch.simulate(n, edges, lens)
    assert len(passes) == 8 and passes[5] == [(1, 5), (2, 0)] and passes[7] == [(1, 7)]
    n_checked = 0
    for line in open(os.path.join(GOLD, "tile_list_example.txt")):
        if not line.strip() or line.startswith("#"):
            continue
        left, right = line.split(":")
        f = left.split()
        want = [int(x) for x in right.split()]
        tab = sch.pass_tables(n, edges, cap, lens, [0] * n, P, passes[int(f[1])])
        if f[2] == "tiles":
            assert tab["tiles"].tolist() == want, line
        elif f[2] == "umask":
            assert [int(x) for x in tab["umask"]] == want, line
        else:
            assert [int(x) for x in tab["mask"][int(f[3])]] == want, line
        n_checked += 1
    assert n_checked == 7


def test_mask_invariants_random():
    for seed in range(60):
        w = wl.random_template(9000 + seed, n_nodes=2 + seed % 8, fixed_hi=seed % 3, prefix_len=seed % 130,
                               cap_hi=40)
        n, lens = w.n_nodes, w.lens[0].tolist()
        anc = sch.ancestors(n, w.edges)
        base = sch.slot_base(w.slot_cap)
        P = w.prefix_len
        for p in sch.simulate(n, w.edges, lens, w.n_fixed):
            tab = sch.pass_tables(n, w.edges, w.slot_cap, lens, w.n_fixed, P, p)
            for b, (v, t) in enumerate(p):
                vis = tab["vis"][b]
                q_row = P + base[v] + t
                assert vis[:P].all() and vis[q_row]
                n_fixed_lower = sum(1 for u in range(n) for j in range(w.n_fixed[u])
                                    if u != v and u not in anc[v] and P + base[u] + j < q_row)
                assert vis[P:].sum() == sum(lens[u] for u in anc[v]) + t + 1 + n_fixed_lower
                for u in range(n):
                    sl = vis[P + base[u]:P + base[u + 1]]
                    assert not sl[lens[u]:].any()                     # padding seen by nobody
                    if u != v and u not in anc[v]:
                        assert not sl[w.n_fixed[u]:].any()            # independent / descendant fields
                # bitmap packing: bit i of word w <-> template row 64w+i
                for r in range(base[-1]):
                    assert bool(int(tab["mask"][b][r // 64]) >> (r % 64) & 1) == bool(vis[P + r])
            union = tab["vis"].any(axis=0)
            assert [i for i in range((len(union) + 63) // 64) if union[64 * i:64 * i + 64].any()] == \
                tab["tiles"].tolist()
            um = tab["umask"]
            for r in range(base[-1]):
                assert bool(int(um[r // 64]) >> (r % 64) & 1) == bool(union[P + r])


def test_chain_mask_is_lower_triangular():
    n, cap = 5, [4, 4, 4, 4, 4]
    edges = [(i, i + 1) for i in range(n - 1)]
    P = 3
    passes = sch.simulate(n, edges, cap)
    for k, p in enumerate(passes):
        (v, t), = p
        tab = sch.pass_tables(n, edges, cap, cap, [0] * n, P, p)
        want = np.arange(P + 20) <= P + k          # causal: rows 0..own
        assert (tab["vis"][0] == want).all()
        assert tab["kv_row"][0] == P + k == tab["pos_id"][0]


def test_workload_shapes():
    """The synthetic configurations have the stated sizes (Sec. 3.1: a CoT of 300-500 tokens, fixed slots)."""
    w1 = wl.cfg1_7b()
    assert (w1.layers, w1.hq, w1.hkv, w1.head_dim, w1.batch, w1.prefix_len) == (28, 28, 4, 128, 1, 2048)
    assert w1.lens.min() >= 32 and w1.lens.max() <= 64 and w1.cot_rows == 512
    assert 300 <= int(w1.lens.sum()) <= 500          # Sec. 3.1: a CoT of 300-500 tokens
    w2 = wl.cfg2_batched()
    assert (w2.batch, w2.prefix_len, w2.cot_rows) == (16, 4096, 768)
    assert w2.lens.min() >= 16 and w2.lens.max() <= 96
    w3 = wl.cfg3_wide()
    anc = sch.ancestors(w3.n_nodes, w3.edges)
    assert len(anc[16]) == 8 and len(anc[17]) == 8 and anc[18] == anc[16] | anc[17] | {16, 17}
    assert len(sch.simulate(w3.n_nodes, w3.edges, w3.lens[0].tolist())) == 144
    for w in (w1, w2, w3):
        for s in range(w.batch):
            assert max(len(p) for p in sch.simulate(w.n_nodes, w.edges, w.lens[s].tolist())) == w.max_active
    w4 = wl.cfg4_sweep(1024, 8, 1)
    assert len(sch.simulate(8, w4.edges, [64] * 8)) == 64
    w4c = wl.cfg4_sweep(1024, 8, 1, chain=True)
    assert len(sch.simulate(8, w4c.edges, [64] * 8)) == 512


def test_a_concurrent_response_field_adds_no_pass():
    """Sec. 4.3 (future work): a fast response decoded beside the chain of thought costs no extra
    forward pass as long as it is shorter than the critical path: the schedule of every scene has
    the same length with and without the extra source field, and only the first passes are wider."""
    w0, w1 = wl.cfg2_batched(layers=1), wl.cfg2_dual_response(layers=1)
    assert w1.n_nodes == w0.n_nodes + 1 and w1.max_active == w0.max_active + 1
    for s in range(w0.batch):
        p0 = sch.simulate(w0.n_nodes, w0.edges, w0.lens[s].tolist())
        p1 = sch.simulate(w1.n_nodes, w1.edges, w1.lens[s].tolist())
        assert len(p0) == len(p1)
        extra = int(w1.lens[s, -1])
        assert [len(b) - len(a) for a, b in zip(p0, p1)] == [1] * extra + [0] * (len(p0) - extra)
        assert sch.average_parallel_degree(p1) > sch.average_parallel_degree(p0)
