"""Pins of the float64 attention checker (oracle/attention.c, oracle/run.py) against things
other than itself: a library causal-attention routine on chain templates, literal
exp/sum brute force, closed-form special cases and invariance to invisible rows."""
import math

import numpy as np
import pytest
import torch

from oracle import attention as oatt
from oracle import run as orun
from oracle import schedule as sch
from paper_2602_02864_b200 import workloads as wl


def _f32(t):
    return t.to(torch.float32).numpy()


def _make_run(w):
    r = orun.OracleRun(w.n_nodes, w.edges, w.slot_cap, w.n_fixed, w.prefix_len, w.lens, w.layers,
                       w.hq, w.hkv, w.head_dim, w.softmax_scale, w.max_active)
    for l in range(w.layers):
        k, v = wl.prefix_kv(w, l)
        r.write_prefix(l, _f32(k), _f32(v))
        if sum(w.n_fixed):
            k, v = wl.fixed_kv(w, l)
            r.write_fixed(l, _f32(k), _f32(v))
    return r


def _play(w, r):
    """Runs every pass; returns {(scene, node, tok): out[hq][D]} and the inputs used."""
    outs, qs = {}, {}
    for step in range(r.n_steps):
        q, k, v = wl.step_qkv(w, step, 0)
        r.append(step, 0, _f32(k), _f32(v))
        o = r.attend(step, 0, _f32(q))
        for s in range(w.batch):
            for b, (node, t) in enumerate(r.active(s, step)):
                outs[(s, node, t)] = o[s, b]
                qs[(s, node, t)] = _f32(q)[s, b]
    return outs, qs


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_chain_equals_library_causal_attention(dtype):
    """A chain template is the autoregressive baseline (Sec. 4.1): the run's outputs must
    equal ordinary causal attention over [prefix + CoT], here torch's SDPA in float64."""
    n, cap, P = 4, 6, 9
    w = wl.cfg4_sweep(P, n, 2, chain=True)
    w.slot_cap, w.lens = [cap] * n, np.full((2, n), cap, np.int32)
    w.hq, w.hkv, w.head_dim, w.dtype = 6, 2, 16, dtype
    r = _make_run(w)
    outs, qs = _play(w, r)
    assert not np.isnan(r.K).any()            # a chain without padding writes every row
    T = n * cap
    for s in range(2):
        Q = np.stack([qs[(s, i // cap, i % cap)] for i in range(T)])        # [T][hq][D]
        qt = torch.from_numpy(Q).double().permute(1, 0, 2)[None]             # [1][hq][T][D]
        kt = torch.from_numpy(r.K[s, 0]).double().repeat_interleave(w.group, 0)[None]
        vt = torch.from_numpy(r.V[s, 0]).double().repeat_interleave(w.group, 0)[None]
        allow = torch.ones(T, P + T, dtype=torch.bool).tril(diagonal=P)      # query i sees rows <= P+i
        ref = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, attn_mask=allow,
                                                               scale=w.softmax_scale)[0]
        for i in range(T):
            got = outs[(s, i // cap, i % cap)]
            assert np.abs(got - ref[:, i].numpy()).max() < 1e-12


def test_tiny_bruteforce_without_max_subtraction():
    rng = np.random.default_rng(3)
    A, Hq, Hkv, R, D = 3, 4, 2, 8, 5
    q = rng.standard_normal((A, Hq, D)).astype(np.float32)
    K = rng.standard_normal((Hkv, R, D)).astype(np.float32)
    V = rng.standard_normal((Hkv, R, D)).astype(np.float32)
    vis = rng.random((A, R)) < 0.6
    vis[:, 0] = True
    scale = 0.37
    got = oatt.attention(q, K, V, vis, scale)
    for a in range(A):
        for h in range(Hq):
            g = h // (Hq // Hkv)
            num = [0.0] * D
            den = 0.0
            for r in range(R):
                if vis[a, r]:
                    e = math.exp(scale * sum(float(q[a, h, d]) * float(K[g, r, d]) for d in range(D)))
                    den += e
                    for d in range(D):
                        num[d] += e * float(V[g, r, d])
            assert np.allclose(got[a, h], [x / den for x in num], rtol=1e-13, atol=1e-14)


def test_special_cases():
    rng = np.random.default_rng(4)
    A, Hq, Hkv, R, D = 2, 6, 3, 40, 8
    q = rng.standard_normal((A, Hq, D)).astype(np.float32)
    K = rng.standard_normal((Hkv, R, D)).astype(np.float32)
    V = rng.standard_normal((Hkv, R, D)).astype(np.float32)
    vis = rng.random((A, R)) < 0.5
    vis[:, 3] = True
    # all visible V rows equal => output is that row, whatever the scores
    Vu = V.copy()
    Vu[:, :, :] = V[:, :1, :]
    out = oatt.attention(q, K, Vu, vis, 0.3)
    for h in range(Hq):
        assert np.allclose(out[:, h], Vu[h // 2, 0], rtol=0, atol=1e-14)
    # one visible row => output is exactly that V row
    one = np.zeros((A, R), bool)
    one[0, 7] = one[1, 11] = True
    out = oatt.attention(q, K, V, one, 0.3)
    for h in range(Hq):
        assert (out[0, h] == V[h // 2, 7]).all() and (out[1, h] == V[h // 2, 11]).all()
    # zero queries => uniform weights => plain mean of the visible V rows
    out = oatt.attention(np.zeros_like(q), K, V, vis, 0.3)
    for a in range(A):
        for h in range(Hq):
            assert np.allclose(out[a, h], V[h // 2][vis[a]].astype(np.float64).mean(0), atol=1e-14)
    # heads of one group with the same q give the same output; other groups differ
    qq = q.copy()
    qq[:, 1] = qq[:, 0]
    qq[:, 2] = qq[:, 0]
    out = oatt.attention(qq, K, V, vis, 0.3)
    assert (out[:, 0] == out[:, 1]).all() and not np.allclose(out[:, 0], out[:, 2])
    # the scale matters and enters the exponent: doubling q == doubling the scale
    assert np.allclose(oatt.attention(2 * q, K, V, vis, 0.3), oatt.attention(q, K, V, vis, 0.6), atol=1e-13)
    with pytest.raises(ValueError):
        oatt.attention(q, K, V, np.zeros((A, R), bool), 0.3)


def test_invisible_rows_do_not_matter():
    """Sec. 3.3 / Fig. 3: independent fields, padding and unwritten rows cannot be attended:
    poisoning them (NaN, huge) leaves every output bitwise unchanged."""
    w = wl.cfg0_tiny()
    w.prefix_len, w.lens = 20, np.array([[16, 9, 16, 3, 12, 16]], np.int32)   # some padding
    r = _make_run(w)
    outs, _ = _play(w, r)
    r2 = _make_run(w)
    base = sch.slot_base(w.slot_cap)
    anc = sch.ancestors(w.n_nodes, w.edges)
    for step in range(r2.n_steps):
        q, k, v = wl.step_qkv(w, step, 0)
        r2.append(step, 0, _f32(k), _f32(v))
        act = r2.active(0, step)
        # poison everything that no active field may see at this pass
        Ksave, Vsave = r2.K.copy(), r2.V.copy()
        tab = r2.tables(0, step)
        hidden = ~tab["vis"].any(axis=0)
        r2.K[0, 0][:, hidden] = np.nan
        r2.V[0, 0][:, hidden] = 1e30
        # and, per branch, what only that branch must not see: checked through the output
        o = r2.attend(step, 0, _f32(q))
        for b, (node, t) in enumerate(act):
            assert (o[0, b] == outs[(0, node, t)]).all()
            sib = [u for u in range(w.n_nodes) if u != node and u not in anc[node]]
            for u in sib:
                assert not tab["vis"][b][w.prefix_len + base[u]:w.prefix_len + base[u + 1]].any()
        r2.K, r2.V = Ksave, Vsave
    # sibling perturbation: change every token of field 2 and fields 1,3,4 must not move
    w3 = wl.cfg0_tiny()
    w3.prefix_len, w3.lens = w.prefix_len, w.lens
    r3 = _make_run(w3)
    for step in range(r3.n_steps):
        q, k, v = wl.step_qkv(w3, step, 0)
        k, v = _f32(k).copy(), _f32(v).copy()
        for b, (node, t) in enumerate(r3.active(0, step)):
            if node == 2:
                k[0, b] += 3.0
                v[0, b] -= 5.0
        r3.append(step, 0, k, v)
        o = r3.attend(step, 0, _f32(q))
        for b, (node, t) in enumerate(r3.active(0, step)):
            same = (o[0, b] == outs[(0, node, t)]).all()
            assert same == (node in (0, 1, 3, 4)), (node, t)   # 2 itself and the summary 5 do move


def test_threads_do_not_change_result():
    rng = np.random.default_rng(5)
    q = rng.standard_normal((4, 4, 16)).astype(np.float32)
    K = rng.standard_normal((2, 100, 16)).astype(np.float32)
    V = rng.standard_normal((2, 100, 16)).astype(np.float32)
    vis = rng.random((4, 100)) < 0.7
    vis[:, 0] = True
    assert (oatt.attention(q, K, V, vis, 0.25, nthreads=1) == oatt.attention(q, K, V, vis, 0.25, nthreads=4)).all()


def test_oracle_run_places_fixed_rows_by_hand_example():
    """OracleRun.write_fixed: the pre-filled field-name rows (Sec. 3.3, Fig. 3: "pre-filled") go to the
    head of their fields' slots.  Hand example: slots of 3, 4 and 3 rows after a prefix of 2 rows, so
    field 0 starts at row 2, field 1 at row 5, field 2 at row 9; one fixed row in field 0 (row 2), none
    in field 1, two in field 2 (rows 9 and 10).  The i-th fixed row carries the value i + 1."""
    from oracle import run as orun
    lens = np.array([[2, 3, 3]], np.int32)
    o = orun.OracleRun(3, [], [3, 4, 3], [1, 0, 2], 2, lens, layers=2, hq=2, hkv=2, head_dim=4, scale=0.5, max_active=3)
    K = np.zeros((1, 2, 3, 4), np.float32)
    for i in range(3):
        K[:, :, i] = i + 1
    o.write_fixed(1, K, -K)
    want = {2: 1.0, 9: 2.0, 10: 3.0}
    for r in range(o.R):
        for h in range(2):
            if r in want:
                assert (o.K[0, 1, h, r] == want[r]).all() and (o.V[0, 1, h, r] == -want[r]).all()
            else:
                assert np.isnan(o.K[0, 1, h, r]).all() and np.isnan(o.V[0, 1, h, r]).all()
    assert np.isnan(o.K[0, 0]).all()                     # the other layer untouched
