"""Shared plumbing of the GPU parity tests: drives the C-ABI library and the CPU checker on
the same seeded inputs and compares them.  Holds no arithmetic of the method."""
from __future__ import annotations

import numpy as np
import torch

from oracle import run as orun
from paper_2602_02864_b200 import workloads as wl

F32_MAX_ABS = 1e-5        # fp32 configuration
BF16_MAX_ABS = 2e-2       # bf16 configurations (fp32 accumulate)
BF16_REL_L2 = 5e-3


def f32(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float32).numpy()


def make_oracle(w: wl.Workload) -> orun.OracleRun:
    return orun.OracleRun(w.n_nodes, w.edges, w.slot_cap, w.n_fixed, w.prefix_len, w.lens, w.layers, w.hq, w.hkv,
                          w.head_dim, w.softmax_scale, w.max_active)


def alloc_cache(w: wl.Workload, device, extra_rows: int = 0, fill: float = float("nan")):
    """K and V [batch][layers][hkv][rows][D] filled with `fill` (NaN: touching a row that was
    never written, e.g. padding, shows up in the output)."""
    shape = (w.batch, w.layers, w.hkv, w.rows + extra_rows, w.head_dim)
    k = torch.full(shape, fill, dtype=w.torch_dtype, device=device)
    v = torch.full(shape, fill, dtype=w.torch_dtype, device=device)
    return k, v


def write_prefix(w: wl.Workload, k, v, oracle=None, gen_device="cuda", sess=None):
    """Prefill: the shared prefix rows and the pre-filled field-name rows of every layer.  With a
    session (its cache bound) the field-name rows are placed by the library (fdc_kv_write_fixed);
    without one they are placed here, independently."""
    for l in range(w.layers):
        pk, pv = wl.prefix_kv(w, l, gen_device)
        k[:, l, :, :w.prefix_len] = pk.to(k.device)
        v[:, l, :, :w.prefix_len] = pv.to(v.device)
        if oracle is not None:
            oracle.write_prefix(l, f32(pk), f32(pv))
        if sum(w.n_fixed) and sess is not None:
            fk, fv = wl.fixed_kv(w, l, gen_device)
            sess.write_fixed(l, fk.to(k.device).contiguous(), fv.to(v.device).contiguous())
            if oracle is not None:
                oracle.write_fixed(l, f32(fk), f32(fv))
        elif sum(w.n_fixed):
            fk, fv = wl.fixed_kv(w, l, gen_device)
            i = 0
            base = np.concatenate([[0], np.cumsum(w.slot_cap)])
            for node in range(w.n_nodes):
                for j in range(w.n_fixed[node]):
                    r = w.prefix_len + int(base[node]) + j
                    k[:, l, :, r] = fk[:, :, i].to(k.device)
                    v[:, l, :, r] = fv[:, :, i].to(v.device)
                    i += 1
            if oracle is not None:
                oracle.write_fixed(l, f32(fk), f32(fv))


def compare_int_tables(sess, oracle, step: int):
    """Bit-exact comparison of everything fdc_frontier / fdc_build_masks produced for this pass."""
    w_words = sess.sizes.mask_words
    n_active = sess.n_active.cpu().numpy()
    node, tok, row, pos = (t.cpu().numpy() for t in (sess.node, sess.tok_idx, sess.kv_row, sess.pos_id))
    mask = sess.mask.cpu().numpy().view(np.uint64)
    umask = sess.umask.cpu().numpy().view(np.uint64)
    tiles, ntiles = sess.tiles.cpu().numpy(), sess.ntiles.cpu().numpy()
    live = False
    for s in range(oracle.batch):
        tab = oracle.tables(s, step)
        A = len(tab["node"])
        assert n_active[s] == A, (step, s, n_active[s], A)
        assert (node[s, :A] == tab["node"]).all() and (node[s, A:] == -1).all()
        assert (tok[s, :A] == tab["tok_idx"]).all() and (tok[s, A:] == -1).all()
        assert (row[s, :A] == tab["kv_row"]).all() and (row[s, A:] == -1).all()
        assert (pos[s, :A] == tab["pos_id"]).all() and (pos[s, A:] == -1).all()
        assert mask.shape[2] == w_words
        assert (mask[s, :A] == tab["mask"]).all(), (step, s)
        assert (mask[s, A:] == 0).all()
        assert (umask[s] == tab["umask"]).all()
        assert ntiles[s] == len(tab["tiles"]), (step, s, ntiles[s], len(tab["tiles"]))
        assert (tiles[s, :ntiles[s]] == tab["tiles"]).all()
        live |= step + 1 < len(oracle.passes[s])
    return live


def check_close(got: np.ndarray, ref: np.ndarray, dtype: str, what=""):
    """got, ref: [..., D].  fp32: max-abs; bf16: max-abs and per-vector relative L2."""
    err = np.abs(got.astype(np.float64) - ref)
    assert np.isfinite(got).all(), f"non-finite output {what}"
    if dtype == "f32":
        assert err.max() <= F32_MAX_ABS, f"max abs {err.max():.3e} {what}"
        return err.max(), 0.0
    rel = np.sqrt((err ** 2).sum(-1)) / np.sqrt((ref ** 2).sum(-1))
    assert err.max() <= BF16_MAX_ABS, f"max abs {err.max():.3e} {what}"
    assert rel.max() <= BF16_REL_L2, f"rel L2 {rel.max():.3e} {what}"
    return err.max(), rel.max()


def run_and_compare(w: wl.Workload, check_steps=None, check_layers=None, extra_rows: int = 0,
                    use_finish_flags: bool = False, kernel: int = 0, device="cuda", max_steps=None,
                    fused_append: bool = False):
    """Plays the whole schedule on the GPU through the C ABI and on the CPU checker.
    Integers are compared at every pass; attention at `check_steps` x `check_layers`
    (None = all).  Returns summary statistics."""
    from paper_2602_02864_b200 import fdc
    oracle = make_oracle(w)
    sess = fdc.DecodeSession(w.n_nodes, w.edges, w.slot_cap, w.n_fixed, w.prefix_len, w.max_active, w.batch, device)
    if kernel:
        fdc.fdc_set_attn_kernel(sess.plan, kernel)
    if fused_append:          # appends are recorded and written by the attention kernel (or on their own when none follows)
        sess.set_fused_append(True)
    k, v = alloc_cache(w, device, extra_rows)
    sess.bind_cache(k, v, w.hq)
    write_prefix(w, k, v, oracle, sess=sess)
    lens_dev = torch.from_numpy(w.lens).to(device)
    sess.init(None if use_finish_flags else lens_dev)
    out = torch.zeros(w.batch, w.max_active, w.hq, w.head_dim, dtype=w.torch_dtype, device=device)
    finish = None
    worst_abs, worst_rel, n_checked, step = 0.0, 0.0, 0, 0
    n_steps = oracle.n_steps if max_steps is None else min(max_steps, oracle.n_steps)
    while step < n_steps:
        sess.frontier(finish)
        sess.build_masks()
        live = compare_int_tables(sess, oracle, step)
        assert int(sess.all_done.item()) == 0
        if use_finish_flags:      # the caller-side "end of field" signal, derived from the true lengths
            fl = np.zeros((w.batch, w.max_active), np.uint8)
            for s in range(w.batch):
                for b, (node, t) in enumerate(oracle.active(s, step)):
                    fl[s, b] = 1 if t + 1 == w.lens[s, node] else 0
            finish = torch.from_numpy(fl).to(device)
        for l in range(w.layers):
            q, kn, vn = wl.step_qkv(w, step, l, device)
            sess.kv_append(l, kn, vn)
            oracle.append(step, l, f32(kn), f32(vn))
            do = (check_steps is None or step in check_steps) and (check_layers is None or l in check_layers)
            if not do:
                continue
            out.fill_(7.0)
            sess.decode_attn(l, q, out, w.softmax_scale)
            ref = oracle.attend(step, l, f32(q))
            got = f32(out)
            for s in range(w.batch):
                A = len(oracle.active(s, step))
                if A:
                    a, r = check_close(got[s, :A], ref[s, :A], w.dtype, f"step {step} layer {l} scene {s}")
                    worst_abs, worst_rel = max(worst_abs, a), max(worst_rel, r)
                    n_checked += A * w.hq
                assert (got[s, A:] == 7.0).all()          # unused branch slots are not touched
        step += 1
        del live
    if max_steps is None:
        sess.frontier(finish)
        assert int(sess.all_done.item()) == 1 and int(sess.n_active.sum().item()) == 0
        # every real row written exactly once, padding never: compare the whole cache bit for bit
        kc, vc = f32(k), f32(v)
        R = w.rows
        assert np.array_equal(kc[:, :, :, :R], oracle.K, equal_nan=True)
        assert np.array_equal(vc[:, :, :, :R], oracle.V, equal_nan=True)
        if extra_rows:
            assert np.isnan(kc[:, :, :, R:]).all()
    assert sess.status() == 0
    sess.close()
    return dict(steps=n_steps, worst_abs=worst_abs, worst_rel=worst_rel, checked=n_checked)
