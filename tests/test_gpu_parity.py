"""GPU parity: the C-ABI CUDA path against the CPU checker on the same seeded inputs.
Integers (schedule, slots, positions, bitmaps, tile lists, cache contents) bit-exact;
attention within the stated tolerances."""
import numpy as np
import pytest
import torch

from paper_2602_02864_b200 import workloads as wl

from harness import run_and_compare

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2602_02864_b200 import build
    build.build()


def test_cfg0_tiny_every_step():
    w = wl.cfg0_tiny()
    r = run_and_compare(w)
    assert r["steps"] == 48 and r["checked"] == 96 * 4


@pytest.mark.parametrize("kernel", [1, 2, 3])
@pytest.mark.parametrize("head_dim", [64, 128])
def test_cfg0_tiny_bf16_all_kernels(kernel, head_dim):
    """The bf16 variant of the tiny case through the CUDA-core kernel (1), the TMA + mma.sync
    kernel (2) and the TMA + tcgen05 kernel (3)."""
    w = wl.cfg0_tiny()
    w.dtype, w.head_dim = "bf16", head_dim
    run_and_compare(w, kernel=kernel)


def test_cfg1_7b_reduced_layers():
    """Config 1 shapes (28 q heads / 4 KV heads -> group 7, prefix 2048), 2 of its layers."""
    w = wl.cfg1_7b(layers=2)
    n = int(w.lens[0, :6].max() + w.lens[0, 6] + w.lens[0, 7])
    steps = set(range(0, n, 9)) | {int(w.lens[0, :6].min()) - 1, int(w.lens[0, :6].min()),
                                   int(w.lens[0, :6].max()) - 1, int(w.lens[0, :6].max()), n - 1}
    r = run_and_compare(w, check_steps=steps)
    assert r["steps"] == n


def test_cfg2_batched_reduced():
    """Config 2 shapes with 4 of its 16 scenes and 1 layer: scenes in different phases."""
    w = wl.cfg2_batched(layers=1, batch=4)
    r = run_and_compare(w, check_steps=set(range(0, 300, 17)) | {15, 16, 95, 96})
    assert r["checked"] > 0


def test_cfg3_wide_reduced():
    """Config 3 shapes (16-wide frontier, 64 query rows per KV head), 2 scenes, 1 layer."""
    w = wl.cfg3_wide(layers=1, batch=2)
    r = run_and_compare(w, check_steps={0, 1, 47, 48, 49, 95, 96, 143})
    assert r["steps"] == 144


@pytest.mark.parametrize("branches,chain", [(1, False), (4, False), (32, False), (4, True)])
def test_cfg4_sweep_points_small_prefix(branches, chain):
    w = wl.cfg4_sweep(1024, branches, 2, chain=chain)
    r = run_and_compare(w, check_steps={0, 1, 31, 63, 64, 255})
    assert r["steps"] == (64 * branches if chain else 64)


@pytest.mark.parametrize("seed", range(12))
def test_random_templates_with_fixed_tokens_and_ragged_prefix(seed):
    """Random DAGs, ragged slots, fixed field-name rows, prefix lengths that are not tile
    multiples (including 0), caches longer than P+T, several scenes."""
    w = wl.random_template(3000 + seed, n_nodes=3 + seed, edge_prob=0.3, cap_lo=2, cap_hi=70, batch=3,
                           prefix_len=[0, 1, 63, 64, 65, 130, 200, 7, 128, 31, 96, 5][seed], fixed_hi=seed % 4,
                           hq=8, hkv=2, head_dim=64 if seed % 2 else 128, dtype="f32" if seed % 3 else "bf16")
    w.max_active = w.n_nodes
    # the fused-append option is on for half of them: only bf16 / head_dim 128 caches take it up, the
    # others must go on appending with the kernel of its own
    run_and_compare(w, extra_rows=seed * 5, fused_append=seed % 2 == 1 or seed == 6)


def test_finish_flags_drive_the_schedule():
    w = wl.random_template(4242, n_nodes=9, edge_prob=0.3, cap_hi=20, batch=4, prefix_len=70)
    run_and_compare(w, use_finish_flags=True)


def test_truncation_to_slot_when_no_length_given():
    """Without lengths or flags every field runs to its slot capacity (Sec. 3.3: truncate)."""
    w = wl.random_template(4243, n_nodes=6, edge_prob=0.4, cap_hi=12, batch=2, prefix_len=10)
    w.lens = np.tile(np.array(w.slot_cap, np.int32), (2, 1))
    from paper_2602_02864_b200 import fdc
    from harness import make_oracle, compare_int_tables
    oracle = make_oracle(w)
    sess = fdc.DecodeSession(w.n_nodes, w.edges, w.slot_cap, w.n_fixed, w.prefix_len, w.max_active, w.batch)
    sess.init(None)
    for step in range(oracle.n_steps):
        sess.frontier(None)
        sess.build_masks()
        compare_int_tables(sess, oracle, step)
    sess.frontier(None)
    assert int(sess.all_done.item()) == 1


def test_device_anomalies_are_flagged_not_fatal():
    from paper_2602_02864_b200 import fdc
    # frontier wider than max_active: clamped, flagged, and the run still completes correctly
    sess = fdc.DecodeSession(4, [], [3, 3, 3, 3], None, 4, 2, 1)
    sess.init(None)
    seen = []
    for _ in range(20):
        sess.frontier(None)
        if int(sess.all_done.item()):
            break
        seen.append(sess.node[0, :int(sess.n_active.item())].tolist())
    assert seen == [[0, 1]] * 3 + [[2, 3]] * 3
    assert sess.status(clear=True) == fdc.FDC_DEV_FRONTIER_WIDE
    assert sess.status() == 0
    # lengths outside the slot are clamped and flagged
    sess.init(torch.tensor([[9, 0, 2, 3]], dtype=torch.int32, device="cuda"))
    assert sess.status(clear=True) == fdc.FDC_DEV_LEN_RANGE
    # a KV row outside the cache is skipped and flagged
    k = torch.zeros(1, 1, 1, 16, 64, device="cuda")
    v = torch.zeros_like(k)
    sess.bind_cache(k, v, 1)
    sess.frontier(None)
    sess.kv_row.fill_(99)
    kn = torch.ones(1, 2, 1, 64, device="cuda")
    sess.kv_append(0, kn, kn)
    # (the 4-wide frontier was clamped to 2 again, so that bit is set too)
    assert sess.status(clear=True) == fdc.FDC_DEV_ROW_RANGE | fdc.FDC_DEV_FRONTIER_WIDE
    assert float(k.abs().sum()) == 0.0
    sess.close()


def test_argument_errors():
    from paper_2602_02864_b200 import fdc
    sess = fdc.DecodeSession(2, [(0, 1)], [4, 4], None, 8, 1, 1)
    k = torch.zeros(1, 1, 2, 16, 64, device="cuda")
    with pytest.raises(fdc.FdcError) as e:
        sess.bind_cache(k, k.clone(), 3)                # hq % hkv
    assert e.value.code == fdc.FDC_ERR_SHAPE
    k = torch.zeros(1, 1, 2, 15, 64, device="cuda")      # rows < P + T
    with pytest.raises(fdc.FdcError) as e:
        sess.bind_cache(k, k.clone(), 2)
    assert e.value.code == fdc.FDC_ERR_SHAPE
    k = torch.zeros(1, 1, 2, 16, 64, device="cuda")
    sess.bind_cache(k, k.clone(), 2)
    q = torch.zeros(1, 1, 2, 64, device="cuda")
    with pytest.raises(fdc.FdcError) as e:
        fdc.fdc_decode_attn(sess.plan, sess.kv, 0, sess.n_active, sess.mask, sess.tiles, sess.ntiles, q, q.clone(),
                            0.125, sess.workspace, 16)
    assert e.value.code == fdc.FDC_ERR_WORKSPACE
    with pytest.raises(fdc.FdcError) as e:
        sess.kv_append(3, q, q)
    assert e.value.code == fdc.FDC_ERR_RANGE
    sess.close()


def test_critical_path_host_call_matches_device_schedule():
    from paper_2602_02864_b200 import fdc
    from oracle import schedule as sch
    for seed in range(10):
        w = wl.random_template(8800 + seed, n_nodes=4 + seed, fixed_hi=2)
        plan = fdc.fdc_plan_graph(w.n_nodes, w.edges, w.slot_cap, w.n_fixed, w.prefix_len, w.max_active)
        steps, fin = fdc.fdc_plan_critical_path(plan, w.lens[0])
        passes = sch.simulate(w.n_nodes, w.edges, w.lens[0].tolist(), w.n_fixed)
        assert steps == len(passes)
        anc, par, base, indeg = fdc.fdc_plan_tables(plan, w.n_nodes)
        ref_anc = sch.ancestors(w.n_nodes, w.edges)
        for v in range(w.n_nodes):
            assert {u for u in range(w.n_nodes) if int(anc[v]) >> u & 1} == ref_anc[v]
            assert fin[v] == 1 + max(k for k, p in enumerate(passes) if any(x == v for x, _ in p))
        assert base.tolist() == sch.slot_base(w.slot_cap)
        fdc.fdc_plan_destroy(plan)


def test_softmax_reference_is_raised_when_scores_jump(monkeypatch):
    """Prefix keys that grow along the rows make later scores exceed the first rounds' maxima
    by far more than 2^16: the kernel has to raise its softmax references and rescale sums and
    accumulator in flight (deferred by two or three rounds), and must still match the checker."""
    from paper_2602_02864_b200 import fdc
    import harness
    orig = wl.prefix_kv

    def growing(w, layer, device="cpu", scenes=None):
        k, v = orig(w, layer, device, scenes)
        scale = torch.ones(w.prefix_len, device=k.device)
        scale[300:] = 4.0
        scale[700:] = 12.0
        scale[1500:] = 0.25
        k = (k.float() * scale[None, None, :, None]).to(k.dtype)
        return k, v

    monkeypatch.setattr(harness.wl, "prefix_kv", growing)
    for branches in (4, 16):
        w = wl.cfg4_sweep(2048, branches, 2)
        r = run_and_compare(w, check_steps={0, 1, 2, 33, 63}, kernel=3)
        assert r["checked"] > 0
    # With few pairs every thread block gets a handful of rounds only.  24 scenes x 8 KV heads are more
    # pairs than thread blocks: a block then walks through whole prefixes (16 rounds and more per
    # segment), so the jumps at rows 300 and 700 arrive in mid-segment, where the raise is deferred
    # (16 fields = 64 query rows: the build with two groups of softmax warps; 4 and 32: one group).
    for branches in (4, 16, 32):
        w = wl.cfg4_sweep(2048, branches, 24)
        r = run_and_compare(w, check_steps={0, 33, 63}, kernel=3)
        assert r["checked"] > 0


def test_work_split_of_the_previous_call_is_reused_only_for_the_same_counts():
    """The work split of a pass is computed once (before its first attention call) and kept in
    the plan.  A repeated call must give the same bits; a call with other counts (one scene
    switched off, in other arrays or in the same ones) must not use the stale split; and going
    back to the first counts must reproduce the first result."""
    from paper_2602_02864_b200 import fdc
    from harness import alloc_cache, write_prefix, BF16_MAX_ABS, f32
    w = wl.cfg2_batched(layers=1, batch=4)
    dev = "cuda"
    sess = fdc.DecodeSession(w.n_nodes, w.edges, w.slot_cap, w.n_fixed, w.prefix_len, w.max_active, w.batch, dev)
    k, v = alloc_cache(w, dev)
    write_prefix(w, k, v)
    sess.bind_cache(k, v, w.hq)
    sess.init(torch.from_numpy(w.lens).to(dev))
    sess.frontier(None)
    sess.build_masks()
    q, kn, vn = wl.step_qkv(w, 0, 0, dev)
    sess.kv_append(0, kn, vn)

    def attend(n_active, ntiles):
        out = torch.full_like(q, 7.0)
        fdc.fdc_decode_attn(sess.plan, sess.kv, 0, n_active, sess.mask, sess.tiles, ntiles, q, out, w.softmax_scale,
                            sess.workspace, sess.ws_bytes)
        torch.cuda.synchronize()
        return out

    first = attend(sess.n_active, sess.ntiles)            # split computed
    again = attend(sess.n_active, sess.ntiles)            # same counts: split reused
    assert torch.equal(first, again)
    assert np.isfinite(f32(first)[sess.n_active.cpu().numpy().nonzero()[0], 0]).all()
    na2, nt2 = sess.n_active.clone(), sess.ntiles.clone()
    na2[1] = 0                                            # scene 1 has finished: no branch, no tile
    nt2[1] = 0
    other = attend(na2, nt2)
    assert bool((other[1] == 7.0).all())                  # nothing written for the scene that is off
    for s in (0, 2, 3):                                   # the others: same result up to the other split's rounding
        A = int(sess.n_active[s])
        assert np.abs(f32(other[s, :A]) - f32(first[s, :A])).max() <= BF16_MAX_ABS
    back = attend(sess.n_active, sess.ntiles)
    assert torch.equal(first, back)
    # the same arrays with other contents (behind the library's back): the kernel itself notices that
    # the kept split was made from other counts and makes its own
    keep = (sess.n_active.clone(), sess.ntiles.clone())
    sess.n_active[1] = 0
    sess.ntiles[1] = 0
    inplace = attend(sess.n_active, sess.ntiles)
    assert torch.equal(inplace, other)
    sess.n_active.copy_(keep[0])
    sess.ntiles.copy_(keep[1])
    assert torch.equal(first, attend(sess.n_active, sess.ntiles))
    assert sess.status() == 0
    sess.close()


@pytest.mark.parametrize("which", ["cfg1", "cfg2", "cfg3", "ragged", "fixed_rows"])
def test_fused_append_writes_the_same_cache_and_gives_the_same_attention(which):
    """fdc_set_fused_append: kv_append is only recorded and the next decode_attn writes the rows
    inside its kernel.  The whole schedule is played with the option on; layers / passes whose
    attention is not checked have no matching attention call, so their appends take the
    stand-alone kernel when the next call flushes them.  Attention matches the checker and at
    the end the whole cache equals the checker's, bit for bit (every real row once, padding never)."""
    if which == "cfg1":
        w = wl.cfg1_7b(layers=2)
        r = run_and_compare(w, check_steps=set(range(0, 200, 7)), check_layers={1}, fused_append=True)
    elif which == "cfg2":
        w = wl.cfg2_batched(layers=1, batch=4)
        r = run_and_compare(w, check_steps=set(range(0, 300, 5)) | {15, 16, 95, 96}, fused_append=True)
    elif which == "cfg3":
        w = wl.cfg3_wide(layers=1, batch=2)
        r = run_and_compare(w, check_steps=set(range(0, 144, 3)), fused_append=True)
    elif which == "ragged":      # prefix length that is no tile multiple, cache longer than P + T, bf16 head_dim 128
        w = wl.random_template(3006, n_nodes=9, edge_prob=0.3, cap_lo=2, cap_hi=70, batch=3, prefix_len=200, fixed_hi=0,
                               hq=8, hkv=2, head_dim=128, dtype="bf16")
        w.max_active = w.n_nodes
        r = run_and_compare(w, extra_rows=30, fused_append=True)
    else:                         # fixed field-name rows ahead of the generated tokens, prefix of 0 rows
        w = wl.random_template(3000, n_nodes=5, edge_prob=0.3, cap_lo=2, cap_hi=70, batch=3, prefix_len=0, fixed_hi=3,
                               hq=8, hkv=2, head_dim=128, dtype="bf16")
        w.max_active = w.n_nodes
        r = run_and_compare(w, fused_append=True)
    assert r["checked"] > 0


def test_fused_append_is_carried_out_even_without_an_attention_call():
    """A recorded append must never be lost: fdc_status, a second append, an attention call for
    another layer and switching the option off each launch it on its own first."""
    from paper_2602_02864_b200 import fdc
    from harness import alloc_cache, write_prefix
    w = wl.cfg2_batched(layers=2, batch=2)
    dev = "cuda"
    sess = fdc.DecodeSession(w.n_nodes, w.edges, w.slot_cap, w.n_fixed, w.prefix_len, w.max_active, w.batch, dev)
    k, v = alloc_cache(w, dev, fill=0.0)
    write_prefix(w, k, v)
    sess.bind_cache(k, v, w.hq)
    sess.init(torch.from_numpy(w.lens).to(dev))
    sess.set_fused_append(True)
    sess.frontier(None)
    sess.build_masks()
    rows = sess.kv_row.cpu().numpy()
    n_act = sess.n_active.cpu().numpy()

    def written(layer, kn):
        torch.cuda.synchronize()
        for s in range(w.batch):
            for b in range(int(n_act[s])):
                if not torch.equal(k[s, layer, :, int(rows[s, b])], kn[s, b]):
                    return False
        return True

    launches = fdc.fdc_launch_count()
    q, kn0, vn0 = wl.step_qkv(w, 0, 0, dev)
    sess.kv_append(0, kn0, vn0)
    assert fdc.fdc_launch_count() == launches            # recorded, nothing launched
    assert sess.status() == 0                            # fdc_status flushes
    assert written(0, kn0)
    _, kn1, vn1 = wl.step_qkv(w, 0, 1, dev)
    sess.kv_append(1, kn1, vn1)
    out = torch.zeros_like(q)
    sess.decode_attn(0, q, out, w.softmax_scale)         # attention for ANOTHER layer: append of layer 1 goes first, on its own
    assert written(1, kn1)
    _, kn2, vn2 = wl.step_qkv(w, 1, 0, dev)
    sess.kv_append(0, kn2, vn2)
    sess.set_fused_append(False)                         # switching off flushes too
    assert written(0, kn2)
    assert sess.status() == 0
    sess.close()


def test_tile_list_that_breaks_the_prefix_rule_is_flagged():
    """The attention kernel decides by list position which V stages have to be cleaned of rows
    nobody may see: the whole prefix tiles come first in a list (that is how fdc_build_masks
    writes it).  A list with a tile from beyond the prefix among the prefix entries is reported
    (the scene's output is then not to be trusted); the other scene is untouched and nothing
    waits for ever."""
    from paper_2602_02864_b200 import fdc
    from harness import alloc_cache, write_prefix
    w = wl.cfg2_batched(layers=1, batch=2)
    dev = "cuda"
    sess = fdc.DecodeSession(w.n_nodes, w.edges, w.slot_cap, w.n_fixed, w.prefix_len, w.max_active, w.batch, dev)
    k, v = alloc_cache(w, dev, fill=0.0)
    write_prefix(w, k, v)
    sess.bind_cache(k, v, w.hq)
    sess.init(torch.from_numpy(w.lens).to(dev))
    sess.frontier(None)
    sess.build_masks()
    q, kn, vn = wl.step_qkv(w, 0, 0, dev)
    sess.kv_append(0, kn, vn)
    good = torch.zeros_like(q)
    sess.decode_attn(0, q, good, w.softmax_scale)
    assert sess.status() == 0
    npre = w.prefix_len // 64
    assert int(sess.ntiles[1]) > npre
    tiles = sess.tiles.clone()
    tiles[1, 3], tiles[1, npre] = sess.tiles[1, npre].clone(), sess.tiles[1, 3].clone()
    out = torch.zeros_like(q)
    fdc.fdc_decode_attn(sess.plan, sess.kv, 0, sess.n_active, sess.mask, tiles, sess.ntiles, q, out, w.softmax_scale,
                        sess.workspace, sess.ws_bytes)
    assert sess.status(clear=True) == fdc.FDC_DEV_TILE_LIST
    assert torch.equal(out[0], good[0])
    assert sess.status() == 0
    sess.close()


@pytest.mark.parametrize("fused_append", [False, True], ids=["append_kernel", "append_inside_attention"])
def test_more_pairs_than_thread_blocks(fused_append):
    """40 scenes x 8 KV heads = 320 (scene, KV head) pairs for 148 thread blocks: every block then
    works through several pairs (weighted split, a new set of queries per pair, whole pairs written
    directly and cut ones merged), which the smaller cases never reach."""
    w = wl.cfg4_sweep(512, 4, 40)
    r = run_and_compare(w, check_steps={0, 1, 2, 31, 62, 63}, fused_append=fused_append)
    assert r["steps"] == 64 and r["checked"] > 0


@pytest.mark.parametrize("branches", [16, 32], ids=["64_query_rows", "128_query_rows"])
def test_more_pairs_than_thread_blocks_wide(branches):
    """The same regime with 64 and 128 query rows per pair (24 scenes x 8 KV heads = 192 pairs)."""
    w = wl.cfg4_sweep(512, branches, 24)
    r = run_and_compare(w, check_steps={0, 33, 63}, fused_append=True)
    assert r["steps"] == 64 and r["checked"] > 0


def _tail_template():
    """A chain of thought followed by the decoding phase after it (Sec. 3.3: padding is invisible
    "including [to] those generated for the subsequent meta-action and trajectory"; Sec. 4.1: the
    VLA-AR head emits the trajectory as 6 tokens): four independent perception fields with long
    slots and short contents (so that whole 64-row tiles are nothing but padding), a summary
    that needs them all, then a meta-action field and six one-token trajectory fields, chained."""
    n = 4 + 1 + 1 + 6
    edges = [(i, 4) for i in range(4)] + [(4, 5)] + [(5 + i, 6 + i) for i in range(6)]
    cap = [160, 150, 170, 160, 40, 8] + [1] * 6
    fixed = [3, 4, 5, 6, 3, 2] + [0] * 6
    lens = np.array([[9, 20, 12, 150, 17, 5] + [1] * 6, [30, 7, 170, 11, 40, 8] + [1] * 6], np.int32)
    return wl.Workload("tail_phase", "bf16", 1, 8, 2, 128, 2, 200, n, edges, cap, fixed, 4, lens, 260202899, 1.0)


def test_tail_phase_after_the_cot_sees_no_padding():
    """The meta-action and trajectory tokens that follow the CoT see every real token of every field
    and none of the padding; tiles that hold nothing but padding are not even visited.  Asserted on
    the checker's tables (which the GPU tables must equal bit for bit), with attention parity on
    those passes."""
    from oracle import schedule as sch
    w = _tail_template()
    base = np.concatenate([[0], np.cumsum(w.slot_cap)])
    tail_steps = set()
    for s in range(w.batch):
        lens = w.lens[s].tolist()
        passes = sch.simulate(w.n_nodes, w.edges, lens, w.n_fixed)
        n_tail = 0
        for i, this in enumerate(passes):
            if not any(v >= 5 for v, _ in this):
                continue
            tail_steps.add(i)
            tab = sch.pass_tables(w.n_nodes, w.edges, w.slot_cap, lens, w.n_fixed, w.prefix_len, this)
            for b, (v, t) in enumerate(this):
                vis = tab["vis"][b]
                for u in range(5 if v > 5 else v):                       # every earlier field: all of its real rows, none of its padding
                    r0 = w.prefix_len + int(base[u])
                    assert vis[r0:r0 + lens[u]].all() and not vis[r0 + lens[u]:r0 + w.slot_cap[u]].any()
                n_tail += 1
            pad_tiles = [ti for ti in range((w.rows + 63) // 64)
                         if ti * 64 >= w.prefix_len and not tab["vis"][:, ti * 64:(ti + 1) * 64].any()]
            assert pad_tiles and not set(pad_tiles) & set(tab["tiles"].tolist())
        assert n_tail == (lens[5] - w.n_fixed[5]) + 6
    r = run_and_compare(w, check_steps=tail_steps | {0, 5}, fused_append=True)
    assert r["checked"] > 0


def test_dual_response_template_reduced():
    """The batched shape with a response field decoded beside the chain of thought (7 fields wide)."""
    w = wl.cfg2_dual_response(layers=1, batch=3)
    r = run_and_compare(w, check_steps={0, 1, 15, 16, 23, 24, 25, 60, 150}, fused_append=True)
    assert r["checked"] > 0


def test_a_wait_that_cannot_end_gives_up_and_is_reported():
    """The bounded wait of the attention kernels, run against a barrier that nothing completes
    (fdc_selftest_bounded_wait): the launch ends by itself, every waiting thread gave up, the
    status word says FDC_DEV_TIMEOUT, and after clearing it the next ordinary run is correct."""
    from paper_2602_02864_b200 import fdc
    w = wl.cfg0_tiny()
    sess = fdc.DecodeSession(w.n_nodes, w.edges, w.slot_cap, w.n_fixed, w.prefix_len, w.max_active, w.batch, "cuda")
    outcome = torch.zeros(1, dtype=torch.int32, device="cuda")
    fdc.fdc_selftest_bounded_wait(sess.plan, outcome)
    torch.cuda.synchronize()
    assert int(outcome.item()) == 64
    assert sess.status(clear=True) == fdc.FDC_DEV_TIMEOUT
    assert sess.status() == 0
    sess.close()
    w2 = wl.cfg0_tiny()
    w2.dtype, w2.head_dim = "bf16", 128
    r = run_and_compare(w2, check_steps={0, 1, 5})
    assert r["checked"] > 0


@pytest.mark.parametrize("case", range(16))
def test_random_templates_larger_shapes(case):
    """Random DAGs on shapes the small random cases do not reach: GQA groups of 1 to 16, up to 24
    parallel fields (all three query-row widths of the tcgen05 kernel), 1 to 40 scenes (fewer and
    more (scene, KV head) pairs than thread blocks), prefixes of 0 to 3000 rows, slots of up to 130
    rows; the first, some middle and the last passes are compared."""
    from oracle import schedule as sch
    rng = np.random.default_rng(77000 + case)
    G = int(rng.choice([1, 2, 4, 7, 8, 16]))
    hkv = int(rng.choice([1, 2, 4, 8]))
    n_nodes = int(rng.integers(2, min(24, 128 // G) + 1))
    batch = int(rng.choice([1, 2, 5, 19, 24, 40]))
    w = wl.random_template(int(rng.integers(1 << 30)), n_nodes=n_nodes, edge_prob=float(rng.choice([0.0, 0.15, 0.4])), cap_lo=2,
                           cap_hi=int(rng.choice([6, 40, 70, 130])), batch=batch, prefix_len=int(rng.choice([0, 64, 100, 640, 1000, 2048, 3000])),
                           fixed_hi=int(rng.integers(0, 3)), hq=hkv * G, hkv=hkv, head_dim=128, dtype="bf16")
    w.max_active = n_nodes
    n = max(len(sch.simulate(w.n_nodes, w.edges, w.lens[s].tolist(), w.n_fixed)) for s in range(w.batch))
    r = run_and_compare(w, check_steps={0, 1, 2, n // 3, n // 2, n - 2, n - 1}, fused_append=bool(rng.integers(2)), kernel=3)
    assert r["steps"] == n and r["checked"] > 0
