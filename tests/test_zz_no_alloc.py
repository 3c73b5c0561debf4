"""fdc_decode_attn_static: the attention call for hosts that cannot allocate device memory.

Some users of this library run where the decode loop may not allocate: an in-vehicle runtime
with a device memory budget fixed at start-up (cudaMalloc would synchronise the device and can
fail once the KV pool owns the GPU), or a plugin-style host whose per-step call must not
allocate.  For them the library carries its own 16 MiB scratch buffer and this entry point
takes no workspace argument.  The test drives it through the C ABI and checks that it gives
what fdc_decode_attn gives with a caller-owned workspace, on two calls in a row (the buffer is
shared and keeps the previous call's contents, so the second call sees stale data), that its
result also matches the float64 CPU checker, that the amount of free device memory is the same
before and after a series of such calls (the property the entry point exists for), and that a
problem too large for the built-in buffer is refused before anything is launched.

Collected last on purpose (file name): a run that stops at the first failure has then already
run every other test.  It does not depend on the other tests having run or not.
"""
import numpy as np
import pytest
import torch

from paper_2602_02864_b200 import workloads as wl

from harness import BF16_MAX_ABS, BF16_REL_L2, F32_MAX_ABS, alloc_cache, f32, write_prefix

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2602_02864_b200 import build
    build.build()


def _advance(sess, w, step, device):
    """Forward pass `step` of the schedule: frontier, bitmaps, append of every layer's new rows."""
    sess.frontier(None)
    sess.build_masks()
    qs = []
    for l in range(w.layers):
        q, kn, vn = wl.step_qkv(w, step, l, device)
        sess.kv_append(l, kn, vn)
        qs.append(q)
    return qs


@pytest.mark.parametrize("make", [lambda: wl.cfg2_batched(layers=1, batch=3), wl.cfg0_tiny],
                         ids=["bf16_batched_shape", "fp32_tiny"])
def test_static_scratch_matches_caller_workspace_twice_in_a_row(make):
    from paper_2602_02864_b200 import fdc
    w = make()
    device = "cuda"
    sess = fdc.DecodeSession(w.n_nodes, w.edges, w.slot_cap, w.n_fixed, w.prefix_len, w.max_active, w.batch, device)
    k, v = alloc_cache(w, device)              # NaN everywhere that is never written
    write_prefix(w, k, v)
    sess.bind_cache(k, v, w.hq)
    assert fdc.fdc_attn_workspace_bytes(sess.plan, sess.kv) <= fdc.FDC_STATIC_WS_BYTES
    sess.init(torch.from_numpy(w.lens).to(device))
    shape = (w.batch, w.max_active, w.hq, w.head_dim)
    launches0 = fdc.fdc_launch_count()
    for step in range(2):                      # two passes; in each, two static calls back to back
        q1 = _advance(sess, w, step, device)[0]
        q2 = (-q1).flip(-1).contiguous()       # different queries for the second call
        got = [torch.full(shape, 7.0, dtype=w.torch_dtype, device=device) for _ in range(2)]
        want = [torch.full(shape, 7.0, dtype=w.torch_dtype, device=device) for _ in range(2)]
        for q, o in zip((q1, q2), got):
            fdc.fdc_decode_attn_static(sess.plan, sess.kv, 0, sess.n_active, sess.mask, sess.tiles, sess.ntiles, q, o,
                                       w.softmax_scale)
        for q, o in zip((q1, q2), want):
            sess.decode_attn(0, q, o, w.softmax_scale)
        torch.cuda.synchronize()
        assert not torch.equal(want[0], want[1])
        n_act = sess.n_active.cpu().numpy()
        assert n_act.sum() > 0
        for call, s in [(c, s) for c in range(2) for s in range(w.batch)]:
            a, b = f32(got[call]), f32(want[call])
            assert np.isfinite(a).all()
            A = int(n_act[s])
            assert (a[s, A:] == 7.0).all()     # rows of idle branch slots are not touched
            err = np.abs(a[s, :A].astype(np.float64) - b[s, :A])
            if w.dtype == "f32":
                assert err.max() <= F32_MAX_ABS
            else:
                rel = np.sqrt((err ** 2).sum(-1)) / np.sqrt((b[s, :A].astype(np.float64) ** 2).sum(-1))
                assert err.max() <= BF16_MAX_ABS and rel.max() <= BF16_REL_L2
    assert fdc.fdc_launch_count() > launches0
    assert sess.status() == 0
    sess.close()


def test_static_calls_take_no_device_memory_and_match_the_checker():
    """After a first call (which may load the library's device image and looks up the buffer's
    address) further calls must leave cudaMemGetInfo's free figure exactly where it was; and what
    they compute is the checker's masked attention, within the bf16 tolerance."""
    from paper_2602_02864_b200 import fdc
    from harness import check_close, make_oracle
    w = wl.cfg2_batched(layers=1, batch=2)
    device = "cuda"
    oracle = make_oracle(w)
    sess = fdc.DecodeSession(w.n_nodes, w.edges, w.slot_cap, w.n_fixed, w.prefix_len, w.max_active, w.batch, device)
    k, v = alloc_cache(w, device)
    write_prefix(w, k, v, oracle)
    sess.bind_cache(k, v, w.hq)
    sess.init(torch.from_numpy(w.lens).to(device))
    outs = [torch.full((w.batch, w.max_active, w.hq, w.head_dim), 7.0, dtype=w.torch_dtype, device=device) for _ in range(3)]
    steps = []
    for step in range(3):                       # everything torch allocates is allocated before the measurement
        steps.append(wl.step_qkv(w, step, 0, device))

    def one_pass(step):
        q, kn, vn = steps[step]
        sess.frontier(None)
        sess.build_masks()
        sess.kv_append(0, kn, vn)
        fdc.fdc_decode_attn_static(sess.plan, sess.kv, 0, sess.n_active, sess.mask, sess.tiles, sess.ntiles, q, outs[step],
                                   w.softmax_scale)

    one_pass(0)                                 # start-up call
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    one_pass(1)
    one_pass(2)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0
    for step in range(3):
        q, kn, vn = steps[step]
        oracle.append(step, 0, f32(kn), f32(vn))
        ref = oracle.attend(step, 0, f32(q))
        for s in range(w.batch):
            A = len(oracle.active(s, step))
            check_close(f32(outs[step])[s, :A], ref[s, :A], w.dtype, f"static call, pass {step} scene {s}")
    assert sess.status() == 0
    sess.close()


def test_static_scratch_refuses_what_does_not_fit():
    """64 scenes x 8 KV heads with 128 query rows each need more than the built-in 16 MiB."""
    from paper_2602_02864_b200 import fdc
    w = wl.cfg4_sweep(64, 32, 64)
    device = "cuda"
    sess = fdc.DecodeSession(w.n_nodes, w.edges, w.slot_cap, w.n_fixed, w.prefix_len, w.max_active, w.batch, device)
    k, v = alloc_cache(w, device, fill=0.0)
    sess.bind_cache(k, v, w.hq)
    assert fdc.fdc_attn_workspace_bytes(sess.plan, sess.kv) > fdc.FDC_STATIC_WS_BYTES
    sess.init(None)
    sess.frontier(None)
    sess.build_masks()
    q = torch.zeros(w.batch, w.max_active, w.hq, w.head_dim, dtype=w.torch_dtype, device=device)
    out = torch.full_like(q, 7.0)
    torch.cuda.synchronize()
    before = fdc.fdc_launch_count()
    with pytest.raises(fdc.FdcError) as e:
        fdc.fdc_decode_attn_static(sess.plan, sess.kv, 0, sess.n_active, sess.mask, sess.tiles, sess.ntiles, q, out,
                                   w.softmax_scale)
    assert e.value.code == fdc.FDC_ERR_STATIC_LIMIT
    assert "static" in str(e.value)
    assert fdc.fdc_launch_count() == before            # refused on the host, nothing launched
    torch.cuda.synchronize()
    assert bool((out == 7.0).all())
    sess.close()
