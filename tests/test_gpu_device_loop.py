"""Algorithm 1's loop kept on the device: one CUDA graph launch decodes the whole template (a WHILE
node whose condition fdc_loop_condition sets from fdc_frontier's all_done), and every pass's
attention output, the pass count and the final cache must be what the CPU checker computes."""
import numpy as np
import pytest
import torch

from harness import alloc_cache, check_close, f32, make_oracle, write_prefix
from paper_2602_02864_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _play_on_device(w, fused_append, max_passes=None):
    from paper_2602_02864_b200 import fdc
    from paper_2602_02864_b200.device_loop import DeviceLoop
    dev = "cuda"
    oracle = make_oracle(w)
    n = oracle.n_steps
    sess = fdc.DecodeSession(w.n_nodes, w.edges, w.slot_cap, w.n_fixed, w.prefix_len, w.max_active, w.batch, dev)
    sess.set_fused_append(fused_append)
    k, v = alloc_cache(w, dev)
    sess.bind_cache(k, v, w.hq)
    write_prefix(w, k, v, oracle, sess=sess)
    # the "model": every pass's q, k_new, v_new of every layer, fetched by a pass counter that lives on the device
    L = w.layers
    qs = torch.stack([torch.stack([wl.step_qkv(w, s, l, dev)[0] for l in range(L)]) for s in range(n)])
    ks = torch.stack([torch.stack([wl.step_qkv(w, s, l, dev)[1] for l in range(L)]) for s in range(n)])
    vs = torch.stack([torch.stack([wl.step_qkv(w, s, l, dev)[2] for l in range(L)]) for s in range(n)])
    q_buf, k_buf, v_buf = torch.empty_like(qs[0]), torch.empty_like(ks[0]), torch.empty_like(vs[0])
    out_buf = torch.full_like(qs[0], 7.0)
    out_log = torch.zeros_like(qs)
    idx = torch.zeros(1, dtype=torch.int64, device=dev)

    def body(stream):
        torch.index_select(qs.view(n, -1), 0, idx, out=q_buf.view(1, -1))
        torch.index_select(ks.view(n, -1), 0, idx, out=k_buf.view(1, -1))
        torch.index_select(vs.view(n, -1), 0, idx, out=v_buf.view(1, -1))
        for l in range(L):
            sess.kv_append(l, k_buf[l], v_buf[l], stream=stream)
            sess.decode_attn(l, q_buf[l], out_buf[l], w.softmax_scale, stream=stream)
        out_log.view(n, -1).index_copy_(0, idx, out_buf.view(1, -1))
        idx.add_(1)
        sess.frontier(None, stream=stream)
        sess.build_masks(stream=stream)

    loop = DeviceLoop(sess, body, max_passes or int(sum(w.slot_cap)))
    sess.init(torch.from_numpy(w.lens).to(dev))
    sess.frontier(None)
    sess.build_masks()
    loop.launch()
    torch.cuda.synchronize()
    passes = int(loop.passes.item())
    status = sess.status(clear=True)
    if max_passes is None:
        assert passes == n and status == 0
        assert int(sess.all_done.item()) == 1 and int(sess.n_active.sum().item()) == 0
        checked = 0
        for s in range(n):
            for l in range(L):
                oracle.append(s, l, f32(ks[s, l]), f32(vs[s, l]))
                ref = oracle.attend(s, l, f32(qs[s, l]))
                got = f32(out_log[s, l])
                for sc in range(w.batch):
                    A = len(oracle.active(sc, s))
                    if A:
                        check_close(got[sc, :A], ref[sc, :A], w.dtype, f"pass {s} layer {l} scene {sc}")
                        checked += A
        assert checked > 0
        R = w.rows
        assert np.array_equal(f32(k)[:, :, :, :R], oracle.K, equal_nan=True)
        assert np.array_equal(f32(v)[:, :, :, :R], oracle.V, equal_nan=True)
    loop.close()
    sess.close()
    return passes, status, n


@pytest.mark.parametrize("fused_append", [False, True], ids=["append_kernel", "append_inside_attention"])
def test_whole_template_in_one_graph_launch(fused_append):
    w = wl.cfg2_batched(layers=2, batch=3)
    passes, status, n = _play_on_device(w, fused_append)
    assert passes == n


def test_loop_limit_stops_the_loop_and_is_flagged():
    """A bound below the schedule's length: the loop ends there and says so."""
    from paper_2602_02864_b200 import fdc
    w = wl.cfg2_batched(layers=1, batch=2)
    passes, status, n = _play_on_device(w, False, max_passes=5)
    assert n > 5 and passes == 5 and status == fdc.FDC_DEV_LOOP_LIMIT
