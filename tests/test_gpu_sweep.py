"""Parity at the sizes of the sweep configuration (prefix x parallel fields x scenes), in the
launch configuration the benchmark times: sampled (pass, layer, scene, KV head) attention outputs
are recomputed by the float64 CPU checker from the cache rows copied back at that moment, with
visibility derived by the checker's own schedule; the integer tables of the sampled scenes are
compared bit for bit.  The parallel template (B independent 64-token fields) and the chain
template (the same fields one after the other: ordinary sequential decoding) are both played to
their last pass."""
import dataclasses

import numpy as np
import pytest
import torch

import bench
from oracle import attention as oatt
from oracle import schedule as sch
from paper_2602_02864_b200 import workloads as wl

from harness import check_close, f32

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2602_02864_b200 import build
    build.build()


def _play(P, B, Bt, chain, samples, layers=2):
    """samples: list of (pass, layer, scene, kv_head); pass -1 = the last one."""
    bench.LAYERS_OVERRIDE = None
    bench.FUSED_APPEND = True
    bench.USE_LENS = True
    w = dataclasses.replace(wl.cfg4_sweep(P, B, Bt, chain=chain), layers=layers)
    n_sched = 64 * B if chain else 64
    samples = [(n_sched - 1 if i < 0 else i, l, s, g) for (i, l, s, g) in samples]
    sb = bench.StepBench(w, n_sched, torch.device("cuda", 0), cheap_fill=True)
    sb.reset()
    by_step = {}
    for (i, l, s, g) in samples:
        by_step.setdefault(i, []).append((l, s, g))
    passes = sch.simulate(w.n_nodes, w.edges, w.lens[0].tolist(), w.n_fixed)      # every scene has the same lengths
    assert len(passes) == n_sched
    G = w.hq // w.hkv
    checked = 0
    for i in range(n_sched):
        sb.step(i)
        for (l, s, g) in by_step.get(i, []):
            torch.cuda.synchronize()
            this = passes[i]
            tab = sch.pass_tables(w.n_nodes, w.edges, w.slot_cap, w.lens[s].tolist(), w.n_fixed, w.prefix_len, this)
            A = len(this)
            assert A == (1 if chain else B) and int(sb.sess.n_active[s]) == A
            assert (sb.sess.node[s, :A].cpu().numpy() == tab["node"]).all()
            assert (sb.sess.kv_row[s, :A].cpu().numpy() == tab["kv_row"]).all()
            assert (sb.sess.mask[s, :A].cpu().numpy().view(np.uint64) == tab["mask"]).all()
            nt = int(sb.sess.ntiles[s])
            assert (sb.sess.tiles[s, :nt].cpu().numpy() == tab["tiles"]).all()
            K, V = f32(sb.k[s, l, g:g + 1]), f32(sb.v[s, l, g:g + 1])              # [1][rows][D] as the kernel saw them
            vis_any = tab["vis"].any(axis=0)
            K[:, ~vis_any] = np.nan                                                # reading a row nobody may see would show
            V[:, ~vis_any] = np.nan
            ref = oatt.attention(f32(sb.q[i, l, s, :A, g * G:(g + 1) * G]), K, V, tab["vis"], w.softmax_scale)
            got = f32(sb.out[l, s, :A, g * G:(g + 1) * G])
            check_close(got, ref, w.dtype, f"P {P} B {B} Bt {Bt} chain {chain} pass {i} layer {l} scene {s} head {g}")
            checked += A * G
    sb.schedule_pass()                                                             # the schedule is over
    assert int(sb.sess.all_done.item()) == 1
    assert sb.sess.status() == 0
    sb.sess.close()
    return checked


@pytest.mark.parametrize("B", [1, 8, 32])
@pytest.mark.parametrize("Bt", [1, 64])
def test_sweep_prefix_4k_first_and_last_pass(B, Bt):
    rng = np.random.default_rng(4096 + 100 * B + Bt)
    pick = lambda: (int(rng.integers(Bt)), int(rng.integers(8)))  # noqa: E731
    samples = [(0, 0) + pick(), (0, 1) + pick(), (-1, 0) + pick(), (-1, 1) + pick(), (31, 1) + pick()]
    assert _play(4096, B, Bt, False, samples) == 5 * B * 4


@pytest.mark.parametrize("P,B,Bt", [(16384, 4, 8), (16384, 32, 8), (32768, 16, 8), (32768, 32, 8), (16384, 4, 64), (1024, 1, 1)])
def test_sweep_long_prefixes_sampled(P, B, Bt):
    rng = np.random.default_rng(P + 100 * B + Bt)
    samples = [(i, int(rng.integers(2)), int(rng.integers(Bt)), int(rng.integers(8))) for i in (0, 17, -1)]
    assert _play(P, B, Bt, False, samples) == 3 * B * 4


@pytest.mark.parametrize("B", [8, 32])
def test_sweep_chain_comparator(B):
    """The same fields one after the other: 64 x B passes of one token, the sequential-decoding baseline."""
    rng = np.random.default_rng(7 + B)
    n = 64 * B
    samples = [(i, 0, int(rng.integers(8)), int(rng.integers(8))) for i in (0, 63, 64, n // 2 + 5, n - 1)]
    assert _play(4096, B, 8, True, samples, layers=1) == 5 * 4
