#!/usr/bin/env python
"""Benchmark of the dependency-masked parallel-decoding step on B200.

One "step" = one forward pass of the whole hot path for one batch of scenes:
fdc_frontier -> fdc_build_masks -> for every layer: fdc_kv_append -> fdc_decode_attn
(split-KV pass + combine pass).  The metric is achieved KV-cache bandwidth: the bytes the
method itself must move per step (every KV row visible to some branch read once for all
branches and GQA heads, plus q, out, the appended rows and the bitmaps) divided by the
step time.  Prints ONE JSON line on stdout (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2|cfg1|cfg3|cfg0]
                  [--impl fdc|reference] [--no-also]
Under torchrun (N > 1) every rank runs an independent replica of the workload (scenes shard
with no exchange): weak scaling, time = max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

# DRAM traffic of the split-KV kernel per algorithmic byte, from the ncu capture summarised in
# profiles/attn_tc_kernel_cfg2.md (dram__bytes_read.sum + dram__bytes_write.sum over the launch's
# algorithmic bytes; traffic grows in proportion to the visited tiles, so it scales to a full-size
# launch).  Only valid for the kernel source it was measured on: keyed by a hash of that source.
NCU_TRAFFIC = {"kernel_sha256_16": "131986594b3087ed", "dram_bytes_per_algorithmic_byte": 1.096}


def kernel_source_hash() -> str:
    import hashlib
    path = os.path.join(ROOT, "paper_2602_02864_b200", "csrc", "fdc_attn_tc_kernel.cuh")
    try:
        return hashlib.sha256(open(path, "rb").read()).hexdigest()[:16]
    except OSError:
        return ""


METRIC = "masked_decode_attn_kv_bandwidth"
UNIT = "GB/s"
NOMINAL_HBM_GBS = 8000.0


def log(*a):
    print(*a, file=sys.stderr, flush=True)


FUSED_APPEND = True         # fdc_set_fused_append: one kernel per layer (--separate-append: two)
LAYERS_OVERRIDE = None      # --layers: fewer layers of the same configuration (profiling captures)


def get_workload(name: str):
    from paper_2602_02864_b200 import workloads as wl
    if name == "cfg0":
        return wl.cfg0_tiny()
    f = {"cfg1": wl.cfg1_7b, "cfg2": wl.cfg2_batched, "cfg3": wl.cfg3_wide}[name]
    return f() if LAYERS_OVERRIDE is None else f(layers=LAYERS_OVERRIDE)


WORKLOAD_TEXT = {
    "cfg0": "configs[0] tiny fp32: 1 layer, 4q/2kv heads, D 64, batch 1, prefix 256, 6-field DAG, 16-token slots",
    "cfg1": "configs[1] 7B-class bf16: 28 layers, 28q/4kv heads, D 128, batch 1, prefix 2048, 8-field DAG, slots 64 (len U32-64)",
    "cfg2": "configs[2] batched scenes bf16: 32 layers, 32q/8kv heads, D 128, batch 16, prefix 4096, 8-field DAG, slots 96 (len U16-96 per scene)",
    "cfg3": "configs[3] wide graph bf16: 32 layers, 32q/8kv heads, D 128, batch 8, prefix 8192, 16 leaves -> 2 aggregators -> final, 48-token slots",
}


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler:
    """Samples SM clock, power and throttle reasons while the timed region runs (read only):
    NVML from a thread every 10 ms, or nvidia-smi in a child process when NVML is not importable."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.thread, self.rows, self.stop_flag = index, None, None, [], False
        self.nvml = self.handle = None
        try:
            import pynvml
            pynvml.nvmlInit()
            # the bench's device index is an index into CUDA_VISIBLE_DEVICES when that is set
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = index
            if vis:
                ent = vis.split(",")[index].strip()
                phys = int(ent) if ent.isdigit() else None
                self.handle = pynvml.nvmlDeviceGetHandleByUUID(ent) if phys is None else None
            if self.handle is None:
                self.handle = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.nvml = pynvml
        except Exception:
            self.nvml = self.handle = None

    def _poll(self):
        n = self.nvml
        bits = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40}
        while not self.stop_flag:
            try:
                sm = n.nvmlDeviceGetClockInfo(self.handle, n.NVML_CLOCK_SM)
                mx = n.nvmlDeviceGetMaxClockInfo(self.handle, n.NVML_CLOCK_SM)
                pw = n.nvmlDeviceGetPowerUsage(self.handle) / 1000.0
                try:
                    rs = n.nvmlDeviceGetCurrentClocksEventReasons(self.handle)
                except Exception:
                    rs = n.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle)
                self.rows.append((float(sm), float(mx), pw, {k for k, b in bits.items() if rs & b}))
            except Exception:
                pass
            time.sleep(0.01)

    def start(self):
        if self.nvml is not None:
            import threading
            self.stop_flag, self.rows = False, []
            self.thread = threading.Thread(target=self._poll, daemon=True)
            self.thread.start()
            return
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.thread is not None:
            self.stop_flag = True
            self.thread.join(timeout=2)
            self.thread = None
            sm = [r[0] for r in self.rows]
            reasons = set().union(*[r[3] for r in self.rows]) if self.rows else set()
            return {"sm_mhz": statistics.median(sm) if sm else None,
                    "sm_max_mhz": max(r[1] for r in self.rows) if self.rows else None,
                    "power_w_max": round(max(r[2] for r in self.rows), 2) if self.rows else None,
                    "samples": len(sm), "source": "nvml, 10 ms", "reasons": sorted(reasons)}
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons, pw = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
                pw.append(float(f[2]))
            except ValueError:
                continue
            for n, val in zip(names, f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None, "samples": len(sm), "source": "nvidia-smi, 100 ms",
                "reasons": sorted(reasons)}


class StepBench:
    """Device-resident state of one workload and the per-step launch sequence."""

    def __init__(self, w, n_steps: int, device, seed_shift: int = 0, cheap_fill: bool = False):
        import torch
        from paper_2602_02864_b200 import fdc, workloads as wl
        self.torch, self.fdc, self.w, self.device = torch, fdc, w, device
        self.n_steps = n_steps
        self.sess = fdc.DecodeSession(w.n_nodes, w.edges, w.slot_cap, w.n_fixed, w.prefix_len, w.max_active, w.batch,
                                      device)
        shape = (w.batch, w.layers, w.hkv, w.rows, w.head_dim)
        self.k = torch.zeros(shape, dtype=w.torch_dtype, device=device)   # padding rows stay zero
        self.v = torch.zeros(shape, dtype=w.torch_dtype, device=device)
        g = torch.Generator(device=device)
        g.manual_seed(w.seed + 7919 * seed_shift)
        if cheap_fill:
            # large sweep points: one seeded block of prefix rows per tensor, repeated over scenes and layers
            for t in (self.k, self.v):
                blk = (torch.randn((w.hkv, w.prefix_len, w.head_dim), generator=g, device=device) * w.kv_scale).to(w.torch_dtype)
                t[:, :, :, :w.prefix_len] = blk
        else:
            for l in range(w.layers):                                      # prefix KV, in HBM before timing
                for t in (self.k, self.v):
                    t[:, l, :, :w.prefix_len] = (torch.randn((w.batch, w.hkv, w.prefix_len, w.head_dim), generator=g,
                                                             device=device) * w.kv_scale).to(w.torch_dtype)
        if sum(w.n_fixed):
            # the pre-filled field-name rows (Fig. 3: "pre-filled"), written once like the prefix
            base = np.concatenate([[0], np.cumsum(w.slot_cap)])
            for node in range(w.n_nodes):
                r0 = w.prefix_len + int(base[node])
                nf = w.n_fixed[node]
                if nf:
                    for t in (self.k, self.v):
                        t[:, :, :, r0:r0 + nf] = (torch.randn((w.batch, w.layers, w.hkv, nf, w.head_dim), generator=g,
                                                              device=device) * w.kv_scale).to(w.torch_dtype)
        self.sess.bind_cache(self.k, self.v, w.hq)
        if FUSED_APPEND:
            self.sess.set_fused_append(True)
        self.lens = None if w.lens is None else torch.from_numpy(w.lens).to(device)
        qs = (n_steps, w.layers, w.batch, w.max_active, w.hq, w.head_dim)
        ks = (n_steps, w.layers, w.batch, w.max_active, w.hkv, w.head_dim)
        self.q = torch.randn(qs, generator=g, device=device).to(w.torch_dtype)
        self.kn = (torch.randn(ks, generator=g, device=device) * w.kv_scale).to(w.torch_dtype)
        self.vn = (torch.randn(ks, generator=g, device=device) * w.kv_scale).to(w.torch_dtype)
        self.out = torch.zeros((w.layers, w.batch, w.max_active, w.hq, w.head_dim), dtype=w.torch_dtype, device=device)
        self.umask_log = torch.zeros((n_steps,) + tuple(self.sess.umask.shape), dtype=torch.int64, device=device)
        self.nact_log = torch.zeros((n_steps, w.batch), dtype=torch.int32, device=device)
        self.launches_per_step = 2 + 3 * w.layers
        self.graphs = {}

    def reset(self):
        self.sess.init(self.lens if USE_LENS else None)

    def schedule_pass(self, log_index=None):
        """Algorithm 1 body and Eq. 1 bitmaps of the next pass (no attention)."""
        s = self.sess
        s.frontier(None)
        s.build_masks()
        if log_index is not None:
            self.umask_log[log_index].copy_(s.umask)
            self.nact_log[log_index].copy_(s.n_active)

    def layers_pass(self, i: int, q=None, kn=None, vn=None, out=None):
        s, w = self.sess, self.w
        out = self.out if out is None else out
        q = self.q[i] if q is None else q
        kn = self.kn[i] if kn is None else kn
        vn = self.vn[i] if vn is None else vn
        for l in range(w.layers):
            s.kv_append(l, kn[l], vn[l])
            s.decode_attn(l, q[l], out[l], w.softmax_scale)

    def step(self, i: int, q=None, kn=None, vn=None, log_masks: bool = False, out=None):
        self.schedule_pass(i if log_masks else None)
        self.layers_pass(i, q, kn, vn, out)

    # ---- CUDA graphs: one per step (its q / k_new / v_new live at their own addresses) ----
    def capture(self, i: int, what: str = "step"):
        """Captures step i (or only its per-layer part) into a CUDA graph and keeps it."""
        torch = self.torch
        key = (what, i)
        if key in self.graphs:
            return self.graphs[key]
        g = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream(self.device)
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.graph(g, stream=side, capture_error_mode="thread_local"):
            if what == "step":
                self.step(i)
            else:
                self.layers_pass(i)
        torch.cuda.current_stream().wait_stream(side)
        self.graphs[key] = g
        return g

    # ---- the method's own traffic (what one launch / one step must move) ----
    def algorithmic_bytes(self, steps):
        """Per step in `steps`: bytes of one layer-step, from the logged union bitmaps."""
        w = self.w
        um = self.umask_log.cpu().numpy().view(np.uint64)
        na = self.nact_log.cpu().numpy()
        row_bytes = 2 * w.hkv * w.head_dim * w.esize
        pop = np.vectorize(lambda x: bin(int(x)).count("1"))
        per = []
        for i in steps:
            act = na[i] > 0
            vis_rows = (w.prefix_len + pop(um[i]).sum(axis=1)) * act
            A = na[i].astype(np.int64)
            b = int(vis_rows.sum()) * row_bytes                         # each visible KV row once
            b += int(A.sum()) * (2 * w.hq * w.head_dim * w.esize)       # q in, out
            b += int(A.sum()) * row_bytes                               # appended rows
            b += int(A.sum()) * um.shape[2] * 8                         # bitmaps
            per.append(b)
        return per


def schedule_length(w) -> int:
    """Forward passes of the whole schedule of a workload (host arithmetic of the binding's plan)."""
    from paper_2602_02864_b200 import fdc
    plan = fdc.fdc_plan_graph(w.n_nodes, w.edges, w.slot_cap, w.n_fixed, w.prefix_len, w.max_active)
    try:
        lens = w.lens if USE_LENS else np.tile(np.array(w.slot_cap, np.int32), (w.batch, 1))
        return max(fdc.fdc_plan_critical_path(plan, lens[s])[0] for s in range(w.batch))
    finally:
        fdc.fdc_plan_destroy(plan)


USE_LENS = True             # False: no lengths are given, every field runs to its slot (truncation, Sec. 3.3)


def timed_region(sb, W: int, K: int, reps: int, use_graphs: bool, sampler=None, barrier=None):
    """reps x (reset, W warm-up steps, K timed steps).  Returns per repetition the total time and the
    per-step times (ms), CUDA events on the launching stream after every step."""
    import torch
    stream = torch.cuda.current_stream()
    sb.sess.use_stream(stream)
    total = W + K
    graphs = None
    if use_graphs:
        sb.reset()
        for i in range(total):
            sb.step(i)                      # eager once: every lazily set attribute is in place before capture
        torch.cuda.synchronize()
        sb.reset()
        graphs = []
        try:
            sb.sess.use_stream(None)        # the capture stream is torch's current stream inside the context
            for i in range(total):
                graphs.append(sb.capture(i))
        except Exception as e:              # capture refused: fall back to stream launches and say so
            log("graph capture failed, using stream launches:", repr(e)[:200])
            graphs = None
            sb.graphs.clear()
        sb.sess.use_stream(stream)
        torch.cuda.synchronize()
    runs = []
    for r in range(reps):
        sb.reset()
        for i in range(W):
            graphs[i].replay() if graphs else sb.step(i)
        if barrier is not None:
            barrier()
        torch.cuda.synchronize()
        if sampler is not None and r == 0:
            sampler.start()
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(K + 1)]
        evs[0].record(stream)
        for i in range(K):
            graphs[W + i].replay() if graphs else sb.step(W + i)
            evs[i + 1].record(stream)
        torch.cuda.synchronize()
        per = [evs[i].elapsed_time(evs[i + 1]) for i in range(K)]
        runs.append((evs[0].elapsed_time(evs[K]), per))
    sb.sess.use_stream(None)
    return runs, graphs is not None


def phase_report(w, per_ms, layer_bytes, nact_mean):
    """Layer-step time and bandwidth of the widest-frontier passes, the narrowest and the whole region."""
    out = {}
    live = [i for i, a in enumerate(nact_mean) if a > 0]
    if not live:
        return out
    amax, amin = max(nact_mean[i] for i in live), min(nact_mean[i] for i in live)
    sel = {"widest_frontier": [i for i in live if nact_mean[i] >= amax - 1e-9],
           "narrowest_frontier": [i for i in live if nact_mean[i] <= amin + 1e-9],
           "whole_region": list(range(len(per_ms)))}
    for name, idx in sel.items():
        t = sum(per_ms[i] for i in idx) * 1e-3
        b = sum(layer_bytes[i] for i in idx) * w.layers
        out[name] = {"passes": len(idx), "avg_active_branches_per_scene": round(float(np.mean([nact_mean[i] for i in idx])), 2),
                     "layer_step_us": round(t / len(idx) / w.layers * 1e6, 2), "GBs": round(b / t / 1e9, 1),
                     "pct_of_8TBs": round(100 * b / t / 1e9 / NOMINAL_HBM_GBS, 1)}
    return out


def run_fdc(args, rank: int, world: int):
    import torch
    import torch.distributed as dist
    from paper_2602_02864_b200 import build as _build
    if rank == 0:
        _build.build()
    if world > 1:
        dist.barrier()
    from paper_2602_02864_b200 import fdc, replicas
    local = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    peak, peak_src = measured_peaks()
    if args.only_device_loop:
        if rank == 0:
            print(json.dumps({"device_loop": device_loop_report(args.workload, device)}), flush=True)
        return

    def measure(name: str, K: int, W: int, with_e2e: bool, sample_clocks: bool, reps: int, w=None):
        w = get_workload(name) if w is None else w
        n_sched = schedule_length(w)
        K = max(1, min(K, n_sched - W))
        total = W + K
        sb = StepBench(w, total, device, seed_shift=replicas.replica_seed_shift(rank))
        ev = lambda: torch.cuda.Event(enable_timing=True)  # noqa: E731
        stream = torch.cuda.current_stream()

        # pass 0: untimed, logs the bitmaps so that the algorithmic bytes are known; also a warm-up
        sb.reset()
        for i in range(total):
            sb.step(i, log_masks=True)
        torch.cuda.synchronize()
        per_layer_bytes = sb.algorithmic_bytes(range(total))
        step_bytes = [b * w.layers for b in per_layer_bytes]
        timed_bytes = sum(step_bytes[W:])
        nact_mean = sb.nact_log[W:].float().mean(dim=1).cpu().tolist()
        status = sb.sess.status(clear=True)

        # pass 1 (the number): reps x (W warm-up steps, exactly K timed steps), device-resident inputs,
        # every step one CUDA graph (frontier + build_masks + layers x attention)
        sampler = ClockSampler(local) if sample_clocks else None
        l0 = fdc.fdc_launch_count()
        runs, graphed = timed_region(sb, W, K, reps, not args.no_graphs, sampler,
                                     (lambda: dist.barrier()) if world > 1 else None)
        clocks = sampler.stop() if sampler is not None else None
        launches_per_region = (fdc.fdc_launch_count() - l0)
        # kernels per timed region: counted on an eager region (a graph replay launches what was captured)
        sb.reset()
        for i in range(W):
            sb.step(i)
        l1 = fdc.fdc_launch_count()
        for i in range(W, total):
            sb.step(i)
        torch.cuda.synchronize()
        launches = fdc.fdc_launch_count() - l1
        totals = sorted(t for t, _ in runs)
        med_total = totals[len(totals) // 2]
        med_run = min(runs, key=lambda r: abs(r[0] - med_total))
        ms = replicas.max_over_ranks(med_total, device)                 # the job's time: the slowest replica
        replicas.barrier()
        phases = phase_report(w, med_run[1], per_layer_bytes[W:], nact_mean)

        # pass 1b (context only): the same steps with kv_append as a kernel of its own
        ms_separate = None
        if FUSED_APPEND and world == 1 and args.separate_too:
            sb.sess.set_fused_append(False)
            sb.graphs.clear()
            r2, _ = timed_region(sb, W, K, 1, not args.no_graphs)
            ms_separate = r2[0][0]
            sb.sess.set_fused_append(True)
            sb.graphs.clear()

        # pass 2: per-launch duration of the dominant kernel (split-KV pass) in isolation: CUDA events
        # recorded by the library itself on the launching stream around every such launch (stream
        # launches; the events also keep consecutive launches from overlapping)
        n_iso = min(K, 12)
        sb.reset()
        for i in range(W):
            sb.step(i)
        torch.cuda.synchronize()
        fdc.fdc_profile(sb.sess.plan, True)
        for i in range(W, W + n_iso):
            sb.step(i)
        prof = fdc.fdc_profile_read(sb.sess.plan)
        fdc.fdc_profile(sb.sess.plan, False)
        split_ms, split_n = prof["split_ms"], prof["split_launches"]
        comb_ms = prof["combine_ms"]
        roof = None
        if split_n:
            iso_bytes = sum(step_bytes[W:W + n_iso]) / split_n
            iso_gbs = iso_bytes / (split_ms / split_n * 1e-3) / 1e9
            n_launch = K * w.layers
            avg_bytes = timed_bytes / n_launch
            in_step_us = ms / n_launch * 1e3
            in_step_gbs = avg_bytes / (in_step_us * 1e-6) / 1e9
            tc = w.dtype == "bf16" and w.head_dim == 128
            traffic = None
            if tc and kernel_source_hash() == NCU_TRAFFIC["kernel_sha256_16"]:
                traffic = int(avg_bytes * NCU_TRAFFIC["dram_bytes_per_algorithmic_byte"])
            kname = ("attn_tc_kernel (tcgen05 split-KV pass; appends the pass's rows and merges its partials itself)" if tc
                     else "attn_ref_kernel (CUDA-core split-KV pass)")
            roof = {"kernel": kname, "bound": "hbm", "achieved": round(in_step_gbs, 1), "peak": peak, "unit": "GB/s",
                    "frac": round(in_step_gbs / peak, 4), "peak_source": peak_src,
                    "frac_is": "frac_in_step: timed region / attention launches; frontier + build_masks (2 small kernels per "
                               "step, < 1 %) are inside the region",
                    "traffic": traffic, "launches": n_launch, "avg_launch_us": round(in_step_us, 2),
                    "algorithmic_bytes_per_launch": int(avg_bytes),
                    "frac_in_step": round(in_step_gbs / peak, 4),
                    "frac_isolated_launch": round(iso_gbs / peak, 4),
                    "isolated": {"achieved": round(iso_gbs, 1), "avg_launch_us": round(split_ms / split_n * 1e3, 2),
                                 "launches": split_n, "how": "CUDA events around every launch (no overlap with its neighbours)"},
                    "combine_avg_launch_us": None if tc else round(comb_ms / split_n * 1e3, 2),
                    "frac_of_nominal_8TBs": round(in_step_gbs / NOMINAL_HBM_GBS, 4)}

        # host side: how long the calling thread needs to issue one pass (stream launches, no graph)
        sb.reset()
        for i in range(W):
            sb.step(i)
        torch.cuda.synchronize()
        sb.sess.use_stream(stream)
        n_host = min(K, 10)
        t0 = time.perf_counter()
        for i in range(W, W + n_host):
            sb.step(i)
        host_issue_us = (time.perf_counter() - t0) / n_host * 1e6
        torch.cuda.synchronize()
        sb.sess.use_stream(None)

        # pass 3: end to end through the C ABI with HOST buffers: every step copies its q / k_new /
        # v_new from pinned host memory and reads the step's attention output back.  The copies run
        # on a second stream with two sets of device buffers, so that the inputs of step i + 1 and the
        # output of step i - 1 move while step i computes; all of them lie inside the timed region.
        e2e = None
        if with_e2e:
            Ke = min(K, 40)
            hq_ = sb.q[W:W + Ke].cpu().pin_memory()
            hk_ = sb.kn[W:W + Ke].cpu().pin_memory()
            hv_ = sb.vn[W:W + Ke].cpu().pin_memory()
            hout = torch.empty_like(sb.out, device="cpu").pin_memory()
            din = [(torch.empty_like(sb.q[0]), torch.empty_like(sb.kn[0]), torch.empty_like(sb.vn[0])) for _ in range(2)]
            dout = [sb.out, torch.empty_like(sb.out)]
            copies = torch.cuda.Stream(device)
            in_ready = [ev() for _ in range(2)]      # inputs of a buffer set have arrived
            computed = [ev() for _ in range(2)]      # the step that used a buffer set is done
            out_read = [ev() for _ in range(2)]      # the output buffer has been copied to the host

            def fetch(i):                            # on the copy stream: inputs of timed step i
                b = i & 1
                with torch.cuda.stream(copies):
                    if i >= 2:
                        copies.wait_event(computed[b])       # step i - 2 no longer reads this set
                    for dst, src in zip(din[b], (hq_[i], hk_[i], hv_[i])):
                        dst.copy_(src, non_blocking=True)
                    in_ready[b].record(copies)

            sb.reset()
            for i in range(W):
                sb.step(i)
            if world > 1:
                dist.barrier()
            torch.cuda.synchronize()
            sb.sess.use_stream(stream)
            e0, e1 = ev(), ev()
            e0.record(stream)
            copies.wait_event(e0)
            fetch(0)
            for i in range(Ke):
                b = i & 1
                if i + 1 < Ke:
                    fetch(i + 1)
                stream.wait_event(in_ready[b])
                if i >= 2:
                    stream.wait_event(out_read[b])           # the output of step i - 2 has left this buffer
                sb.step(W + i, *din[b], out=dout[b])
                computed[b].record(stream)
                with torch.cuda.stream(copies):
                    copies.wait_event(computed[b])
                    hout.copy_(dout[b], non_blocking=True)
                    out_read[b].record(copies)
            stream.wait_stream(copies)                       # the last output is on the host
            e1.record(stream)
            torch.cuda.synchronize()
            sb.sess.use_stream(None)
            ems = replicas.max_over_ranks(e0.elapsed_time(e1), device)
            h2d = sum(t.numel() for t in din[0]) * w.esize
            d2h = sb.out.numel() * w.esize
            e2e = {"value": round(world * sum(step_bytes[W:W + Ke]) / (ems * 1e-3) / 1e9, 1), "unit": UNIT, "steps": Ke,
                   "ms_per_step": round(ems / Ke, 4), "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                   "launch": "stream launches from the calling thread (no graph: the buffers alternate)"}

        value = world * timed_bytes / (ms * 1e-3) / 1e9
        res = {"workload": name, "value": value, "ms": ms, "ms_per_step": ms / K, "launches": launches, "K": K, "W": W,
               "roofline": roof, "e2e": e2e, "clocks": clocks, "status": status, "graphs": graphed,
               "region_ms": {"median": round(med_total, 3), "min": round(totals[0], 3), "max": round(totals[-1], 3), "repeats": len(totals)},
               "phases": phases, "host_issue_us_per_step": round(host_issue_us, 1),
               "host_issue_us_per_layer": round(host_issue_us / w.layers, 2),
               "schedule_passes": n_sched,
               "step_us": round(ms / K * 1e3, 1), "layer_step_us": round(ms / K / w.layers * 1e3, 2),
               "layer_step_us_separate_append": None if ms_separate is None else round(ms_separate / K / w.layers * 1e3, 2),
               "bytes_per_step": int(timed_bytes / K), "avg_active_per_scene": float(np.mean(nact_mean)),
               "pct_of_8TBs": round(100 * value / world / NOMINAL_HBM_GBS, 1),
               "pct_of_measured_copy": round(100 * value / world / peak, 1)}
        sb.graphs.clear()
        sb.sess.close()
        del sb
        torch.cuda.empty_cache()
        return res, w

    main, w = measure(args.workload, args.steps, args.warmup, True, True, args.repeats)
    also = {}
    keep = ("value", "step_us", "layer_step_us", "layer_step_us_separate_append", "bytes_per_step", "pct_of_8TBs",
            "pct_of_measured_copy", "roofline", "avg_active_per_scene", "region_ms", "phases", "host_issue_us_per_layer",
            "schedule_passes", "K", "graphs")
    if not args.no_also and world == 1:
        for other in ("cfg1", "cfg3"):
            if other == args.workload:
                continue
            r, _ = measure(other, args.steps, max(3, min(args.warmup, 5)), False, False, 3)
            also[other] = {k: (round(v, 2) if isinstance(v, float) else v) for k, v in r.items() if k in keep}
            also[other]["workload"] = WORKLOAD_TEXT[other]
        # Sec. 3.1 / 3.3 at scale: pre-filled field-name rows at the head of every slot, and no lengths
        # given, so that every field is cut off at its slot (pad or truncate)
        global USE_LENS
        from paper_2602_02864_b200 import workloads as wl
        wf = wl.cfg2_batched()
        rng = np.random.default_rng(wf.seed)
        wf.n_fixed = [int(x) for x in rng.integers(3, 7, size=wf.n_nodes)]
        USE_LENS = False
        try:
            r, _ = measure("cfg2_fixed_rows_truncated", args.steps, max(3, min(args.warmup, 5)), False, False, 3, w=wf)
        finally:
            USE_LENS = True
        also["cfg2_fixed_rows_truncated"] = {k: (round(v, 2) if isinstance(v, float) else v) for k, v in r.items() if k in keep}
        also["cfg2_fixed_rows_truncated"]["workload"] = ("configs[2] shapes with 3-6 pre-filled field-name rows per slot (n_fixed) and no "
                                                         "lengths given: every field runs to its 96-row slot")
        # Sec. 4.3 (future work): a fast response decoded beside the CoT.  One more source field of 24
        # tokens: the schedule keeps its length, the first 24 passes carry one more query row per scene.
        wd = wl.cfg2_dual_response()
        r, _ = measure("cfg2_dual_response", args.steps, max(3, min(args.warmup, 5)), False, False, 3, w=wd)
        also["cfg2_dual_response"] = {k: (round(v, 2) if isinstance(v, float) else v) for k, v in r.items() if k in keep}
        also["cfg2_dual_response"]["workload"] = ("configs[2] plus one independent 24-token response field decoded concurrently "
                                                  "(7 instead of 6 branches in the first passes)")
        also["cfg2_dual_response"]["passes_without_the_response_field"] = main["schedule_passes"]
        also["cfg4_sweep"] = cfg4_sweep(args, device, peak)
        also["device_loop"] = device_loop_report(args.workload, device)

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        cpu = cpu_baseline(args.workload, budget_s=12.0)

    if rank == 0:
        line = {
            "metric": METRIC, "value": round(main["value"], 1), "unit": UNIT, "n_gpus": world, "steps": main["K"],
            "warmup": main["W"], "ms_per_step": round(main["ms_per_step"], 4), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
            "config": {"workload": WORKLOAD_TEXT[args.workload], "scenes_per_gpu": w.batch, "layers": w.layers,
                       "l2": "inputs larger than L2: each layer reads its own KV buffer, %.1f GB of KV per step"
                             % (main["bytes_per_step"] / 1e9),
                       "parallelism": "replicas" if world > 1 else "1 GPU",
                       "launch": "one CUDA graph per step, replayed in order" if main["graphs"] else "stream launches",
                       "timing": "%d repeats of (reset, %d warm-up steps, %d timed steps of the schedule's %d); value from the median repeat"
                                 % (main["region_ms"]["repeats"], main["W"], main["K"], main["schedule_passes"]),
                       "step": ("frontier + build_masks + layers x (kv_append recorded, carried out inside decode_attn "
                                "[fdc_set_fused_append]: one kernel that appends, runs the split-KV pass and combines)")
                               if FUSED_APPEND else
                               "frontier + build_masks + layers x (kv_append + decode_attn[split-KV pass with the combine fused in])"},
            "step_us": main["step_us"], "layer_step_us": main["layer_step_us"],
            "layer_step_us_separate_append": main["layer_step_us_separate_append"],
            "region_ms": main["region_ms"], "phases": main["phases"],
            "host_issue_us_per_step": main["host_issue_us_per_step"],
            "bytes_per_step": main["bytes_per_step"], "avg_active_branches_per_scene": round(main["avg_active_per_scene"], 2),
            "pct_of_8TBs": main["pct_of_8TBs"], "pct_of_measured_copy": main["pct_of_measured_copy"],
            "roofline": main["roofline"], "cpu_baseline": cpu, "e2e": main["e2e"], "clocks": main["clocks"],
            "gpu_launches": int(main["launches"]), "device_status": main["status"], "also": also,
            "paper_context": "paper reports 3.1-4.1x CoT speedup end to end on 1x A100 80GB (bf16); no kernel-level number",
        }
        print(json.dumps(line), flush=True)


def device_loop_report(name: str, device):
    """Algorithm 1's whole loop as ONE graph launch (a WHILE node kept going by fdc_loop_condition)
    against the same passes replayed from the host as one graph each.  Both decode the workload's
    whole schedule from fdc_state_init to the last pass with one set of per-pass inputs; timed with
    CUDA events from the reset to the end, median of 3."""
    import torch
    from paper_2602_02864_b200.device_loop import DeviceLoop
    w = get_workload(name)
    n_pass = schedule_length(w)
    sb = StepBench(w, 1, device)
    stream = torch.cuda.current_stream()
    sb.sess.use_stream(stream)
    sb.reset()
    sb.step(0)                                   # eager once
    torch.cuda.synchronize()
    sb.sess.use_stream(None)
    g = sb.capture(0)                            # frontier + build_masks + layers x (append, attention)

    def body(st):
        sb.layers_pass(0)
        sb.schedule_pass()

    loop = DeviceLoop(sb.sess, body, int(sum(w.slot_cap)))
    sb.sess.use_stream(stream)

    def run_host():
        sb.reset()
        for _ in range(n_pass):
            g.replay()

    def run_device():
        sb.reset()
        sb.schedule_pass()
        loop.launch(stream)

    res = {}
    for key, fn in (("host_replays_one_graph_per_pass", run_host), ("device_loop_one_graph_launch", run_device)):
        fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(3):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            fn()
            e1.record(stream)
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        ms = sorted(ts)[1]
        res[key] = {"whole_schedule_ms": round(ms, 3), "layer_step_us": round(ms / n_pass / w.layers * 1e3, 2)}
    res["passes_by_host_arithmetic"] = n_pass
    res["passes_counted_on_device"] = int(loop.passes.item())
    res["device_status"] = sb.sess.status(clear=True)
    res["workload"] = WORKLOAD_TEXT[name] + "; every pass reads the same q / k_new / v_new buffers"
    sb.sess.use_stream(None)
    loop.close()
    sb.graphs.clear()
    sb.sess.close()
    del sb
    torch.cuda.empty_cache()
    return res


# configs[4]: prefix x branches x scenes.  A bounded part of the grid: every prefix x branches at 8
# scenes, and four corners at 1 and 64 scenes.
SWEEP_PREFIX = (1024, 4096, 16384, 32768)
SWEEP_BRANCHES = (1, 4, 8, 16, 32)
SWEEP_CORNERS = ((1024, 1, 1), (32768, 32, 64), (4096, 32, 64), (16384, 4, 64))
L2_BYTES = 126 << 20


def cfg4_sweep(args, device, peak):
    """Sec. 4.3 on synthetic templates: `branches` independent 64-token fields decoded in parallel
    (64 passes, `branches` tokens each) against the same fields decoded one after the other (the chain
    template: 64 x branches passes of one token, i.e. ordinary autoregressive decoding).  Per point a
    sample of passes spread evenly over each schedule is timed (their per-layer part as one CUDA graph,
    median of 3 replays; the cache of every layer is a buffer of its own, enough of them to exceed L2)."""
    import dataclasses
    import torch
    from paper_2602_02864_b200 import workloads as wl
    points = [(P, B, 8) for P in SWEEP_PREFIX for B in SWEEP_BRANCHES] + list(SWEEP_CORNERS)
    if args.sweep_points:
        points = [tuple(int(x) for x in pt.split(",")) for pt in args.sweep_points.split(";")]
    n_samples = 6
    rows = []
    for idx, (P, B, Bt) in enumerate(points):
        row = {"prefix": P, "branches": B, "scenes": Bt}
        for chain in (False, True):
            if chain and B == 1:
                row["chain"] = dict(row["parallel"])                     # one field: the two templates coincide
                continue
            w0 = wl.cfg4_sweep(P, B, Bt, chain=chain, point=idx)
            layer_kv = 2 * Bt * w0.hkv * w0.rows * w0.head_dim * w0.esize
            layers = int(min(48, max(2, -(-3 * L2_BYTES // (2 * layer_kv)))))      # >= 1.5 x L2 of distinct KV per step
            w = dataclasses.replace(w0, layers=layers)
            n_sched = 64 * B if chain else 64
            sample = sorted(set(int(round(x)) for x in np.linspace(0, n_sched - 1, n_samples)))
            sb = StepBench(w, len(sample), device, cheap_fill=True)
            stream = torch.cuda.current_stream()
            sb.sess.use_stream(stream)
            sb.reset()
            times, byts = [], []
            k = 0
            for step in range(n_sched):
                sb.schedule_pass(k if step in sample else None)
                if step not in sample:
                    continue
                sb.layers_pass(k)                                           # eager once (also appends the rows)
                torch.cuda.synchronize()
                try:
                    sb.sess.use_stream(None)
                    g = sb.capture(k, "layers")
                    sb.sess.use_stream(stream)
                    run = g.replay
                except Exception:
                    sb.sess.use_stream(stream)
                    run = (lambda kk=k: sb.layers_pass(kk))
                run()
                ts = []
                for _ in range(3):
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record(stream)
                    run()
                    e1.record(stream)
                    torch.cuda.synchronize()
                    ts.append(e0.elapsed_time(e1))
                times.append(sorted(ts)[1] / layers * 1e3)                  # us per layer-step
                k += 1
            byts = sb.algorithmic_bytes(range(len(sample)))
            status = sb.sess.status(clear=True)
            sb.sess.use_stream(None)
            sb.graphs.clear()
            sb.sess.close()
            del sb
            torch.cuda.empty_cache()
            us = float(np.mean(times))
            mb = float(np.mean(byts)) / 1e6
            gbs = float(np.mean(byts)) / (us * 1e-6) / 1e9
            row["chain" if chain else "parallel"] = {
                "passes": n_sched, "layer_step_us": round(us, 2), "MB_per_launch": round(mb, 1), "GBs": round(gbs, 1),
                "frac_of_measured": round(gbs / peak, 3), "pct_of_8TBs": round(100 * gbs / NOMINAL_HBM_GBS, 1),
                "attention_us_per_layer_whole_schedule": round(us * n_sched, 1), "layers_timed": layers,
                "latency_bound": mb < 64.0, "device_status": status}
        par, ch = row["parallel"], row["chain"]
        row["critical_path_tokens"] = {"parallel": par["passes"], "chain": ch["passes"]}
        row["avg_parallel_degree"] = float(B)
        row["speedup_over_chain"] = round(ch["attention_us_per_layer_whole_schedule"] / par["attention_us_per_layer_whole_schedule"], 2)
        rows.append(row)
        log("cfg4", row["prefix"], row["branches"], row["scenes"], "par", par["layer_step_us"], "us", par["GBs"], "GB/s | chain",
            ch["layer_step_us"], "us | speedup", row["speedup_over_chain"], "of", B)
    return {"what": "configs[4]: B independent 64-token fields in parallel (64 passes) vs the same fields in a chain (64 x B passes); "
                    "32 q / 8 KV heads, D 128, bf16; attention time per layer over the whole schedule, from 6 sampled passes each",
            "fig4_analogue": "attention time is proportional to the passes on the critical path (Sec. 4.3, Fig. 4a) and the speed-up "
                             "over the chain follows the average parallel degree from below (Fig. 4b): speedup_over_chain vs avg_parallel_degree",
            "points": rows}


def cpu_baseline(name: str, budget_s: float = 12.0, steps=None, warmup=0):
    """The float64 CPU checker as it stands, timed on this machine's host cores on a bounded sample
    of the workload: whole (scene, layer) attention calls at the first pass of the schedule
    (widest frontier, prefix + first template rows visible)."""
    import torch
    from oracle import attention as oatt
    from oracle import schedule as sch
    from paper_2602_02864_b200 import workloads as wl
    w = get_workload(name)
    passes = sch.simulate(w.n_nodes, w.edges, w.lens[0].tolist(), w.n_fixed)
    tab = sch.pass_tables(w.n_nodes, w.edges, w.slot_cap, w.lens[0].tolist(), w.n_fixed, w.prefix_len, passes[0])
    A = len(passes[0])
    g = torch.Generator().manual_seed(w.seed)
    K = (torch.randn((w.hkv, w.rows, w.head_dim), generator=g) * w.kv_scale).to(w.torch_dtype).float().numpy()
    V = (torch.randn((w.hkv, w.rows, w.head_dim), generator=g) * w.kv_scale).to(w.torch_dtype).float().numpy()
    q = torch.randn((A, w.hq, w.head_dim), generator=g).to(w.torch_dtype).float().numpy()
    row_bytes = 2 * w.hkv * w.head_dim * w.esize
    vis_rows = int(tab["vis"].any(axis=0).sum())
    call_bytes = vis_rows * row_bytes + 2 * A * w.hq * w.head_dim * w.esize + A * row_bytes + A * tab["mask"].shape[1] * 8
    oatt.attention(q, K, V, tab["vis"], w.softmax_scale)            # builds/loads the library, warms caches
    for _ in range(warmup):
        oatt.attention(q, K, V, tab["vis"], w.softmax_scale)
    n, t0 = 0, time.perf_counter()
    while True:
        oatt.attention(q, K, V, tab["vis"], w.softmax_scale)
        n += 1
        el = time.perf_counter() - t0
        if (steps is not None and n >= steps) or (steps is None and el >= budget_s):
            break
    cores = int(oatt.attention.last_threads)
    return {"value": round(n * call_bytes / el / 1e9, 4), "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{n} (scene, layer) attention calls of {name} at the first pass ({A} branches x {w.hq} heads, "
                      f"{vis_rows} visible rows), float64, {el:.1f} s",
            "ms_per_call": round(el / n * 1e3, 2), "calls": n}


def run_reference(args, rank: int):
    """`--impl reference`: the CPU checker timed on the host cores; each step is one bounded sample."""
    if rank != 0:
        return
    cb = cpu_baseline(args.workload, steps=args.steps, warmup=min(args.warmup, 2))
    w = get_workload(args.workload)
    line = {"impl": "reference", "metric": METRIC, "value": cb["value"], "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": cb["ms_per_call"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD_TEXT[args.workload], "step": "one (scene, layer) attention call of the first pass",
                       "scenes_per_gpu": w.batch, "layers": w.layers},
            "cpu_baseline": cb, "e2e": {"value": cb["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200, help="timed steps (clamped to what the schedule has after the warm-up)")
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--repeats", type=int, default=7, help="repetitions of the timed region (median reported)")
    ap.add_argument("--no-graphs", action="store_true", help="launch from the calling thread instead of replaying CUDA graphs")
    ap.add_argument("--separate-too", action="store_true", help="also time the steps with kv_append as a kernel of its own")
    ap.add_argument("--sweep-points", default=None, help="configs[4] points to run instead of the default grid: 'P,B,Bt;P,B,Bt;...'")
    ap.add_argument("--workload", default="cfg2", choices=["cfg0", "cfg1", "cfg2", "cfg3"])
    ap.add_argument("--impl", default="fdc", choices=["fdc", "reference"])
    ap.add_argument("--no-also", action="store_true", help="skip the short runs of the other configurations")
    ap.add_argument("--only-device-loop", action="store_true", help="run only the whole-schedule comparison (host-replayed graphs vs one device loop)")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU baseline leg")
    ap.add_argument("--separate-append", action="store_true",
                    help="launch kv_append as a kernel of its own instead of inside the attention kernel")
    ap.add_argument("--layers", type=int, default=None,
                    help="run only this many layers of the configuration (small ncu captures; not a bench number)")
    args = ap.parse_args()
    global LAYERS_OVERRIDE
    LAYERS_OVERRIDE = args.layers
    global FUSED_APPEND
    FUSED_APPEND = not args.separate_append
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    if args.impl == "reference":
        run_reference(args, rank)
        return
    if args.warmup < 3:
        args.warmup = 3
    if world > 1:
        import torch
        import torch.distributed as dist
        torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", 0)))
        dist.init_process_group("nccl")
    run_fdc(args, rank, world)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
