"""Thin ctypes binding of libfdc.so: same names as the C ABI, argument marshalling only.

Every step of the path (scheduling, bitmaps, KV append, attention) runs in the library's
CUDA kernels; PyTorch is used here for device memory and streams.  Importing this module
loads the library and raises if it has not been built (there is no CPU fallback)."""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence, Tuple

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("FDC_LIBRARY", os.path.join(_HERE, "libfdc.so"))

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2602_02864_b200.build` "
                      "(there is no fallback path)")
_lib = ctypes.CDLL(LIB_PATH)

FDC_MAX_NODES, FDC_TILE_ROWS, FDC_MAX_QROWS, FDC_MAX_BATCH = 64, 64, 128, 4096
FDC_OK = 0
FDC_ERR_NULL, FDC_ERR_CYCLE, FDC_ERR_RANGE, FDC_ERR_SHAPE = -1, -2, -3, -4
FDC_ERR_DTYPE, FDC_ERR_WORKSPACE, FDC_ERR_CUDA, FDC_ERR_DEVICE = -5, -6, -7, -8
FDC_ERR_STATIC_LIMIT = -9
FDC_STATIC_WS_BYTES = 16 << 20
FDC_F32, FDC_BF16 = 0, 1
FDC_DEV_ROW_RANGE, FDC_DEV_FRONTIER_WIDE, FDC_DEV_LEN_RANGE, FDC_DEV_TIMEOUT = 1, 2, 4, 8
FDC_DEV_SCORE_RANGE = 16
FDC_DEV_TILE_LIST = 32
FDC_DEV_LOOP_LIMIT = 64

c_i32, c_i64, c_vp, c_sz = ctypes.c_int32, ctypes.c_int64, ctypes.c_void_p, ctypes.c_size_t


class fdc_graph_desc(ctypes.Structure):
    _fields_ = [("n_nodes", c_i32), ("n_edges", c_i32), ("edges", c_vp), ("slot_cap", c_vp),
                ("n_fixed", c_vp), ("prefix_len", c_i32), ("max_active", c_i32)]


class fdc_kv_desc(ctypes.Structure):
    _fields_ = [("k", c_vp), ("v", c_vp), ("dtype", c_i32), ("batch", c_i32), ("layers", c_i32),
                ("hkv", c_i32), ("hq", c_i32), ("head_dim", c_i32), ("rows", c_i32),
                ("stride_scene", c_i64), ("stride_layer", c_i64), ("stride_head", c_i64),
                ("stride_row", c_i64)]


class fdc_sizes(ctypes.Structure):
    _fields_ = [("cot_rows", c_i32), ("mask_words", c_i32), ("ntile_max", c_i32), ("max_active", c_i32),
                ("state_bytes", c_sz), ("mask_bytes", c_sz), ("umask_bytes", c_sz), ("tiles_bytes", c_sz)]


def _sig(name, restype, *argtypes):
    f = getattr(_lib, name)
    f.restype = restype
    f.argtypes = list(argtypes)
    return f


_plan_graph = _sig("fdc_plan_graph", c_i32, ctypes.POINTER(fdc_graph_desc), ctypes.POINTER(c_vp))
_plan_destroy = _sig("fdc_plan_destroy", c_i32, c_vp)
_plan_query = _sig("fdc_plan_query", c_i32, c_vp, c_i32, ctypes.POINTER(fdc_sizes))
_plan_tables = _sig("fdc_plan_tables", c_i32, c_vp, c_vp, c_vp, c_vp, c_vp)
_plan_critical_path = _sig("fdc_plan_critical_path", c_i32, c_vp, c_vp, ctypes.POINTER(c_i32), c_vp)
_state_init = _sig("fdc_state_init", c_i32, c_vp, c_i32, c_vp, c_vp, c_vp)
_frontier = _sig("fdc_frontier", c_i32, c_vp, c_i32, c_vp, c_vp, c_vp, c_vp, c_vp, c_vp, c_vp, c_vp, c_vp)
_build_masks = _sig("fdc_build_masks", c_i32, c_vp, c_i32, c_vp, c_vp, c_vp, c_vp, c_vp, c_vp)
_kv_append = _sig("fdc_kv_append", c_i32, c_vp, ctypes.POINTER(fdc_kv_desc), c_i32, c_vp, c_vp, c_vp, c_vp, c_vp)
_kv_write_fixed = _sig("fdc_kv_write_fixed", c_i32, c_vp, ctypes.POINTER(fdc_kv_desc), c_i32, c_vp, c_vp, c_vp)
_attn_ws = _sig("fdc_attn_workspace_bytes", c_i32, c_vp, ctypes.POINTER(fdc_kv_desc), ctypes.POINTER(c_sz))
_decode_attn = _sig("fdc_decode_attn", c_i32, c_vp, ctypes.POINTER(fdc_kv_desc), c_i32, c_vp, c_vp, c_vp, c_vp,
                    c_vp, c_vp, ctypes.c_float, c_vp, c_sz, c_vp)
_decode_attn_static = _sig("fdc_decode_attn_static", c_i32, c_vp, ctypes.POINTER(fdc_kv_desc), c_i32, c_vp, c_vp, c_vp,
                           c_vp, c_vp, c_vp, ctypes.c_float, c_vp)
_status = _sig("fdc_status", c_i32, c_vp, ctypes.POINTER(c_i32), c_i32, c_vp)
_set_attn_kernel = _sig("fdc_set_attn_kernel", c_i32, c_vp, c_i32)
_set_fused_append = _sig("fdc_set_fused_append", c_i32, c_vp, c_i32)
_kernel_name = _sig("fdc_kernel_name", ctypes.c_char_p, c_i32)
_profile = _sig("fdc_profile", c_i32, c_vp, c_i32)
_selftest_bounded_wait = _sig("fdc_selftest_bounded_wait", c_i32, c_vp, c_vp, c_vp)
_loop_condition = _sig("fdc_loop_condition", c_i32, c_vp, c_vp, c_vp, c_i32, ctypes.c_uint64, c_vp)
_profile_read = _sig("fdc_profile_read", c_i32, c_vp, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_float),
                     ctypes.POINTER(c_i32))
_launch_count = _sig("fdc_launch_count", c_i64)
_strerror = _sig("fdc_strerror", ctypes.c_char_p, c_i32)
_last_cuda_error = _sig("fdc_last_cuda_error", ctypes.c_char_p)


class FdcError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = f"{where}: {_strerror(code).decode()} ({code})"
        if code == FDC_ERR_CUDA:
            msg += f" [{_last_cuda_error().decode()}]"
        super().__init__(msg)


def _check(code: int, where: str) -> None:
    if code != FDC_OK:
        raise FdcError(code, where)


def _ptr(t) -> Optional[int]:
    """Raw address of a tensor / numpy array / int / None."""
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        return t.data_ptr()
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return int(t)


def _stream(stream) -> Optional[int]:
    """cudaStream_t of a torch stream / raw handle; None = torch's current stream (looked up per call:
    callers with a hot loop pass the handle, see DecodeSession.use_stream)."""
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return int(stream.cuda_stream) if hasattr(stream, "cuda_stream") else int(stream)


# --------------------------------------------------------------------------------------
# the C ABI, one Python function per entry point
# --------------------------------------------------------------------------------------

def fdc_plan_graph(n_nodes: int, edges: Sequence[Tuple[int, int]], slot_cap: Sequence[int],
                   n_fixed: Optional[Sequence[int]], prefix_len: int, max_active: int) -> int:
    """Returns the plan handle (an address).  The CUDA device current now owns the plan."""
    e = np.ascontiguousarray(np.array(list(edges), dtype=np.int32).reshape(-1, 2))
    c = np.ascontiguousarray(np.array(list(slot_cap), dtype=np.int32))
    f = None if n_fixed is None else np.ascontiguousarray(np.array(list(n_fixed), dtype=np.int32))
    desc = fdc_graph_desc(int(n_nodes), int(e.shape[0]), e.ctypes.data if e.size else None, c.ctypes.data,
                          None if f is None else f.ctypes.data, int(prefix_len), int(max_active))
    out = c_vp()
    _check(_plan_graph(ctypes.byref(desc), ctypes.byref(out)), "fdc_plan_graph")
    return out.value


def fdc_plan_destroy(plan: int) -> None:
    _check(_plan_destroy(plan), "fdc_plan_destroy")


def fdc_plan_query(plan: int, batch: int) -> fdc_sizes:
    s = fdc_sizes()
    _check(_plan_query(plan, batch, ctypes.byref(s)), "fdc_plan_query")
    return s


def fdc_plan_tables(plan: int, n_nodes: int):
    anc = np.zeros(n_nodes, np.uint64)
    par = np.zeros(n_nodes, np.uint64)
    base = np.zeros(n_nodes + 1, np.int32)
    indeg = np.zeros(n_nodes, np.int32)
    _check(_plan_tables(plan, anc.ctypes.data, par.ctypes.data, base.ctypes.data, indeg.ctypes.data),
           "fdc_plan_tables")
    return anc, par, base, indeg


def fdc_plan_critical_path(plan: int, lens: Sequence[int]):
    l = np.ascontiguousarray(np.array(list(lens), dtype=np.int32))
    fin = np.zeros(l.shape[0], np.int32)
    steps = c_i32()
    _check(_plan_critical_path(plan, l.ctypes.data, ctypes.byref(steps), fin.ctypes.data), "fdc_plan_critical_path")
    return steps.value, fin


def fdc_state_init(plan, batch, d_len, d_state, stream=None) -> None:
    _check(_state_init(plan, batch, _ptr(d_len), _ptr(d_state), _stream(stream)), "fdc_state_init")


def fdc_frontier(plan, batch, d_state, d_finish, d_n_active, d_node, d_tok_idx, d_kv_row, d_pos_id, d_all_done,
                 stream=None) -> None:
    _check(_frontier(plan, batch, _ptr(d_state), _ptr(d_finish), _ptr(d_n_active), _ptr(d_node), _ptr(d_tok_idx),
                     _ptr(d_kv_row), _ptr(d_pos_id), _ptr(d_all_done), _stream(stream)), "fdc_frontier")


def fdc_build_masks(plan, batch, d_state, d_mask, d_umask, d_tiles, d_ntiles, stream=None) -> None:
    _check(_build_masks(plan, batch, _ptr(d_state), _ptr(d_mask), _ptr(d_umask), _ptr(d_tiles), _ptr(d_ntiles),
                        _stream(stream)), "fdc_build_masks")


def fdc_kv_append(plan, kv: fdc_kv_desc, layer, d_n_active, d_kv_row, d_k_new, d_v_new, stream=None) -> None:
    _check(_kv_append(plan, ctypes.byref(kv), layer, _ptr(d_n_active), _ptr(d_kv_row), _ptr(d_k_new), _ptr(d_v_new),
                      _stream(stream)), "fdc_kv_append")


def fdc_kv_write_fixed(plan, kv: fdc_kv_desc, layer, d_k_fixed, d_v_fixed, stream=None) -> None:
    _check(_kv_write_fixed(plan, ctypes.byref(kv), layer, _ptr(d_k_fixed), _ptr(d_v_fixed), _stream(stream)),
           "fdc_kv_write_fixed")


def fdc_attn_workspace_bytes(plan, kv: fdc_kv_desc) -> int:
    b = c_sz()
    _check(_attn_ws(plan, ctypes.byref(kv), ctypes.byref(b)), "fdc_attn_workspace_bytes")
    return b.value


def fdc_decode_attn(plan, kv: fdc_kv_desc, layer, d_n_active, d_mask, d_tiles, d_ntiles, d_q, d_out, scale,
                    d_workspace, ws_bytes, stream=None) -> None:
    _check(_decode_attn(plan, ctypes.byref(kv), layer, _ptr(d_n_active), _ptr(d_mask), _ptr(d_tiles), _ptr(d_ntiles),
                        _ptr(d_q), _ptr(d_out), float(scale), _ptr(d_workspace), int(ws_bytes), _stream(stream)),
           "fdc_decode_attn")


def fdc_decode_attn_static(plan, kv: fdc_kv_desc, layer, d_n_active, d_mask, d_tiles, d_ntiles, d_q, d_out, scale,
                           stream=None) -> None:
    """fdc_decode_attn for callers that may not allocate device memory: the split partials go to
    the library's built-in 16 MiB buffer (shared by all calls on the GPU; overlapping calls race).
    Raises FdcError(FDC_ERR_STATIC_LIMIT) when the problem needs more scratch than that."""
    _check(_decode_attn_static(plan, ctypes.byref(kv), layer, _ptr(d_n_active), _ptr(d_mask), _ptr(d_tiles),
                               _ptr(d_ntiles), _ptr(d_q), _ptr(d_out), float(scale), _stream(stream)),
           "fdc_decode_attn_static")


def fdc_status(plan, clear: bool = False, stream=None) -> int:
    """Returns the sticky FDC_DEV_* bits (synchronises the stream)."""
    bits = c_i32()
    rc = _status(plan, ctypes.byref(bits), int(clear), _stream(stream))
    if rc not in (FDC_OK, FDC_ERR_DEVICE):
        raise FdcError(rc, "fdc_status")
    return bits.value


def fdc_set_attn_kernel(plan, which: int) -> None:
    _check(_set_attn_kernel(plan, which), "fdc_set_attn_kernel")


def fdc_set_fused_append(plan, on: bool) -> None:
    _check(_set_fused_append(plan, 1 if on else 0), "fdc_set_fused_append")


def fdc_selftest_bounded_wait(plan, d_outcome, stream=None) -> None:
    _check(_selftest_bounded_wait(plan, _ptr(d_outcome), _stream(stream)), "fdc_selftest_bounded_wait")


def fdc_loop_condition(plan, d_all_done, d_pass_count, max_passes: int, cond_handle: int, stream=None) -> None:
    _check(_loop_condition(plan, _ptr(d_all_done), _ptr(d_pass_count), int(max_passes), int(cond_handle), _stream(stream)),
           "fdc_loop_condition")


def fdc_kernel_name(which: int) -> Optional[str]:
    s = _kernel_name(which)
    return s.decode() if s else None


def fdc_profile(plan, enable: bool) -> None:
    _check(_profile(plan, int(enable)), "fdc_profile")


def fdc_profile_read(plan) -> dict:
    a, b, n = ctypes.c_float(), ctypes.c_float(), c_i32()
    _check(_profile_read(plan, ctypes.byref(a), ctypes.byref(b), ctypes.byref(n)), "fdc_profile_read")
    return {"split_ms": a.value, "combine_ms": b.value, "split_launches": n.value, "kernel": "split_kv"}


def fdc_launch_count() -> int:
    return int(_launch_count())


def fdc_strerror(code: int) -> str:
    return _strerror(code).decode()


# --------------------------------------------------------------------------------------
# buffer plumbing (allocation only; no arithmetic)
# --------------------------------------------------------------------------------------

def kv_desc_from_tensors(k: torch.Tensor, v: torch.Tensor, hq: int) -> fdc_kv_desc:
    """k, v: [batch][layers][hkv][rows][D] views with identical strides (D contiguous)."""
    assert k.dim() == 5 and k.shape == v.shape and k.stride() == v.stride() and k.stride(4) == 1
    dt = {torch.float32: FDC_F32, torch.bfloat16: FDC_BF16}[k.dtype]
    b, l, hkv, rows, d = k.shape
    return fdc_kv_desc(k.data_ptr(), v.data_ptr(), dt, b, l, hkv, hq, d, rows, k.stride(0), k.stride(1), k.stride(2),
                       k.stride(3))


class DecodeSession:
    """Owns the device buffers of one batch of scenes and forwards to the C ABI.

    plan / state / pass tables / masks / tile lists / workspace live here; the KV cache, the
    per-pass q, k_new, v_new and the output are the caller's tensors."""

    def __init__(self, n_nodes, edges, slot_cap, n_fixed, prefix_len, max_active, batch, device="cuda"):
        self.device = torch.device(device)
        self.batch, self.max_active, self.n_nodes = batch, max_active, n_nodes
        with torch.cuda.device(self.device):
            self.plan = fdc_plan_graph(n_nodes, edges, slot_cap, n_fixed, prefix_len, max_active)
        self.sizes = fdc_plan_query(self.plan, batch)
        dev = self.device
        self.state = torch.zeros(self.sizes.state_bytes, dtype=torch.uint8, device=dev)
        i32 = dict(dtype=torch.int32, device=dev)
        self.n_active = torch.zeros(batch, **i32)
        self.node = torch.zeros(batch, max_active, **i32)
        self.tok_idx = torch.zeros(batch, max_active, **i32)
        self.kv_row = torch.zeros(batch, max_active, **i32)
        self.pos_id = torch.zeros(batch, max_active, **i32)
        self.all_done = torch.zeros(1, **i32)
        W = self.sizes.mask_words
        self.mask = torch.zeros(batch, max_active, W, dtype=torch.int64, device=dev)
        self.umask = torch.zeros(batch, W, dtype=torch.int64, device=dev)
        self.tiles = torch.zeros(batch, self.sizes.ntile_max, **i32)
        self.ntiles = torch.zeros(batch, **i32)
        self.workspace = None
        self.ws_bytes = 0
        self.kv = None
        self._append_refs = None
        self.stream = None                   # None: torch's current stream at every call

    def close(self):
        if self.plan:
            fdc_plan_destroy(self.plan)
            self.plan = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def use_stream(self, stream) -> None:
        """Fixes the stream of all later calls (a torch stream, a raw cudaStream_t or None for "torch's
        current stream at every call"): the per-call look-up costs more than a small launch."""
        self.stream = None if stream is None else _stream(stream)

    def _st(self, stream):
        return self.stream if stream is None else stream

    def bind_cache(self, k: torch.Tensor, v: torch.Tensor, hq: int) -> None:
        self.kv = kv_desc_from_tensors(k, v, hq)
        self._k, self._v = k, v
        need = fdc_attn_workspace_bytes(self.plan, self.kv)
        if need > self.ws_bytes:
            self.workspace = torch.empty(need, dtype=torch.uint8, device=self.device)
            self.ws_bytes = need

    def init(self, lens: Optional[torch.Tensor], stream=None) -> None:
        """lens: int32 device tensor [batch][n_nodes] or None (fields run to their slot)."""
        self._lens = lens
        fdc_state_init(self.plan, self.batch, lens, self.state, self._st(stream))

    def frontier(self, finish: Optional[torch.Tensor] = None, stream=None) -> None:
        fdc_frontier(self.plan, self.batch, self.state, finish, self.n_active, self.node, self.tok_idx, self.kv_row,
                     self.pos_id, self.all_done, self._st(stream))

    def build_masks(self, stream=None) -> None:
        fdc_build_masks(self.plan, self.batch, self.state, self.mask, self.umask, self.tiles, self.ntiles, self._st(stream))

    def kv_append(self, layer, k_new, v_new, stream=None) -> None:
        fdc_kv_append(self.plan, self.kv, layer, self.n_active, self.kv_row, k_new, v_new, self._st(stream))
        self._append_refs = (k_new, v_new)      # a recorded (fused) append reads them in the next decode_attn

    def write_fixed(self, layer, k_fixed, v_fixed, stream=None) -> None:
        """The pre-filled field-name rows of one layer: [batch][hkv][sum n_fixed][D] each."""
        fdc_kv_write_fixed(self.plan, self.kv, layer, k_fixed, v_fixed, self._st(stream))

    def decode_attn(self, layer, q, out, scale, stream=None) -> None:
        fdc_decode_attn(self.plan, self.kv, layer, self.n_active, self.mask, self.tiles, self.ntiles, q, out, scale,
                        self.workspace, self.ws_bytes, self._st(stream))
        self._append_refs = None

    def set_fused_append(self, on: bool) -> None:
        """fdc_set_fused_append: kv_append is recorded and carried out by the next decode_attn."""
        fdc_set_fused_append(self.plan, on)

    def status(self, clear=False) -> int:
        return fdc_status(self.plan, clear)
