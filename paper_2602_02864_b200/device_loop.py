"""Algorithm 1's decode loop as ONE CUDA graph launch: a WHILE conditional node whose body is one
pass (the caller's launches) and whose condition the library's fdc_loop_condition sets from
fdc_frontier's `all_done`, so that the host takes no part between the first pass and the last.

Only graph plumbing lives here (through cuda-python's runtime bindings): the graph, the
conditional handle, the capture of the body.  Everything the body computes is launched by the
caller's `body` callable on the stream it is given."""
from __future__ import annotations

from typing import Callable

import torch

from . import fdc

try:
    from cuda.bindings import runtime as _rt
except ImportError:                                   # older cuda-python layout
    from cuda import cudart as _rt


def _ok(res, what: str):
    err = res[0]
    if int(err) != 0:
        raise RuntimeError(f"{what}: {_rt.cudaGetErrorString(err)[1].decode()}")
    return res[1] if len(res) == 2 else res[1:]


class DeviceLoop:
    """while (fields are ready) { body }   as an executable CUDA graph.

    sess        the DecodeSession whose plan and `all_done` the loop test reads
    body        callable(stream): launches ONE pass on `stream` (a torch.cuda.Stream): the model's
                kernels with fdc_kv_append / fdc_decode_attn per layer for the pass whose tables are
                current, then fdc_frontier and fdc_build_masks for the next pass.  It is called once,
                under stream capture: no allocation, no synchronisation, no host reads.
    max_passes  upper bound of the loop (the sum of the slot capacities is always enough)

    Before launch() the caller runs fdc_state_init, fdc_frontier and fdc_build_masks for the first
    pass.  `passes` (int32 [1], device) counts the passes the loop decoded."""

    def __init__(self, sess: "fdc.DecodeSession", body: Callable[[torch.cuda.Stream], None], max_passes: int):
        self.sess = sess
        self.passes = torch.zeros(1, dtype=torch.int32, device=sess.device)
        self._exec = None
        self._graph = None
        with torch.cuda.device(sess.device):
            stream = torch.cuda.Stream(device=sess.device)
            graph = _ok(_rt.cudaGraphCreate(0), "cudaGraphCreate")
            self._graph = graph
            # default value 1, applied at the start of every launch (flag cudaGraphCondAssignDefault = 1)
            handle = _ok(_rt.cudaGraphConditionalHandleCreate(graph, 1, 1), "cudaGraphConditionalHandleCreate")
            params = _rt.cudaGraphNodeParams()
            params.type = _rt.cudaGraphNodeType.cudaGraphNodeTypeConditional
            params.conditional.handle = handle
            params.conditional.type = _rt.cudaGraphConditionalNodeType.cudaGraphCondTypeWhile
            params.conditional.size = 1
            _ok(_rt.cudaGraphAddNode(graph, None, 0, params), "cudaGraphAddNode(conditional)")
            body_graph = params.conditional.phGraph_out[0]
            raw = _rt.cudaStream_t(stream.cuda_stream)
            stream.wait_stream(torch.cuda.current_stream(sess.device))
            _ok(_rt.cudaStreamBeginCaptureToGraph(raw, body_graph, None, None, 0,
                                                  _rt.cudaStreamCaptureMode.cudaStreamCaptureModeThreadLocal),
                "cudaStreamBeginCaptureToGraph")
            try:
                with torch.cuda.stream(stream):
                    body(stream)
                    fdc.fdc_loop_condition(sess.plan, sess.all_done, self.passes, max_passes, int(handle), stream)
            finally:
                res = _rt.cudaStreamEndCapture(raw)
            _ok(res, "cudaStreamEndCapture")
            self._exec = _ok(_rt.cudaGraphInstantiate(graph, 0), "cudaGraphInstantiate")
        self._keep = (stream, handle)

    def launch(self, stream=None) -> None:
        """Zeroes the pass counter and launches the loop on `stream` (default: torch's current stream)."""
        st = torch.cuda.current_stream(self.sess.device) if stream is None else stream
        with torch.cuda.stream(st):
            self.passes.zero_()
        _ok(_rt.cudaGraphLaunch(self._exec, _rt.cudaStream_t(st.cuda_stream)), "cudaGraphLaunch")

    def close(self) -> None:
        if self._exec is not None:
            _rt.cudaGraphExecDestroy(self._exec)
            self._exec = None
        if self._graph is not None:
            _rt.cudaGraphDestroy(self._graph)
            self._graph = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
