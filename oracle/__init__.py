"""CPU checker for the dependency-masked parallel-decoding path (TEST INFRASTRUCTURE ONLY).

Plain, slow, float64 / exact-integer restatement of what the path computes, written from
the paper: Algorithm 1 (ready-set scheduling on the field DAG, Sec. 3.2), Eq. 1 (a token
may attend a field iff that field is an ancestor, Sec. 3.3), fixed slots / position ids /
invisible padding (Sec. 3.3), and ordinary softmax attention restricted to the visible
rows.  It shares no code with the CUDA library and never imports it.  Only tests, the
smoke check and the benchmark's CPU-baseline leg may use it; the product path must not.

Every function here is pinned by CPU tests against something other than itself (brute
force on tiny inputs, closed forms, textbook causal attention, invariances); nothing in
this package is "parity unpinned".
"""
from . import schedule, attention, run  # noqa: F401
