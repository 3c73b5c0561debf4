"""ctypes front of the float64 attention checker (attention.c).  TEST INFRASTRUCTURE ONLY."""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "attention.c")
_SO = os.path.join(_HERE, "_attention.so")
_lib: Optional[ctypes.CDLL] = None


def build(force: bool = False) -> str:
    """Compile attention.c with gcc (-O2, OpenMP) next to its source."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", _SRC,
                               "-o", tmp, "-lm"])
        os.replace(tmp, _SO)
    return _SO


def _load() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.fdc_oracle_attention.restype = ctypes.c_int
        lib.fdc_oracle_attention.argtypes = [ctypes.c_void_p] * 4 + [ctypes.c_int] * 5 + [
            ctypes.c_double, ctypes.c_void_p, ctypes.c_int]
        _lib = lib
    return _lib


def attention(q: np.ndarray, K: np.ndarray, V: np.ndarray, vis: np.ndarray, scale: float,
              nthreads: int = 0) -> np.ndarray:
    """Masked softmax attention of one scene, one layer, in float64.

    q   float32 [A][Hq][D]   packed queries (one per parallel field)
    K,V float32 [Hkv][R][D]  the scene's cache for this layer
    vis bool    [A][R]       which rows each query may attend
    returns float64 [A][Hq][D].  Raises if some query sees no row."""
    q = np.ascontiguousarray(q, dtype=np.float32)
    K = np.ascontiguousarray(K, dtype=np.float32)
    V = np.ascontiguousarray(V, dtype=np.float32)
    vis8 = np.ascontiguousarray(vis, dtype=np.uint8)
    A, Hq, D = q.shape
    Hkv, R, D2 = K.shape
    assert D2 == D and V.shape == K.shape and vis8.shape == (A, R) and Hq % Hkv == 0
    out = np.zeros((A, Hq, D), dtype=np.float64)
    if A == 0:
        return out
    rc = _load().fdc_oracle_attention(q.ctypes.data, K.ctypes.data, V.ctypes.data, vis8.ctypes.data,
                                      A, Hq, Hkv, R, D, float(scale), out.ctypes.data, int(nthreads))
    if rc < 0:
        raise ValueError("a query has an empty visibility set")
    attention.last_threads = rc
    return out


attention.last_threads = 0
