"""ctypes loader for the plain-C float64 oracle (oracle/sparq_oracle.c).

TEST INFRASTRUCTURE ONLY, like everything under ``oracle/``.  ``build()`` compiles the C file
with gcc into ``oracle/liboracle.so``; the wrappers take numpy arrays holding fp16 caches.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sparq_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle if the library is missing or older than its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.run(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"], check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.sparq_oracle_decode.restype = ctypes.c_int
        _lib.sparq_oracle_dense.restype = ctypes.c_int
        _lib.sparq_oracle_max_threads.restype = ctypes.c_int
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _u16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.float16
    return a.view(np.uint16)


def max_threads() -> int:
    return int(_load().sparq_oracle_max_threads())


def sparq_decode(q, K, V, seq_lens, r, k, v_bar=None, heads=None, n_threads=0):
    """q [B,Hq,d], K,V [B,Hkv,S_max,d] float16 arrays; seq_lens [B]; heads: optional [n,2]
    (b, h) pairs.  Returns a dict of per-unit arrays (see sparq_oracle.c)."""
    lib = _load()
    q16, K16, V16 = _u16(q), _u16(K), _u16(V)
    B, Hq, d = q.shape
    Hkv, S_max = K.shape[1], K.shape[2]
    sl = np.ascontiguousarray(seq_lens, dtype=np.int32)
    hd = None if heads is None else np.ascontiguousarray(heads, dtype=np.int32)
    n = B * Hq if hd is None else hd.shape[0]
    vb = None if v_bar is None else np.ascontiguousarray(v_bar, dtype=np.float64)
    out = np.zeros((n, d), dtype=np.float64)
    i1 = np.zeros((n, r), dtype=np.int32)
    i2 = np.zeros((n, max(k, 0)), dtype=np.int32)
    alpha = np.zeros(n, dtype=np.float64)
    gap_r = np.zeros(n, dtype=np.float64)
    gap_k = np.zeros(n, dtype=np.float64)
    rc = lib.sparq_oracle_decode(_p(q16), _p(K16), _p(V16), _p(vb), _p(sl), B, Hq, Hkv, d, S_max, r, k,
                                 _p(hd), n, _p(out), _p(i1), _p(i2), _p(alpha), _p(gap_r), _p(gap_k),
                                 int(n_threads))
    if rc != 0:
        raise ValueError("sparq_oracle_decode: bad argument")
    return dict(out=out, i1=i1, i2=i2, alpha=alpha, gap_r=gap_r, gap_k=gap_k)


def dense_decode(q, K, V, seq_lens, heads=None, n_threads=0):
    lib = _load()
    q16, K16, V16 = _u16(q), _u16(K), _u16(V)
    B, Hq, d = q.shape
    Hkv, S_max = K.shape[1], K.shape[2]
    sl = np.ascontiguousarray(seq_lens, dtype=np.int32)
    hd = None if heads is None else np.ascontiguousarray(heads, dtype=np.int32)
    n = B * Hq if hd is None else hd.shape[0]
    out = np.zeros((n, d), dtype=np.float64)
    rc = lib.sparq_oracle_dense(_p(q16), _p(K16), _p(V16), _p(sl), B, Hq, Hkv, d, S_max, _p(hd), n, _p(out),
                                int(n_threads))
    if rc != 0:
        raise ValueError("sparq_oracle_dense: bad argument")
    return out
