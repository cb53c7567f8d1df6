"""ctypes loader for the plain-C fp64 attention oracle.  TEST INFRASTRUCTURE ONLY.

`build()` compiles oracle/attn_oracle.c with gcc (+OpenMP) into
oracle/_attn_oracle.so; `attention_rows()` calls it.  The mask predicate the C
code applies is the one of Sec. 3.2 / 3.3 / Appendix A, driven by the
per-token classes computed in hilberta_oracle.token_classes.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "attn_oracle.c")
_SO = os.path.join(_HERE, "_attn_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _SO, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _SO


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        f = lib.hilberta_oracle_attention_rows
        f.restype = ctypes.c_int
        f.argtypes = [ctypes.c_void_p] * 5 + [ctypes.c_int] * 3 + [ctypes.c_void_p] * 3 + [
            ctypes.c_int, ctypes.c_double]
        g = lib.hilberta_oracle_attention_backward
        g.restype = ctypes.c_int
        g.argtypes = [ctypes.c_void_p] * 7 + [ctypes.c_int] * 3 + [ctypes.c_void_p] * 3 + [
            ctypes.c_int, ctypes.c_void_p, ctypes.c_int, ctypes.c_double]
        _lib = lib
    return _lib


def attention_rows(q, k, v, is_global, group, rows=None, scale=None, return_lse=False,
                   return_threads=False):
    """fp64 masked attention for the listed query rows (all rows if None).

    q, k, v: float32 arrays [B, heads, S, D], original token order.
    Returns out [B, heads, n_rows, D] float64 (and lse [B, heads, n_rows]).
    """
    lib = _load()
    q = np.ascontiguousarray(q, dtype=np.float32)
    k = np.ascontiguousarray(k, dtype=np.float32)
    v = np.ascontiguousarray(v, dtype=np.float32)
    B, Hh, S, D = q.shape
    if rows is None:
        rows = np.arange(S, dtype=np.int32)
    rows = np.ascontiguousarray(rows, dtype=np.int32)
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    is_global = np.ascontiguousarray(is_global, dtype=np.uint8)
    group = np.ascontiguousarray(group, dtype=np.int32)
    out = np.empty((B, Hh, rows.size, D), dtype=np.float64)
    lse = np.empty((B, Hh, rows.size), dtype=np.float64)
    nthreads = lib.hilberta_oracle_attention_rows(
        q.ctypes.data, k.ctypes.data, v.ctypes.data, out.ctypes.data, lse.ctypes.data,
        B * Hh, S, D, is_global.ctypes.data, group.ctypes.data, rows.ctypes.data,
        int(rows.size), float(scale))
    if nthreads < 0:
        raise MemoryError("oracle scratch allocation failed")
    res = (out,)
    if return_lse:
        res += (lse,)
    if return_threads:
        res += (nthreads,)
    return res[0] if len(res) == 1 else res


def attention_backward(q, k, v, dout, is_global, group, rows=None, cols=None, scale=None):
    """fp64 gradients of sum(O * dout) for the listed query rows (dq) and key columns (dk, dv).

    q, k, v, dout: float32 arrays [B, heads, S, D], original token order; rows / cols
    default to all tokens.  Returns dq [B, heads, n_rows, D], dk and dv [B, heads, n_cols, D].
    """
    lib = _load()
    q = np.ascontiguousarray(q, dtype=np.float32)
    k = np.ascontiguousarray(k, dtype=np.float32)
    v = np.ascontiguousarray(v, dtype=np.float32)
    dout = np.ascontiguousarray(dout, dtype=np.float32)
    B, Hh, S, D = q.shape
    rows = np.arange(S, dtype=np.int32) if rows is None else np.ascontiguousarray(rows, dtype=np.int32)
    cols = np.arange(S, dtype=np.int32) if cols is None else np.ascontiguousarray(cols, dtype=np.int32)
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    is_global = np.ascontiguousarray(is_global, dtype=np.uint8)
    group = np.ascontiguousarray(group, dtype=np.int32)
    dq = np.empty((B, Hh, rows.size, D), dtype=np.float64)
    dk = np.empty((B, Hh, cols.size, D), dtype=np.float64)
    dv = np.empty((B, Hh, cols.size, D), dtype=np.float64)
    nthreads = lib.hilberta_oracle_attention_backward(
        q.ctypes.data, k.ctypes.data, v.ctypes.data, dout.ctypes.data, dq.ctypes.data, dk.ctypes.data,
        dv.ctypes.data, B * Hh, S, D, is_global.ctypes.data, group.ctypes.data, rows.ctypes.data,
        int(rows.size), cols.ctypes.data, int(cols.size), float(scale))
    if nthreads < 0:
        raise MemoryError("oracle scratch allocation failed")
    return dq, dk, dv
