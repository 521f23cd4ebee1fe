"""CPU oracle for exact attention -- TEST INFRASTRUCTURE, not a product path.

Thin ctypes wrapper around ``oracle_attn.cpp`` (plain double-precision C++,
the definition of Section 2 steps 2-4 of the paper written out row by row).
Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the CUDA library never does, and this package never imports
the CUDA binding.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "oracle_attn.cpp")
_LIB = os.path.join(_HERE, "liboracle_attn.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (-O2, no fast-math) if missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-pthread", _SRC, "-o", tmp])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.oracle_attn_rows.restype = ctypes.c_int
        lib.oracle_attn_rows.argtypes = [
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int,
            ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, ctypes.c_float,
            ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_int64,
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.POINTER(ctypes.c_int)]
        lib.oracle_hardware_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def hardware_threads() -> int:
    return int(_load().oracle_hardware_threads())


def attention(Q, K, V, scale, valid_len=None, rows=None, want_logits=False, want_weights=False,
              nthreads: int = 0, causal: bool = False):
    """Exact attention in double precision.

    Q: [B,H,Nq,d], K/V: [B,H,Nk,d]; dtype uint16 (bf16 bit patterns) or float32.
    rows: optional int64 array of flat row ids ((b*H+h)*Nq + i); default all rows.
    causal: query i attends keys j <= i + (Nk - Nq) only (intersected with valid_len).
    Returns dict with 'O' ([B,H,Nq,d] or [nrows,d] float64), optionally 'L' and
    'A' ([..., Nk]), and 'threads' (threads used).
    """
    Q = np.ascontiguousarray(Q); K = np.ascontiguousarray(K); V = np.ascontiguousarray(V)
    if Q.dtype == np.uint16:
        dtype = 0
    elif Q.dtype == np.float32:
        dtype = 1
    else:
        raise TypeError("Q/K/V must be uint16 (bf16 bits) or float32")
    if K.dtype != Q.dtype or V.dtype != Q.dtype:
        raise TypeError("Q, K, V must share a dtype")
    B, H, Nq, d = Q.shape
    Nk = K.shape[2]
    if K.shape != (B, H, Nk, d) or V.shape != (B, H, Nk, d):
        raise ValueError("shape mismatch")
    vl = None
    if valid_len is not None:
        vl = np.ascontiguousarray(valid_len, dtype=np.int32)
        if vl.shape != (B,):
            raise ValueError("valid_len must have shape [B]")
    if rows is not None:
        rows = np.ascontiguousarray(rows, dtype=np.int64)
        n = rows.shape[0]
        oshape, lshape = (n, d), (n, Nk)
    else:
        n = B * H * Nq
        oshape, lshape = (B, H, Nq, d), (B, H, Nq, Nk)
    O = np.empty(oshape, dtype=np.float64)
    L = np.empty(lshape, dtype=np.float64) if want_logits else None
    A = np.empty(lshape, dtype=np.float64) if want_weights else None
    used = ctypes.c_int(0)
    ptr = lambda a: None if a is None else a.ctypes.data_as(ctypes.c_void_p)
    rc = _load().oracle_attn_rows(ptr(Q), ptr(K), ptr(V), dtype, B, H, Nq, Nk, d, float(np.float32(scale)),
                                  ptr(vl), 1 if causal else 0, ptr(rows), n, ptr(O), ptr(L), ptr(A), int(nthreads),
                                  ctypes.byref(used))
    if rc != 0:
        raise ValueError("oracle_attn_rows rejected its arguments (code %d)" % rc)
    out = {"O": O, "threads": used.value}
    if L is not None:
        out["L"] = L
    if A is not None:
        out["A"] = A
    return out
