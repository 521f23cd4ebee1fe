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
_SRCS = [os.path.join(_HERE, "oracle_attn.cpp"), os.path.join(_HERE, "oracle_attn_bwd.cpp")]
_LIB = os.path.join(_HERE, "liboracle_attn.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (-O2, no fast-math) if missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < max(os.path.getmtime(f) for f in _SRCS):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-pthread"] + _SRCS + ["-o", tmp])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.oracle_attn_rows_sparse.restype = ctypes.c_int
        lib.oracle_attn_rows_sparse.argtypes = [
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int,
            ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, ctypes.c_float,
            ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_int64,
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
            ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_int64,
            ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, ctypes.c_int,
            ctypes.POINTER(ctypes.c_int)]
        lib.oracle_attn_bwd_heads.restype = ctypes.c_int
        lib.oracle_attn_bwd_heads.argtypes = [
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int,
            ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, ctypes.c_float,
            ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_int64,
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int,
            ctypes.POINTER(ctypes.c_int)]
        lib.oracle_hardware_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def hardware_threads() -> int:
    return int(_load().oracle_hardware_threads())


def attention(Q, K, V, scale, valid_len=None, rows=None, want_logits=False, want_weights=False,
              nthreads: int = 0, causal: bool = False, want_lse=False, bias=None, block_mask=None, block: int = 128):
    """Exact attention in double precision.

    Q: [B,H,Nq,d], K/V: [B,H,Nk,d]; dtype uint16 (bf16 bit patterns) or float32.
    rows: optional int64 array of flat row ids ((b*H+h)*Nq + i); default all rows.
    causal: query i attends keys j <= i + (Nk - Nq) only (intersected with valid_len).
    Returns dict with 'O' ([B,H,Nq,d] or [nrows,d] float64), optionally 'L' and
    'A' ([..., Nk]), 'LSE' ([B,H,Nq] or [nrows]: log of the row's sum of exp(scaled logit) over its
    valid keys, -inf for a row without any), and 'threads' (threads used).
    bias: optional additive term of the scaled logits, [B or 1, H or 1, Nq, Nk], uint16 (bf16 bits) or
    float32; size-1 batch / head axes are repeated; -inf switches a (query, key) pair off.
    block_mask: optional uint8 map [B or 1, H or 1, ceil(Nq / block), ceil(Nk / block)] of the blocks of the
    logit matrix that are kept (non-zero) or pruned (0): pruned pairs take no part.
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
    LSE = np.empty(oshape[:-1], dtype=np.float64) if want_lse else None
    bias_dtype = bias_sb = bias_sh = 0
    if bias is not None:
        bias = np.ascontiguousarray(bias)
        if bias.dtype == np.uint16:
            bias_dtype = 0
        elif bias.dtype == np.float32:
            bias_dtype = 1
        else:
            raise TypeError("bias must be uint16 (bf16 bits) or float32")
        if bias.ndim != 4 or bias.shape[2:] != (Nq, Nk) or bias.shape[0] not in (1, B) or bias.shape[1] not in (1, H):
            raise ValueError("bias must be [B or 1, H or 1, Nq, Nk]")
        bias_sh = 0 if bias.shape[1] == 1 else Nq * Nk
        bias_sb = 0 if bias.shape[0] == 1 else bias.shape[1] * Nq * Nk
    bm_sb = bm_sh = 0
    if block_mask is not None:
        block_mask = np.ascontiguousarray(block_mask, dtype=np.uint8)
        tq, tk = -(-Nq // block), -(-Nk // block)
        if block_mask.ndim != 4 or block_mask.shape[2:] != (tq, tk) or block_mask.shape[0] not in (1, B) or block_mask.shape[1] not in (1, H):
            raise ValueError("block_mask must be [B or 1, H or 1, ceil(Nq/block), ceil(Nk/block)]")
        bm_sh = 0 if block_mask.shape[1] == 1 else tq * tk
        bm_sb = 0 if block_mask.shape[0] == 1 else block_mask.shape[1] * tq * tk
    used = ctypes.c_int(0)
    ptr = lambda a: None if a is None else a.ctypes.data_as(ctypes.c_void_p)
    rc = _load().oracle_attn_rows_sparse(ptr(Q), ptr(K), ptr(V), dtype, B, H, Nq, Nk, d, float(np.float32(scale)),
                                       ptr(vl), 1 if causal else 0, ptr(rows), n, ptr(O), ptr(L), ptr(A), ptr(LSE),
                                       ptr(bias), bias_dtype, bias_sb, bias_sh, ptr(block_mask), bm_sb, bm_sh, int(block),
                                       int(nthreads), ctypes.byref(used))
    if rc != 0:
        raise ValueError("oracle_attn_rows rejected its arguments (code %d)" % rc)
    out = {"O": O, "threads": used.value}
    if L is not None:
        out["L"] = L
    if A is not None:
        out["A"] = A
    if LSE is not None:
        out["LSE"] = LSE
    return out


def attention_bwd(Q, K, V, dO, scale, valid_len=None, causal: bool = False, heads=None, nthreads: int = 0):
    """Gradient of exact attention (the chain rule on Section 2's steps 2-4) in double precision.

    Q, dO: [B,H,Nq,d], K, V: [B,H,Nk,d]; uint16 (bf16 bit patterns) or float32, one dtype for all.
    heads: optional int64 array of flat head ids b*H + h to compute (each complete); default all.
    Returns dict: 'dQ' [B,H,Nq,d] (or [nheads,Nq,d]), 'dK', 'dV' [B,H,Nk,d] (or [nheads,Nk,d]),
    'LSE' [B,H,Nq] (or [nheads,Nq]), all float64, and 'threads'.
    """
    Q, K, V, dO = (np.ascontiguousarray(x) for x in (Q, K, V, dO))
    if Q.dtype == np.uint16:
        dtype = 0
    elif Q.dtype == np.float32:
        dtype = 1
    else:
        raise TypeError("Q/K/V/dO must be uint16 (bf16 bits) or float32")
    if any(x.dtype != Q.dtype for x in (K, V, dO)):
        raise TypeError("Q, K, V, dO must share a dtype")
    B, H, Nq, d = Q.shape
    Nk = K.shape[2]
    if K.shape != (B, H, Nk, d) or V.shape != (B, H, Nk, d) or dO.shape != Q.shape:
        raise ValueError("shape mismatch")
    vl = None
    if valid_len is not None:
        vl = np.ascontiguousarray(valid_len, dtype=np.int32)
        if vl.shape != (B,):
            raise ValueError("valid_len must have shape [B]")
    if heads is not None:
        heads = np.ascontiguousarray(heads, dtype=np.int64)
        lead = (heads.shape[0],)
    else:
        lead = (B, H)
    dQ = np.empty(lead + (Nq, d), dtype=np.float64)
    dK = np.empty(lead + (Nk, d), dtype=np.float64)
    dV = np.empty(lead + (Nk, d), dtype=np.float64)
    LSE = np.empty(lead + (Nq,), dtype=np.float64)
    used = ctypes.c_int(0)
    ptr = lambda a: None if a is None else a.ctypes.data_as(ctypes.c_void_p)
    rc = _load().oracle_attn_bwd_heads(ptr(Q), ptr(K), ptr(V), ptr(dO), dtype, B, H, Nq, Nk, d, float(np.float32(scale)),
                                       ptr(vl), 1 if causal else 0, ptr(heads), 0 if heads is None else heads.shape[0],
                                       ptr(dQ), ptr(dK), ptr(dV), ptr(LSE), int(nthreads), ctypes.byref(used))
    if rc != 0:
        raise ValueError("oracle_attn_bwd_heads rejected its arguments (code %d)" % rc)
    return {"dQ": dQ, "dK": dK, "dV": dV, "LSE": LSE, "threads": used.value}


# ------------------------------------------------------------------------------------------------
# The attention layer: Section 2, "Computation operators", steps 1-5 (Q/K/V projections, Logit,
# softmax, Attend, Output projection).  The paper states the operators, not a number format; the
# tensors between operators are stored as bf16 here (the storage type of the whole path), so the
# oracle rounds Q, K, V and O to bf16 where they are stored and does everything else in double.

def bf16_bits_to_f64(bits):
    """uint16 bf16 bit patterns -> float64 (exact)."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def round_to_bf16_bits(x):
    """float64 -> nearest bf16 (ties to even), returned as uint16 bit patterns.

    Goes through float32 first (also round-to-nearest-even); a value can land one bf16 step away
    from the directly rounded one only if it lies within 2^-29 (relative) of a bf16 tie.
    """
    b = np.ascontiguousarray(x, dtype=np.float64).astype(np.float32).view(np.uint32)
    return ((b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)).astype(np.uint16)


def qkv_projection(X, Wqkv, H, d):
    """Step 1: X [B,N,Dm], Wqkv [3*H*d, Dm] (uint16 bf16 bits; rows: Query, Key, Value features, head
    by head) -> Q, K, V [B,H,N,d] as float64, before any rounding:  Q[b,h,n,c] = sum_k X[b,n,k] W[h*d+c, k]."""
    B, N, Dm = X.shape
    if Wqkv.shape != (3 * H * d, Dm):
        raise ValueError("Wqkv must be [3*H*d, Dm]")
    x = bf16_bits_to_f64(X).reshape(B * N, Dm)
    w = bf16_bits_to_f64(Wqkv)
    y = x @ w.T                                                    # [B*N, 3*H*d], double
    y = y.reshape(B, N, 3, H, d).transpose(2, 0, 3, 1, 4)           # [3, B, H, N, d]
    return np.ascontiguousarray(y[0]), np.ascontiguousarray(y[1]), np.ascontiguousarray(y[2])


def out_projection(O, Wo):
    """Step 5: O [B,H,N,d] float64, Wo [Dm, H*d] bf16 bits -> Y [B,N,Dm] float64:
    Y[b,n,j] = sum_{h,c} O[b,h,n,c] Wo[j, h*d+c] (the heads are concatenated along the feature index)."""
    B, H, N, d = O.shape
    if Wo.shape[1] != H * d:
        raise ValueError("Wo must be [Dm, H*d]")
    o = np.ascontiguousarray(O.transpose(0, 2, 1, 3)).reshape(B * N, H * d)
    return (o @ bf16_bits_to_f64(Wo).T).reshape(B, N, Wo.shape[0])


def fully_connected(X, W):
    """A fully connected operator of the block (Section 2): X [..., K], W [Nout, K] bf16 bits ->
    Y [..., Nout] float64, Y[..., j] = sum_k X[..., k] W[j, k]; no bias, no activation."""
    x = bf16_bits_to_f64(X)
    return (x.reshape(-1, x.shape[-1]) @ bf16_bits_to_f64(W).T).reshape(x.shape[:-1] + (W.shape[0],))


def layer_norm(X, gamma, beta, eps, residual=None):
    """The block's normalisation layer (Section 2 names it without defining it; reading: layer
    normalisation over the features of each token, after the residual add, biased variance):
    z = X + residual, Y = gamma * (z - mean z) / sqrt(var z + eps) + beta.  X, residual [..., D] and
    gamma, beta [D] are uint16 bf16 bits; returns Y float64 (not rounded).  Written as plain loops over
    the rows so that it can be read against the formula."""
    x = bf16_bits_to_f64(X)
    if residual is not None:
        x = x + bf16_bits_to_f64(residual)
    g, b = bf16_bits_to_f64(gamma), bf16_bits_to_f64(beta)
    D = x.shape[-1]
    rows = x.reshape(-1, D)
    out = np.empty_like(rows)
    e = float(np.float32(eps))
    for i in range(rows.shape[0]):
        z = rows[i]
        mean = z.sum() / D
        var = ((z - mean) ** 2).sum() / D
        out[i] = g * (z - mean) / np.sqrt(var + e) + b
    return out.reshape(x.shape)


def attention_layer(X, Wqkv, Wo, H, d, scale, causal=False, nthreads: int = 0):
    """Steps 1-5 for self-attention.  Returns dict: 'Q','K','V','O' (uint16 bf16 bits, as stored
    between the operators) and 'Y' [B,N,Dm] float64 (not rounded)."""
    q, k, v = qkv_projection(X, Wqkv, H, d)
    Qb, Kb, Vb = round_to_bf16_bits(q), round_to_bf16_bits(k), round_to_bf16_bits(v)
    o = attention(Qb, Kb, Vb, scale, causal=causal, nthreads=nthreads)["O"]
    Ob = round_to_bf16_bits(o)
    return {"Q": Qb, "K": Kb, "V": Vb, "O": Ob, "Y": out_projection(bf16_bits_to_f64(Ob), Wo)}


def attention_varlen(Q, K, V, cu_seqlens_q, cu_seqlens_k, scale, causal=False, nthreads: int = 0):
    """Exact attention over a packed batch: Q [total_q, H, d], K, V [total_k, H, d] (uint16 bf16 bits
    or float32); sequence s owns query tokens cu_seqlens_q[s] .. cu_seqlens_q[s+1]-1 and key tokens
    cu_seqlens_k[s] .. cu_seqlens_k[s+1]-1.  Each sequence is the plain definition (steps 2-4 of
    Section 2) on its own tokens; a sequence without keys gives O = 0.  Returns O [total_q, H, d] float64."""
    cq = np.asarray(cu_seqlens_q, dtype=np.int64); ck = np.asarray(cu_seqlens_k, dtype=np.int64)
    total_q, H, d = Q.shape
    O = np.zeros((total_q, H, d), dtype=np.float64)
    for s in range(len(cq) - 1):
        q0, q1, k0, k1 = int(cq[s]), int(cq[s + 1]), int(ck[s]), int(ck[s + 1])
        if q1 <= q0 or k1 <= k0:
            continue
        q = np.ascontiguousarray(Q[q0:q1].transpose(1, 0, 2))[None]      # [1, H, nq, d]
        k = np.ascontiguousarray(K[k0:k1].transpose(1, 0, 2))[None]
        v = np.ascontiguousarray(V[k0:k1].transpose(1, 0, 2))[None]
        o = attention(q, k, v, scale, causal=causal, nthreads=nthreads)["O"][0]   # [H, nq, d]
        O[q0:q1] = o.transpose(1, 0, 2)
    return O
