"""ctypes binding of libflat_attn.so: argument marshalling only, same names as include/flat_attn.h.

Importing this module loads the CUDA library and raises if it is missing -- there is no
CPU fallback.  Tensor arguments are torch tensors (device memory and streams are all
PyTorch is used for); every computation happens inside the library's kernels.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libflat_attn.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        "libflat_attn.so is not built (run `python -m paper_2107_06419_b200.build` or "
        "`__graft_entry__.build()`); there is no fallback path")

_lib = ctypes.CDLL(LIB_PATH)

FLAT_OK = 0
FLAT_DTYPE_BF16, FLAT_DTYPE_F32 = 0, 1
FLAT_VARIANT_AUTO, FLAT_VARIANT_SIMT, FLAT_VARIANT_TC, FLAT_VARIANT_TC2, FLAT_VARIANT_TC2_SINGLE = 0, 1, 2, 3, 4
FLAT_VARIANT_TC3 = 5
FLAT_VARIANT_RGRAN = 6
FLAT_VARIANT_TF32 = 7
FLAT_VARIANT_TC2_SPLIT2, FLAT_VARIANT_TC2_SPLIT4, FLAT_VARIANT_TC2_SPLIT8 = 8, 9, 10
FLAT_VARIANT_TC2_HALVES, FLAT_VARIANT_TC2_HALVES_SPLIT2, FLAT_VARIANT_TC2_HALVES_SPLIT4, FLAT_VARIANT_TC2_HALVES_SPLIT8 = 11, 12, 13, 14
FLAT_VARIANT_TC2_SPLIT16, FLAT_VARIANT_TC2_HALVES_SPLIT16 = 15, 16

EXPORTS = ["flat_attn_fwd", "flat_attn_fwd_ex", "flat_attn_naive_fwd", "flat_attn_naive_fwd_ex",
           "flat_attn_naive_fwd_static", "flat_attn_selftest_wait_timeout", "flat_attn_selftest_exp2_poly",
           "flat_attn_fwd_host", "flat_attn_host_workspace_bytes", "flat_attn_last_launch_count",
           "flat_attn_status_string", "flat_attn_version",
           "flat_qkv_proj_fwd", "flat_out_proj_fwd", "flat_attn_layer_fwd", "flat_fc_fwd",
           "flat_attn_varlen_fwd", "flat_attn_last_variant", "flat_attn_last_device_error",
           "flat_attn_clear_device_error", "flat_attn_bwd", "flat_attn_bwd_ex", "flat_layernorm_fwd",
           "flat_attn_last_schedule"]
FLAT_SCHEDULE_ITEMS, FLAT_SCHEDULE_PERSISTENT, FLAT_SCHEDULE_EVEN_DEAL = 1, 2, 3


class flat_attn_params_t(ctypes.Structure):
    _fields_ = [("Q", ctypes.c_void_p), ("K", ctypes.c_void_p), ("V", ctypes.c_void_p), ("O", ctypes.c_void_p),
                ("B", ctypes.c_int), ("H", ctypes.c_int), ("Nq", ctypes.c_int), ("Nk", ctypes.c_int),
                ("d", ctypes.c_int), ("scale", ctypes.c_float), ("dtype", ctypes.c_int),
                ("k_valid_len", ctypes.c_void_p), ("status", ctypes.c_void_p), ("variant", ctypes.c_int),
                ("causal", ctypes.c_int), ("lse", ctypes.c_void_p), ("bias", ctypes.c_void_p),
                ("bias_dtype", ctypes.c_int), ("bias_stride_b", ctypes.c_longlong), ("bias_stride_h", ctypes.c_longlong),
                ("block_mask", ctypes.c_void_p), ("block_mask_stride_b", ctypes.c_longlong),
                ("block_mask_stride_h", ctypes.c_longlong)]


class flat_attn_bwd_params_t(ctypes.Structure):
    _fields_ = [("Q", ctypes.c_void_p), ("K", ctypes.c_void_p), ("V", ctypes.c_void_p), ("O", ctypes.c_void_p),
                ("dO", ctypes.c_void_p), ("lse", ctypes.c_void_p), ("dQ", ctypes.c_void_p), ("dK", ctypes.c_void_p),
                ("dV", ctypes.c_void_p), ("delta", ctypes.c_void_p),
                ("B", ctypes.c_int), ("H", ctypes.c_int), ("Nq", ctypes.c_int), ("Nk", ctypes.c_int),
                ("d", ctypes.c_int), ("scale", ctypes.c_float), ("k_valid_len", ctypes.c_void_p),
                ("status", ctypes.c_void_p), ("causal", ctypes.c_int)]


_vp, _i, _f = ctypes.c_void_p, ctypes.c_int, ctypes.c_float
_lib.flat_attn_bwd_ex.argtypes = [ctypes.POINTER(flat_attn_bwd_params_t), _vp]
_lib.flat_attn_bwd_ex.restype = _i
_lib.flat_attn_bwd.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _f, _vp]
_lib.flat_attn_bwd.restype = _i
_lib.flat_attn_fwd.argtypes = [_vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _f, _vp]
_lib.flat_attn_fwd.restype = _i
_lib.flat_attn_fwd_ex.argtypes = [ctypes.POINTER(flat_attn_params_t), _vp]
_lib.flat_attn_fwd_ex.restype = _i
_lib.flat_attn_naive_fwd.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _f, _vp]
_lib.flat_attn_naive_fwd.restype = _i
_lib.flat_attn_naive_fwd_ex.argtypes = [ctypes.POINTER(flat_attn_params_t), _vp, _vp, _vp]
_lib.flat_attn_naive_fwd_ex.restype = _i
_lib.flat_attn_naive_fwd_static.argtypes = [_vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _f, _vp]
_lib.flat_attn_naive_fwd_static.restype = _i
_lib.flat_attn_selftest_exp2_poly.argtypes = [_vp, _vp, _i, _vp]
_lib.flat_attn_selftest_exp2_poly.restype = _i
_lib.flat_attn_selftest_wait_timeout.argtypes = [_vp, _vp]
_lib.flat_attn_selftest_wait_timeout.restype = _i
_lib.flat_attn_fwd_host.argtypes = [ctypes.POINTER(flat_attn_params_t), _vp, ctypes.c_size_t, _vp]
_lib.flat_attn_fwd_host.restype = _i
_lib.flat_qkv_proj_fwd.argtypes = [_vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _vp, _vp]
_lib.flat_qkv_proj_fwd.restype = _i
_lib.flat_out_proj_fwd.argtypes = [_vp, _vp, _vp, _i, _i, _i, _i, _i, _vp, _vp]
_lib.flat_out_proj_fwd.restype = _i
_lib.flat_attn_layer_fwd.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _f, _i, _vp, _vp]
_lib.flat_attn_layer_fwd.restype = _i
_lib.flat_fc_fwd.argtypes = [_vp, _vp, _vp, _i, _i, _i, _vp, _vp]
_lib.flat_fc_fwd.restype = _i
_lib.flat_layernorm_fwd.argtypes = [_vp, _vp, _vp, _vp, _vp, ctypes.c_longlong, _i, _f, _vp]
_lib.flat_layernorm_fwd.restype = _i
_lib.flat_attn_varlen_fwd.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, ctypes.c_longlong, ctypes.c_longlong,
                                      _i, _f, _i, _vp, _vp]
_lib.flat_attn_varlen_fwd.restype = _i
_lib.flat_attn_host_workspace_bytes.argtypes = [_i, _i, _i, _i, _i, _i]
_lib.flat_attn_host_workspace_bytes.restype = ctypes.c_size_t
_lib.flat_attn_last_launch_count.restype = _i
_lib.flat_attn_last_variant.restype = _i
_lib.flat_attn_last_schedule.restype = _i
_lib.flat_attn_last_device_error.argtypes = [ctypes.POINTER(ctypes.c_int32)]
_lib.flat_attn_last_device_error.restype = _i
_lib.flat_attn_clear_device_error.restype = _i
_lib.flat_attn_status_string.argtypes = [_i]
_lib.flat_attn_status_string.restype = ctypes.c_char_p
_lib.flat_attn_version.restype = _i


class FlatAttnError(RuntimeError):
    def __init__(self, code: int):
        self.code = code
        super().__init__("flat_attn error %d: %s" % (code, flat_attn_status_string(code)))


def flat_attn_status_string(code: int) -> str:
    return _lib.flat_attn_status_string(int(code)).decode()


def flat_attn_version() -> int:
    return int(_lib.flat_attn_version())


def flat_attn_last_launch_count() -> int:
    return int(_lib.flat_attn_last_launch_count())


def flat_attn_last_variant() -> int:
    """The FLAT_VARIANT_* the most recent fused call on this thread ran (what AUTO resolved to)."""
    return int(_lib.flat_attn_last_variant())


def flat_attn_last_schedule() -> int:
    """FLAT_SCHEDULE_* of the most recent FLAT_VARIANT_TC3 launch on this thread (how its items went to the SMs)."""
    return int(_lib.flat_attn_last_schedule())


def flat_attn_last_device_error() -> int:
    """The library's sticky per-device give-up code (0 = none); synchronise your streams first."""
    code = ctypes.c_int32(0)
    _check(_lib.flat_attn_last_device_error(ctypes.byref(code)))
    return int(code.value)


def flat_attn_clear_device_error() -> None:
    _check(_lib.flat_attn_clear_device_error())


def _stream_ptr(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _dtype_code(t) -> int:
    if t.dtype == torch.bfloat16:
        return FLAT_DTYPE_BF16
    if t.dtype == torch.float32:
        return FLAT_DTYPE_F32
    raise TypeError("Q/K/V/O must be bfloat16 or float32")


def _params(Q, K, V, O, scale, k_valid_len, status, variant, host=False, causal=False, lse=None, bias=None,
            block_mask=None):
    B, H, Nq, d = Q.shape
    Nk = K.shape[2]
    if tuple(K.shape) != (B, H, Nk, d) or tuple(V.shape) != (B, H, Nk, d) or tuple(O.shape) != (B, H, Nq, d):
        raise ValueError("expected Q,O [B,H,Nq,d] and K,V [B,H,Nk,d]")
    for t in (Q, K, V, O):
        if not t.is_contiguous():
            raise ValueError("tensors must be contiguous")
        if t.dtype != Q.dtype:
            raise TypeError("Q, K, V, O must share a dtype")
        if t.is_cuda == host:
            raise ValueError("tensors must be %s tensors" % ("host" if host else "CUDA"))
    if k_valid_len is not None:
        if k_valid_len.dtype != torch.int32 or tuple(k_valid_len.shape) != (B,) or k_valid_len.is_cuda == host:
            raise ValueError("k_valid_len must be int32 [B] on the same side as Q")
    p = flat_attn_params_t()
    p.Q, p.K, p.V, p.O = Q.data_ptr(), K.data_ptr(), V.data_ptr(), O.data_ptr()
    p.B, p.H, p.Nq, p.Nk, p.d = B, H, Nq, Nk, d
    p.scale = float(scale)
    p.dtype = _dtype_code(Q)
    p.k_valid_len = None if k_valid_len is None else k_valid_len.data_ptr()
    p.status = None if status is None else status.data_ptr()
    p.variant = int(variant)
    p.causal = 1 if causal else 0
    if lse is not None:
        if lse.dtype != torch.float32 or tuple(lse.shape) != (B, H, Nq) or not lse.is_cuda or not lse.is_contiguous():
            raise ValueError("lse must be a contiguous CUDA float32 tensor [B,H,Nq]")
        p.lse = lse.data_ptr()
    else:
        p.lse = None
    if bias is not None:
        if (bias.dim() != 4 or tuple(bias.shape[2:]) != (Nq, Nk) or bias.shape[0] not in (1, B) or bias.shape[1] not in (1, H)
                or not bias.is_cuda or not bias.is_contiguous() or bias.dtype not in (torch.bfloat16, torch.float32)):
            raise ValueError("bias must be a contiguous CUDA bfloat16 / float32 tensor [B or 1, H or 1, Nq, Nk]")
        p.bias = bias.data_ptr()
        p.bias_dtype = _dtype_code(bias)
        p.bias_stride_h = 0 if bias.shape[1] == 1 else Nq * Nk
        p.bias_stride_b = 0 if bias.shape[0] == 1 else bias.shape[1] * Nq * Nk
    else:
        p.bias = None
    if block_mask is not None:
        tq, tk = -(-Nq // 128), -(-Nk // 128)
        if (block_mask.dim() != 4 or tuple(block_mask.shape[2:]) != (tq, tk) or block_mask.shape[0] not in (1, B)
                or block_mask.shape[1] not in (1, H) or not block_mask.is_cuda or not block_mask.is_contiguous()
                or block_mask.dtype != torch.uint8):
            raise ValueError("block_mask must be a contiguous CUDA uint8 tensor [B or 1, H or 1, ceil(Nq/128), ceil(Nk/128)]")
        p.block_mask = block_mask.data_ptr()
        p.block_mask_stride_h = 0 if block_mask.shape[1] == 1 else tq * tk
        p.block_mask_stride_b = 0 if block_mask.shape[0] == 1 else block_mask.shape[1] * tq * tk
    else:
        p.block_mask = None
    return p


def _check(rc: int):
    if rc != FLAT_OK:
        raise FlatAttnError(rc)


def flat_attn_fwd(Q, K, V, O, scale, stream=None):
    """Fused attention, bf16 CUDA tensors Q,O [B,H,Nq,d] and K,V [B,H,Nk,d]; writes O in place."""
    p = _params(Q, K, V, O, scale, None, None, FLAT_VARIANT_AUTO)
    if p.dtype != FLAT_DTYPE_BF16:
        raise TypeError("flat_attn_fwd takes bfloat16 tensors; use flat_attn_fwd_ex for float32")
    _check(_lib.flat_attn_fwd(p.Q, p.K, p.V, p.O, p.B, p.H, p.Nq, p.Nk, p.d, p.scale, _stream_ptr(stream)))
    return O


def flat_attn_fwd_ex(Q, K, V, O, scale, k_valid_len=None, status=None, variant=FLAT_VARIANT_AUTO, stream=None,
                     causal=False, lse=None, bias=None, block_mask=None):
    """Fused attention with dtype choice (from the tensors), key-padding mask, kernel choice and
    causal mask (query i sees keys j <= i + (Nk - Nq)); `lse` [B,H,Nq] float32 receives each row's
    log-sum-exp of the scaled logits (what the backward pass needs); `bias` [B or 1, H or 1, Nq, Nk]
    (bfloat16 or float32) is added to the scaled logits before the softmax (-inf switches a pair off);
    `block_mask` (uint8 [B or 1, H or 1, ceil(Nq/128), ceil(Nk/128)]) prunes 128 x 128 blocks of the logit
    matrix (0 = the block takes no part)."""
    p = _params(Q, K, V, O, scale, k_valid_len, status, variant, causal=causal, lse=lse, bias=bias,
                block_mask=block_mask)
    _check(_lib.flat_attn_fwd_ex(ctypes.byref(p), _stream_ptr(stream)))
    return O


def _bwd_params(Q, K, V, O, dO, lse, dQ, dK, dV, delta, scale, k_valid_len, status, causal):
    B, H, Nq, d = Q.shape
    Nk = K.shape[2]
    for name, t, shape in (("Q", Q, (B, H, Nq, d)), ("O", O, (B, H, Nq, d)), ("dO", dO, (B, H, Nq, d)),
                           ("dQ", dQ, (B, H, Nq, d)), ("K", K, (B, H, Nk, d)), ("V", V, (B, H, Nk, d)),
                           ("dK", dK, (B, H, Nk, d)), ("dV", dV, (B, H, Nk, d))):
        _bf16_cuda(name, t, shape)
    for name, t in (("lse", lse), ("delta", delta)):
        if t.dtype != torch.float32 or tuple(t.shape) != (B, H, Nq) or not t.is_cuda or not t.is_contiguous():
            raise ValueError(name + " must be a contiguous CUDA float32 tensor [B,H,Nq]")
    if k_valid_len is not None and (k_valid_len.dtype != torch.int32 or tuple(k_valid_len.shape) != (B,)
                                    or not k_valid_len.is_cuda):
        raise ValueError("k_valid_len must be a CUDA int32 tensor [B]")
    p = flat_attn_bwd_params_t()
    p.Q, p.K, p.V, p.O, p.dO = Q.data_ptr(), K.data_ptr(), V.data_ptr(), O.data_ptr(), dO.data_ptr()
    p.lse, p.dQ, p.dK, p.dV, p.delta = lse.data_ptr(), dQ.data_ptr(), dK.data_ptr(), dV.data_ptr(), delta.data_ptr()
    p.B, p.H, p.Nq, p.Nk, p.d = B, H, Nq, Nk, d
    p.scale = float(scale)
    p.k_valid_len = None if k_valid_len is None else k_valid_len.data_ptr()
    p.status = None if status is None else status.data_ptr()
    p.causal = 1 if causal else 0
    return p


def flat_attn_bwd_ex(Q, K, V, O, dO, lse, dQ, dK, dV, delta, scale, k_valid_len=None, status=None, causal=False,
                     stream=None):
    """Backward pass: writes dQ [B,H,Nq,d], dK, dV [B,H,Nk,d] (bf16 CUDA tensors) from Q, K, V, the
    forward's O and lse [B,H,Nq] (float32), and dO; `delta` [B,H,Nq] float32 is scratch."""
    p = _bwd_params(Q, K, V, O, dO, lse, dQ, dK, dV, delta, scale, k_valid_len, status, causal)
    _check(_lib.flat_attn_bwd_ex(ctypes.byref(p), _stream_ptr(stream)))
    return dQ, dK, dV


def flat_attn_bwd(Q, K, V, O, dO, lse, dQ, dK, dV, delta, scale, stream=None):
    """flat_attn_bwd_ex without masks and without a status word."""
    p = _bwd_params(Q, K, V, O, dO, lse, dQ, dK, dV, delta, scale, None, None, False)
    _check(_lib.flat_attn_bwd(p.Q, p.K, p.V, p.O, p.dO, p.lse, p.dQ, p.dK, p.dV, p.delta, p.B, p.H, p.Nq, p.Nk, p.d,
                              p.scale, _stream_ptr(stream)))
    return dQ, dK, dV


def flat_attn_naive_fwd(Q, K, V, O, L, A, scale, stream=None):
    """The unfused baseline: L (fp32) and A (bf16) [B,H,Nq,Nk] are caller-allocated CUDA tensors."""
    p = _params(Q, K, V, O, scale, None, None, FLAT_VARIANT_AUTO)
    _check_la(p, L, A)
    _check(_lib.flat_attn_naive_fwd(p.Q, p.K, p.V, p.O, _ptr(L), _ptr(A), p.B, p.H, p.Nq, p.Nk, p.d, p.scale,
                                    _stream_ptr(stream)))
    return O


def flat_attn_naive_fwd_ex(Q, K, V, O, L, A, scale, k_valid_len=None, stream=None, causal=False):
    p = _params(Q, K, V, O, scale, k_valid_len, None, FLAT_VARIANT_AUTO, causal=causal)
    _check_la(p, L, A)
    _check(_lib.flat_attn_naive_fwd_ex(ctypes.byref(p), _ptr(L), _ptr(A), _stream_ptr(stream)))
    return O


FLAT_STATIC_MAX_ELEMS = 4 * 1024 * 1024


def flat_attn_naive_fwd_static(Q, K, V, O, scale, stream=None):
    """The unfused baseline without caller-provided L and A: for callers that may not allocate
    device memory, the two [B,H,Nq,Nk] intermediates live in a 24 MiB array inside the library.
    bf16 CUDA tensors; B*H*Nq*Nk must not exceed FLAT_STATIC_MAX_ELEMS (error 5 otherwise).
    Calls on one device share that array: do not let two of them overlap on the GPU."""
    p = _params(Q, K, V, O, scale, None, None, FLAT_VARIANT_AUTO)
    if p.dtype != FLAT_DTYPE_BF16:
        raise TypeError("flat_attn_naive_fwd_static takes bfloat16 tensors")
    _check(_lib.flat_attn_naive_fwd_static(p.Q, p.K, p.V, p.O, p.B, p.H, p.Nq, p.Nk, p.d, p.scale,
                                           _stream_ptr(stream)))
    return O


FLAT_SELFTEST_TIMEOUT_CODE = 0x7E57


def flat_attn_selftest_exp2_poly(x, y, stream=None):
    """y = the kernel's polynomial 2^x of the CUDA float32 tensor x (same shape, contiguous)."""
    if not (x.is_cuda and y.is_cuda and x.dtype == torch.float32 and y.dtype == torch.float32):
        raise ValueError("x and y must be CUDA float32 tensors")
    if x.numel() != y.numel() or not x.is_contiguous() or not y.is_contiguous():
        raise ValueError("x and y must be contiguous and of equal size")
    _check(_lib.flat_attn_selftest_exp2_poly(_ptr(x), _ptr(y), x.numel(), _stream_ptr(stream)))
    return y


def flat_attn_selftest_wait_timeout(status, stream=None):
    """Runs the bounded-wait self-test; `status` is a zeroed CUDA int32 tensor of one element, or None."""
    if status is not None and (not status.is_cuda or status.dtype != torch.int32):
        raise ValueError("status must be a CUDA int32 tensor (or None: the library's own word)")
    _check(_lib.flat_attn_selftest_wait_timeout(_ptr(status), _stream_ptr(stream)))


def _bf16_cuda(name, t, shape):
    if t.dtype != torch.bfloat16 or not t.is_cuda or not t.is_contiguous() or tuple(t.shape) != tuple(shape):
        raise ValueError("%s must be a contiguous CUDA bfloat16 tensor of shape %s" % (name, tuple(shape)))


def flat_qkv_proj_fwd(X, Wqkv, Q, K, V, status=None, stream=None):
    """Q/K/V projection: X [B,N,Dm], Wqkv [3*H*d, Dm] (Query, Key, Value rows, head by head) -> Q, K, V [B,H,N,d]."""
    B, H, N, d = Q.shape
    Dm = X.shape[2]
    _bf16_cuda("X", X, (B, N, Dm)); _bf16_cuda("Wqkv", Wqkv, (3 * H * d, Dm))
    for name, t in (("Q", Q), ("K", K), ("V", V)):
        _bf16_cuda(name, t, (B, H, N, d))
    _check(_lib.flat_qkv_proj_fwd(_ptr(X), _ptr(Wqkv), _ptr(Q), _ptr(K), _ptr(V), B, N, H, d, Dm, _ptr(status),
                                  _stream_ptr(stream)))
    return Q, K, V


def flat_out_proj_fwd(O, Wo, Y, status=None, stream=None):
    """Output projection: O [B,H,N,d], Wo [Dm, H*d] -> Y [B,N,Dm]."""
    B, H, N, d = O.shape
    Dm = Y.shape[2]
    _bf16_cuda("O", O, (B, H, N, d)); _bf16_cuda("Wo", Wo, (Dm, H * d)); _bf16_cuda("Y", Y, (B, N, Dm))
    _check(_lib.flat_out_proj_fwd(_ptr(O), _ptr(Wo), _ptr(Y), B, N, H, d, Dm, _ptr(status), _stream_ptr(stream)))
    return Y


def flat_attn_layer_fwd(X, Wqkv, Wo, Y, Q, K, V, O, scale, causal=False, status=None, stream=None):
    """A self-attention layer: Q/K/V projection, fused attention, Output projection.  Q, K, V, O
    [B,H,N,d] are caller-owned buffers for the intermediates."""
    B, H, N, d = Q.shape
    Dm = X.shape[2]
    _bf16_cuda("X", X, (B, N, Dm)); _bf16_cuda("Wqkv", Wqkv, (3 * H * d, Dm)); _bf16_cuda("Wo", Wo, (Dm, H * d))
    _bf16_cuda("Y", Y, (B, N, Dm))
    for name, t in (("Q", Q), ("K", K), ("V", V), ("O", O)):
        _bf16_cuda(name, t, (B, H, N, d))
    _check(_lib.flat_attn_layer_fwd(_ptr(X), _ptr(Wqkv), _ptr(Wo), _ptr(Y), _ptr(Q), _ptr(K), _ptr(V), _ptr(O),
                                    B, N, H, d, Dm, float(scale), 1 if causal else 0, _ptr(status),
                                    _stream_ptr(stream)))
    return Y


def flat_fc_fwd(X, W, Y, status=None, stream=None):
    """Fully connected operator: X [..., K], W [Nout, K] -> Y [..., Nout] (bf16, no bias)."""
    K, Nout = X.shape[-1], W.shape[0]
    M = X.numel() // K
    _bf16_cuda("X", X, X.shape); _bf16_cuda("W", W, (Nout, K)); _bf16_cuda("Y", Y, tuple(X.shape[:-1]) + (Nout,))
    _check(_lib.flat_fc_fwd(_ptr(X), _ptr(W), _ptr(Y), M, K, Nout, _ptr(status), _stream_ptr(stream)))
    return Y


def flat_layernorm_fwd(X, gamma, beta, Y, eps=1e-5, residual=None, stream=None):
    """Y = gamma * layer_norm(X + residual) + beta over the last axis (bf16 CUDA tensors; gamma, beta [D])."""
    D = X.shape[-1]
    M = X.numel() // D
    _bf16_cuda("X", X, X.shape); _bf16_cuda("Y", Y, X.shape); _bf16_cuda("gamma", gamma, (D,)); _bf16_cuda("beta", beta, (D,))
    if residual is not None:
        _bf16_cuda("residual", residual, X.shape)
    _check(_lib.flat_layernorm_fwd(_ptr(X), _ptr(residual), _ptr(gamma), _ptr(beta), _ptr(Y), M, D, float(eps),
                                   _stream_ptr(stream)))
    return Y


def flat_attn_varlen_fwd(Q, K, V, O, cu_seqlens_q, cu_seqlens_k, max_seqlen_q, scale, causal=False, status=None,
                         stream=None):
    """Fused attention over a packed batch: Q, O [total_q, H, d], K, V [total_k, H, d] (bf16 CUDA);
    cu_seqlens_q / _k int32 CUDA tensors of num_seqs + 1 offsets."""
    total_q, H, d = Q.shape
    total_k = K.shape[0]
    _bf16_cuda("Q", Q, (total_q, H, d)); _bf16_cuda("O", O, (total_q, H, d))
    _bf16_cuda("K", K, (total_k, H, d)); _bf16_cuda("V", V, (total_k, H, d))
    for name, t in (("cu_seqlens_q", cu_seqlens_q), ("cu_seqlens_k", cu_seqlens_k)):
        if t.dtype != torch.int32 or not t.is_cuda or t.dim() != 1 or not t.is_contiguous():
            raise ValueError(name + " must be a contiguous int32 CUDA vector")
    if cu_seqlens_q.numel() != cu_seqlens_k.numel() or cu_seqlens_q.numel() < 2:
        raise ValueError("cu_seqlens_q and cu_seqlens_k must have num_seqs + 1 entries each")
    _check(_lib.flat_attn_varlen_fwd(_ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(cu_seqlens_q), _ptr(cu_seqlens_k),
                                     cu_seqlens_q.numel() - 1, H, d, total_q, total_k, int(max_seqlen_q), float(scale),
                                     1 if causal else 0, _ptr(status), _stream_ptr(stream)))
    return O


def _check_la(p, L, A):
    shape = (p.B, p.H, p.Nq, p.Nk)
    if tuple(L.shape) != shape or tuple(A.shape) != shape or not L.is_contiguous() or not A.is_contiguous():
        raise ValueError("L and A must be contiguous [B,H,Nq,Nk]")
    if L.dtype != torch.float32:
        raise TypeError("L must be float32")
    want = torch.bfloat16 if p.dtype == FLAT_DTYPE_BF16 else torch.float32
    if A.dtype != want:
        raise TypeError("A must have the dtype of Q")
    if not (L.is_cuda and A.is_cuda):
        raise ValueError("L and A must be CUDA tensors")


def flat_attn_host_workspace_bytes(B, H, Nq, Nk, d, dtype=FLAT_DTYPE_BF16) -> int:
    return int(_lib.flat_attn_host_workspace_bytes(B, H, Nq, Nk, d, dtype))


def flat_attn_fwd_host(Q, K, V, O, scale, workspace, k_valid_len=None, status=None,
                       variant=FLAT_VARIANT_AUTO, stream=None, causal=False):
    """Q, K, V, O (and k_valid_len) are HOST tensors (pinned for asynchrony); `workspace` is a CUDA
    uint8 tensor of at least flat_attn_host_workspace_bytes(...) bytes.  Asynchronous on `stream`."""
    p = _params(Q, K, V, O, scale, k_valid_len, status, variant, host=True, causal=causal)
    if not workspace.is_cuda:
        raise ValueError("workspace must be a CUDA tensor")
    _check(_lib.flat_attn_fwd_host(ctypes.byref(p), _ptr(workspace), workspace.numel() * workspace.element_size(),
                                   _stream_ptr(stream)))
    return O
