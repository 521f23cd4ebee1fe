"""Seeded synthetic inputs for the attention workloads (numpy only).

This module is the one piece shared by the CPU oracle's tests and the CUDA
path's tests/bench: it produces bytes, and contains none of the attention
arithmetic.  Every element is a pure function of (seed, tensor id, element
index), so any slice can be regenerated independently and in any order.

Workload shapes follow the paper's problem statement (Section 2, steps 2-4:
Q, K, V of shape [B, H, N, d]) at BERT-base / BERT-large head sizes and the
long sequence lengths of its evaluation (Section 6.1: 512 ... 64K tokens).
Values are iid N(0,1) rounded to bf16, as the configuration list of this
build prescribes; the paper's own workloads are model shapes, not datasets.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np

DEFAULT_SEED = 20210706

TENSOR_Q, TENSOR_K, TENSOR_V, TENSOR_LEN, TENSOR_ROWS = 0, 1, 2, 3, 4

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)


def _splitmix64(x: np.ndarray) -> np.ndarray:
    """SplitMix64 finaliser applied element-wise to a uint64 array."""
    with np.errstate(over="ignore"):
        z = (x + np.uint64(0x9E3779B97F4A7C15)) & _M64
        z = ((z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)) & _M64
        z = ((z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)) & _M64
        return z ^ (z >> np.uint64(31))


def _key(seed: int, tensor: int) -> np.uint64:
    return np.uint64((seed ^ (tensor << 60)) & 0xFFFFFFFFFFFFFFFF)


def hash_u64(seed: int, tensor: int, index) -> np.ndarray:
    idx = np.asarray(index, dtype=np.uint64)
    return _splitmix64(idx ^ _key(seed, tensor))


def normal_f32(seed: int, tensor: int, start: int, count: int) -> np.ndarray:
    """`count` iid N(0,1) float32 values for element indices start..start+count-1.

    Box-Muller on two 24-bit uniforms cut from one 64-bit hash word.
    """
    out = np.empty(count, dtype=np.float32)
    chunk = 1 << 22
    two_pi = 2.0 * math.pi
    for lo in range(0, count, chunk):
        hi = min(count, lo + chunk)
        z = hash_u64(seed, tensor, np.arange(start + lo, start + hi, dtype=np.uint64))
        u1 = ((z >> np.uint64(40)).astype(np.float64) + 1.0) * (1.0 / 16777216.0)  # (0, 1]
        u2 = ((z >> np.uint64(16)) & np.uint64(0xFFFFFF)).astype(np.float64) * (1.0 / 16777216.0)
        out[lo:hi] = (np.sqrt(-2.0 * np.log(u1)) * np.cos(two_pi * u2)).astype(np.float32)
    return out


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float32 -> bfloat16, returned as uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass(frozen=True)
class Workload:
    """One attention problem: Q [B,H,Nq,d], K/V [B,H,Nk,d], optional key-padding mask."""
    name: str
    B: int
    H: int
    Nq: int
    Nk: int
    d: int
    masked: bool = False

    @property
    def scale(self) -> float:
        return float(np.float32(1.0 / math.sqrt(self.d)))

    @property
    def flops(self) -> int:
        # Two contractions (logit, attend), one multiply-add = 2 FLOP each.
        return 4 * self.B * self.H * self.Nq * self.Nk * self.d

    def qkvo_bytes(self, elem_bytes: int = 2) -> int:
        return elem_bytes * self.B * self.H * self.d * (2 * self.Nq + 2 * self.Nk)


# The five benchmark configurations, plus small cases the oracle finishes at once.
WORKLOADS = {
    "c1_bert_base_512": Workload("c1_bert_base_512", 1, 12, 512, 512, 64),
    "c2_bert_large_4k": Workload("c2_bert_large_4k", 16, 16, 4096, 4096, 64),
    "c3_16k": Workload("c3_16k", 4, 16, 16384, 16384, 64),
    "c4_64k_d128": Workload("c4_64k_d128", 1, 8, 65536, 65536, 128),
    "c5_cross_masked": Workload("c5_cross_masked", 8, 12, 1024, 16384, 64, masked=True),
    # reduced copies of c2 / c4 for profiler captures (same tile shapes, a few hundred MB at most)
    "p_4k_small": Workload("p_4k_small", 4, 16, 4096, 4096, 64),
    # half of c2: 2048 row slabs, enough for the persistent grid (14 items per CTA on 148 SMs)
    "p_4k_half": Workload("p_4k_half", 8, 16, 4096, 4096, 64),
    "p_16k_d128_small": Workload("p_16k_d128_small", 1, 4, 16384, 16384, 128),
}


def make_qkv_bf16(w: Workload, seed: int = DEFAULT_SEED):
    """Q, K, V as uint16 bf16 bit patterns, shapes [B,H,Nq,d] and [B,H,Nk,d]."""
    nq = w.B * w.H * w.Nq * w.d
    nk = w.B * w.H * w.Nk * w.d
    q = f32_to_bf16_bits(normal_f32(seed, TENSOR_Q, 0, nq)).reshape(w.B, w.H, w.Nq, w.d)
    k = f32_to_bf16_bits(normal_f32(seed, TENSOR_K, 0, nk)).reshape(w.B, w.H, w.Nk, w.d)
    v = f32_to_bf16_bits(normal_f32(seed, TENSOR_V, 0, nk)).reshape(w.B, w.H, w.Nk, w.d)
    return q, k, v


def make_valid_len(w: Workload, seed: int = DEFAULT_SEED) -> np.ndarray:
    """Per-batch number of valid keys, uniform integer in [Nk/2, Nk] (int32, shape [B])."""
    h = hash_u64(seed, TENSOR_LEN, np.arange(w.B, dtype=np.uint64))
    half = w.Nk // 2
    return (half + (h % np.uint64(w.Nk - half + 1)).astype(np.int64)).astype(np.int32)


def sample_rows(w: Workload, per_head: int, seed: int = DEFAULT_SEED) -> np.ndarray:
    """Flat row indices ((b*H + h)*Nq + i, int64, sorted, unique) to check at full size.

    Per (b,h): row 0, row Nq-1, rows around a few 128-row tile boundaries, and
    seeded random rows up to `per_head` in total.
    """
    out = []
    for bh in range(w.B * w.H):
        fixed = {0, w.Nq - 1}
        for t in (128, 256, w.Nq // 2, w.Nq - 128):
            for off in (-1, 0):
                r = t + off
                if 0 <= r < w.Nq:
                    fixed.add(r)
        rows = set(sorted(fixed)[:per_head])
        ctr = 0
        while len(rows) < min(per_head, w.Nq):
            h = hash_u64(seed, TENSOR_ROWS, np.arange(ctr, ctr + per_head, dtype=np.uint64) + np.uint64(bh << 32))
            for r in (h % np.uint64(w.Nq)).tolist():
                if len(rows) < per_head:
                    rows.add(int(r))
            ctr += per_head
        out.extend(bh * w.Nq + r for r in sorted(rows))
    return np.asarray(out, dtype=np.int64)


def make_planted_qkv_bf16(w: Workload, seed: int = DEFAULT_SEED, strength: float = 6.0):
    """Structured inputs that make a dropped, duplicated or mis-masked key tile visible.

    K rows are random unit-scale vectors; query i is `strength` times the K row
    of a planted key position p(i) that sweeps tile boundaries, so row i's
    softmax is sharply peaked on key p(i); V[j, t] encodes the key position j
    (a smooth ramp plus a per-column offset), so O[i] ~ V[p(i)].  Returns
    (Q, K, V, planted) with planted[b, i] the key index (same for all heads).
    """
    q, k, v = make_qkv_bf16(w, seed)
    kf = bf16_bits_to_f32(k)
    valid = make_valid_len(w, seed) if w.masked else np.full(w.B, w.Nk, dtype=np.int32)
    planted = np.empty((w.B, w.Nq), dtype=np.int64)
    anchors = [0, 1, 63, 64, 127, 128, 129, 255, 256, 383, 384, 511]
    for b in range(w.B):
        n = int(valid[b])
        cand = [a for a in anchors if a < n] + [n - 1 - a for a in (0, 1, 127, 128, 129) if n - 1 - a >= 0]
        h = hash_u64(seed, TENSOR_ROWS, np.arange(w.Nq, dtype=np.uint64) + np.uint64((b + 1) << 40))
        rnd = (h % np.uint64(n)).astype(np.int64)
        for i in range(w.Nq):
            planted[b, i] = cand[(i // 2) % len(cand)] if i % 2 == 0 else rnd[i]
    qf = np.empty((w.B, w.H, w.Nq, w.d), dtype=np.float32)
    for b in range(w.B):
        qf[b] = strength * kf[b][:, planted[b], :]
    j = np.arange(w.Nk, dtype=np.float32)[:, None]
    t = np.arange(w.d, dtype=np.float32)[None, :]
    vf = (j / np.float32(w.Nk)) * 4.0 - 2.0 + 0.03125 * t
    vfull = np.broadcast_to(vf.astype(np.float32), (w.B, w.H, w.Nk, w.d))
    return f32_to_bf16_bits(qf).reshape(q.shape), k, f32_to_bf16_bits(np.ascontiguousarray(vfull)).reshape(v.shape), planted
