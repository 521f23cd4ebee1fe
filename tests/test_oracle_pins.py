"""Pins for the CPU oracle: what the paper and the mathematics fix, independent of the oracle.

Each test would fail under a plausible mistake in oracle_attn.cpp (a dropped
term, a wrong sign or index, a transposed operand, a mask off by one).
"""
import math
import os

import numpy as np
import pytest

import oracle
from paper_2107_06419_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rand_bf16(rng, shape, sigma=1.0):
    return inputs.f32_to_bf16_bits((rng.standard_normal(shape) * sigma).astype(np.float32)).reshape(shape)


def f32(bits):
    return inputs.bf16_bits_to_f32(bits).reshape(bits.shape)


def brute_force(Q, K, V, scale, valid_len=None):
    """Independent second implementation: long double, explicit full weight matrix,
    no max subtraction, key-outer loop order, pure numpy/Python."""
    ld = np.longdouble
    Q = Q.astype(ld); K = K.astype(ld); V = V.astype(ld)
    B, H, Nq, d = Q.shape
    Nk = K.shape[2]
    O = np.zeros((B, H, Nq, d), dtype=ld)
    A = np.zeros((B, H, Nq, Nk), dtype=ld)
    sc = ld(np.float32(scale))
    for b in range(B):
        n = Nk if valid_len is None else int(valid_len[b])
        for h in range(H):
            W = np.zeros((Nq, Nk), dtype=ld)
            for j in range(n):                      # key-outer order
                for i in range(Nq):
                    acc = ld(0)
                    for t in reversed(range(d)):    # reversed contraction order
                        acc += K[b, h, j, t] * Q[b, h, i, t]
                    W[i, j] = np.exp(sc * acc)      # no max subtraction
            den = W.sum(axis=1)
            for i in range(Nq):
                if n > 0:
                    A[b, h, i] = W[i] / den[i]
            O[b, h] = A[b, h] @ V[b, h]
    return O, A


# P1 -- closed-form worked example (hand-computed; the paper prints no numeric example).
def test_closed_form_example():
    # d = 1, q = 1, keys 0, ln2, ln3 -> exp(logits) = 1, 2, 3 -> weights 1/6, 2/6, 3/6.
    Q = np.array([1.0], dtype=np.float32).reshape(1, 1, 1, 1)
    K = np.array([0.0, math.log(2.0), math.log(3.0)], dtype=np.float32).reshape(1, 1, 3, 1)
    V = np.array([6.0, 12.0, 18.0], dtype=np.float32).reshape(1, 1, 3, 1)
    r = oracle.attention(Q, K, V, 1.0, want_weights=True, want_logits=True)
    kd = K.astype(np.float64).ravel()           # the stored float32 keys, widened
    w = np.exp(kd) / np.exp(kd).sum()
    assert np.allclose(r["A"].ravel(), w, rtol=0, atol=1e-15)
    assert abs(r["O"].item() - float(w @ np.array([6.0, 12.0, 18.0]))) < 1e-14
    assert abs(r["O"].item() - 14.0) < 1e-6     # float32 rounding of ln2, ln3 only
    assert np.allclose(r["L"].ravel(), kd, atol=1e-16)
    # scale enters before the softmax: scale = 2 squares the un-normalised weights.
    r2 = oracle.attention(Q, K, V, 2.0, want_weights=True)
    w2 = np.exp(2 * kd) / np.exp(2 * kd).sum()
    assert np.allclose(r2["A"].ravel(), w2, atol=1e-15)


# Two-key example where the transposition Q<->K or a swapped V index would show.
def test_two_by_two_hand_example():
    # d = 2. q0 = (1,0), q1 = (0,2). k0 = (ln2, 0), k1 = (0, ln3/2... ) chosen so logits are logs.
    Q = np.array([[1.0, 0.0], [0.0, 2.0]], dtype=np.float32).reshape(1, 1, 2, 2)
    K = np.array([[math.log(2.0), 0.0], [0.0, math.log(3.0) / 2]], dtype=np.float32).reshape(1, 1, 2, 2)
    V = np.array([[1.0, 10.0], [100.0, 1000.0]], dtype=np.float32).reshape(1, 1, 2, 2)
    r = oracle.attention(Q, K, V, 1.0, want_weights=True)
    # row 0 logits: (ln2, 0) -> weights 2/3, 1/3 ; row 1 logits: (0, ln3) -> 1/4, 3/4
    A = r["A"].reshape(2, 2)
    assert np.allclose(A, [[2 / 3, 1 / 3], [1 / 4, 3 / 4]], atol=1e-7)
    O = r["O"].reshape(2, 2)
    assert np.allclose(O, [[2 / 3 + 100 / 3, 20 / 3 + 1000 / 3], [0.25 + 75, 2.5 + 750]], rtol=1e-6)


# P2 -- every softmax row sums to 1, entries in (0, 1].
@pytest.mark.parametrize("shape", [(1, 1, 3, 5, 4), (2, 2, 17, 129, 8), (1, 2, 5, 300, 64)])
def test_rows_sum_to_one(shape):
    B, H, Nq, Nk, d = shape
    rng = np.random.default_rng(1)
    Q, K, V = rand_bf16(rng, (B, H, Nq, d)), rand_bf16(rng, (B, H, Nk, d)), rand_bf16(rng, (B, H, Nk, d))
    A = oracle.attention(Q, K, V, 1 / math.sqrt(d), want_weights=True)["A"]
    assert np.all(np.abs(A.sum(-1) - 1.0) < 1e-15 * Nk + 1e-14)
    assert np.all(A > 0) and np.all(A <= 1)


# P3 -- Q = 0 gives the column mean of V over the valid keys.
def test_zero_query_gives_mean_of_v():
    rng = np.random.default_rng(2)
    B, H, Nq, Nk, d = 2, 2, 4, 37, 8
    Q = np.zeros((B, H, Nq, d), dtype=np.uint16)
    K, V = rand_bf16(rng, (B, H, Nk, d)), rand_bf16(rng, (B, H, Nk, d))
    O = oracle.attention(Q, K, V, 0.7)["O"]
    mean = f32(V).astype(np.float64).mean(axis=2, keepdims=True)
    assert np.allclose(O, np.broadcast_to(mean, O.shape), atol=1e-14)
    vl = np.array([11, 37], dtype=np.int32)
    Om = oracle.attention(Q, K, V, 0.7, valid_len=vl)["O"]
    for b in range(B):
        mean_b = f32(V)[b, :, :vl[b]].astype(np.float64).mean(axis=1, keepdims=True)
        assert np.allclose(Om[b], np.broadcast_to(mean_b, Om[b].shape), atol=1e-14)


# P4 -- identical K rows give uniform weights.
def test_identical_keys_uniform_weights():
    rng = np.random.default_rng(3)
    B, H, Nq, Nk, d = 1, 2, 5, 19, 16
    Q, V = rand_bf16(rng, (B, H, Nq, d)), rand_bf16(rng, (B, H, Nk, d))
    K = np.broadcast_to(rand_bf16(rng, (B, H, 1, d)), (B, H, Nk, d)).copy()
    r = oracle.attention(Q, K, V, 0.25, want_weights=True)
    assert np.allclose(r["A"], 1.0 / Nk, atol=1e-16)
    assert np.allclose(r["O"], np.broadcast_to(f32(V).astype(np.float64).mean(2, keepdims=True), r["O"].shape), atol=1e-14)


# P5 -- permuting keys together with their V rows leaves O unchanged.
def test_key_permutation_invariance():
    rng = np.random.default_rng(4)
    B, H, Nq, Nk, d = 2, 1, 6, 50, 8
    Q, K, V = rand_bf16(rng, (B, H, Nq, d)), rand_bf16(rng, (B, H, Nk, d)), rand_bf16(rng, (B, H, Nk, d))
    perm = rng.permutation(Nk)
    O1 = oracle.attention(Q, K, V, 0.35)["O"]
    O2 = oracle.attention(Q, K[:, :, perm], V[:, :, perm], 0.35)["O"]
    assert np.max(np.abs(O1 - O2)) < 1e-13
    # permuting only K (not V) must change the result: catches a V index that ignores j.
    O3 = oracle.attention(Q, K[:, :, perm], V, 0.35)["O"]
    assert np.max(np.abs(O1 - O3)) > 1e-3


# P6 -- adding one vector u to every key adds a per-row constant to the logits: O unchanged.
def test_key_shift_invariance():
    rng = np.random.default_rng(5)
    B, H, Nq, Nk, d = 1, 2, 7, 33, 4
    Q = rng.integers(-4, 5, (B, H, Nq, d)).astype(np.float32)
    K = rng.integers(-4, 5, (B, H, Nk, d)).astype(np.float32)
    V = rng.standard_normal((B, H, Nk, d)).astype(np.float32)
    u = rng.integers(-3, 4, (1, 1, 1, d)).astype(np.float32)
    O1 = oracle.attention(Q, K, V, 0.125)["O"]
    O2 = oracle.attention(Q, K + u, V, 0.125)["O"]       # integer data: K + u exact in float32
    assert np.max(np.abs(O1 - O2)) < 1e-13


# P7 -- constant V returns that constant; O is linear in V.
def test_constant_v_and_linearity():
    rng = np.random.default_rng(6)
    B, H, Nq, Nk, d = 1, 1, 9, 41, 8
    Q, K = rand_bf16(rng, (B, H, Nq, d)), rand_bf16(rng, (B, H, Nk, d))
    c = rng.standard_normal(d).astype(np.float32)
    Vc = np.broadcast_to(c, (B, H, Nk, d)).copy()
    Oc = oracle.attention(f32(Q), f32(K), Vc, 0.3)["O"]
    assert np.allclose(Oc, np.broadcast_to(c.astype(np.float64), Oc.shape), atol=1e-15)
    V1 = rng.integers(-8, 9, (B, H, Nk, d)).astype(np.float32)
    V2 = rng.integers(-8, 9, (B, H, Nk, d)).astype(np.float32)
    O1 = oracle.attention(f32(Q), f32(K), V1, 0.3)["O"]
    O2 = oracle.attention(f32(Q), f32(K), V2, 0.3)["O"]
    O12 = oracle.attention(f32(Q), f32(K), V1 + V2, 0.3)["O"]
    assert np.max(np.abs(O12 - O1 - O2)) < 1e-13


# P8 -- one-hot limit: a huge scale with a unique maximum selects V[argmax]; no overflow/NaN.
def test_one_hot_limit_large_logits():
    rng = np.random.default_rng(7)
    B, H, Nq, Nk, d = 1, 1, 8, 64, 4
    Q = rng.integers(1, 5, (B, H, Nq, d)).astype(np.float32)
    K = rng.standard_normal((B, H, Nk, d)).astype(np.float32)
    V = rng.standard_normal((B, H, Nk, d)).astype(np.float32)
    r = oracle.attention(Q, K, V, 5000.0, want_logits=True)
    assert np.all(np.isfinite(r["O"]))
    arg = np.argmax(r["L"].reshape(Nq, Nk), axis=1)
    assert np.allclose(r["O"].reshape(Nq, d), V[0, 0, arg].astype(np.float64), atol=1e-12)


# P9 -- split-merge identity: the recurrence a streaming kernel relies on.
def test_split_merge_identity():
    rng = np.random.default_rng(8)
    B, H, Nq, Nk, d = 1, 2, 5, 70, 8
    Q, K, V = rand_bf16(rng, (B, H, Nq, d)), rand_bf16(rng, (B, H, Nk, d)), rand_bf16(rng, (B, H, Nk, d))
    sc = 0.4
    full = oracle.attention(Q, K, V, sc, want_logits=True)
    cut = 27
    p1 = oracle.attention(Q, K[:, :, :cut], V[:, :, :cut], sc, want_logits=True)
    p2 = oracle.attention(Q, K[:, :, cut:], V[:, :, cut:], sc, want_logits=True)
    m1 = p1["L"].max(-1, keepdims=True); l1 = np.exp(p1["L"] - m1).sum(-1, keepdims=True)
    m2 = p2["L"].max(-1, keepdims=True); l2 = np.exp(p2["L"] - m2).sum(-1, keepdims=True)
    m = np.maximum(m1, m2)
    w1, w2 = l1 * np.exp(m1 - m), l2 * np.exp(m2 - m)
    merged = (w1 * p1["O"] + w2 * p2["O"]) / (w1 + w2)
    assert np.max(np.abs(merged - full["O"])) < 1e-13


# P10 -- mask semantics.
def test_mask_equivalences():
    rng = np.random.default_rng(9)
    B, H, Nq, Nk, d = 3, 2, 4, 40, 8
    Q, K, V = rand_bf16(rng, (B, H, Nq, d)), rand_bf16(rng, (B, H, Nk, d)), rand_bf16(rng, (B, H, Nk, d))
    vl = np.array([40, 13, 1], dtype=np.int32)
    Om = oracle.attention(Q, K, V, 0.3, valid_len=vl, want_weights=True)
    for b in range(B):
        n = int(vl[b])
        Ot = oracle.attention(Q[b:b + 1], K[b:b + 1, :, :n], V[b:b + 1, :, :n], 0.3)["O"]
        assert np.max(np.abs(Om["O"][b:b + 1] - Ot)) == 0.0
        assert np.all(Om["A"][b, :, :, n:] == 0.0)
    O_all = oracle.attention(Q, K, V, 0.3, valid_len=np.full(B, Nk, np.int32))["O"]
    assert np.array_equal(O_all, oracle.attention(Q, K, V, 0.3)["O"])
    # finite garbage in the masked rows changes nothing
    K2, V2 = f32(K).copy(), f32(V).copy()
    for b in range(B):
        K2[b, :, vl[b]:] = 3.0e4
        V2[b, :, vl[b]:] = -7.0e4
    Og = oracle.attention(f32(Q), K2, V2, 0.3, valid_len=vl)["O"]
    assert np.array_equal(Og, oracle.attention(f32(Q), f32(K), f32(V), 0.3, valid_len=vl)["O"])
    # valid_len = 1: the row copies V[0]
    assert np.allclose(Om["O"][2], np.broadcast_to(f32(V)[2, :, 0:1].astype(np.float64), Om["O"][2].shape), atol=0)
    # fully masked batch: O = 0, no NaN
    Oz = oracle.attention(Q, K, V, 0.3, valid_len=np.array([0, 5, 40], np.int32))["O"]
    assert np.all(Oz[0] == 0.0) and np.all(np.isfinite(Oz))


# P11 -- brute force on tiny shapes (long double, explicit matrix, other loop order).
@pytest.mark.parametrize("Nq,Nk,d,B,H", [(1, 1, 1, 1, 1), (2, 3, 4, 1, 2), (3, 17, 4, 2, 1), (17, 129, 4, 1, 1),
                                         (2, 129, 64, 1, 1), (3, 2, 64, 2, 2)])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_brute_force_tiny(Nq, Nk, d, B, H, dtype):
    rng = np.random.default_rng(100 + Nq * 7 + Nk)
    if dtype == "bf16":
        Q, K, V = rand_bf16(rng, (B, H, Nq, d)), rand_bf16(rng, (B, H, Nk, d)), rand_bf16(rng, (B, H, Nk, d))
        Qf, Kf, Vf = f32(Q), f32(K), f32(V)
    else:
        Q = Qf = rng.standard_normal((B, H, Nq, d)).astype(np.float32)
        K = Kf = rng.standard_normal((B, H, Nk, d)).astype(np.float32)
        V = Vf = rng.standard_normal((B, H, Nk, d)).astype(np.float32)
    sc = 1 / math.sqrt(d)
    vl = None if B == 1 else np.array([Nk, max(1, Nk // 2)], dtype=np.int32)[:B]
    r = oracle.attention(Q, K, V, sc, valid_len=vl, want_weights=True)
    Ob, Ab = brute_force(Qf, Kf, Vf, sc, vl)
    assert np.max(np.abs(r["O"] - Ob.astype(np.float64))) < 1e-12
    assert np.max(np.abs(r["A"] - Ab.astype(np.float64))) < 1e-12


# Row selection returns exactly the rows of the full result, and bf16 bits == widened float32.
@pytest.mark.parametrize("Nq,Nk", [(5, 5), (3, 9), (9, 3), (1, 7), (17, 130)])
def test_causal_mask_pins(Nq, Nk):
    """Causal reading: query i sees keys j <= i + (Nk - Nq).  Pinned against an explicit mask matrix
    (independent numpy softmax over the kept logits), against per-row truncation through the unmasked
    oracle, and by two closed cases: the last query row equals the unmasked row, and with Nq = Nk the
    first row is V[0]."""
    rng = np.random.default_rng(100 * Nq + Nk)
    B, H, d = 2, 2, 4
    Q = rng.standard_normal((B, H, Nq, d)).astype(np.float32)
    K = rng.standard_normal((B, H, Nk, d)).astype(np.float32)
    V = rng.standard_normal((B, H, Nk, d)).astype(np.float32)
    vl = np.array([Nk, max(1, Nk - 2)], dtype=np.int32)
    scale = 0.7
    got = oracle.attention(Q, K, V, scale, valid_len=vl, causal=True, want_weights=True)
    O, A = got["O"], got["A"]
    # explicit mask matrix
    sc = np.float64(np.float32(scale))
    L = sc * np.einsum("bhid,bhjd->bhij", Q.astype(np.float64), K.astype(np.float64))
    i = np.arange(Nq)[:, None]; j = np.arange(Nk)[None, :]
    for b in range(B):
        keep = (j <= i + (Nk - Nq)) & (j < vl[b])
        for h in range(H):
            W = np.where(keep, np.exp(L[b, h] - L[b, h].max()), 0.0)
            den = W.sum(-1, keepdims=True)
            Wn = np.divide(W, den, out=np.zeros_like(W), where=den > 0)
            np.testing.assert_allclose(A[b, h], Wn, rtol=0, atol=1e-14)
            np.testing.assert_allclose(O[b, h], Wn @ V[b, h].astype(np.float64), rtol=0, atol=1e-13)
            assert np.all(A[b, h][~keep] == 0.0)
    # per-row truncation through the unmasked oracle
    for b in range(B):
        for ii in range(Nq):
            n = min(int(vl[b]), ii + 1 + Nk - Nq)
            if n <= 0:
                assert np.all(O[b, :, ii] == 0.0)
                continue
            ref = oracle.attention(Q[b:b + 1, :, ii:ii + 1], K[b:b + 1, :, :n], V[b:b + 1, :, :n], scale)["O"]
            np.testing.assert_allclose(O[b, :, ii], ref[0, :, 0], rtol=0, atol=1e-14)
    # the last query row is unaffected by the causal mask; with Nq == Nk the first row is V[0]
    plain = oracle.attention(Q, K, V, scale, valid_len=vl)["O"]
    np.testing.assert_allclose(O[:, :, -1], plain[:, :, -1], rtol=0, atol=1e-15)
    if Nq == Nk:
        np.testing.assert_allclose(O[:, :, 0], V[:, :, 0].astype(np.float64), rtol=0, atol=1e-15)


def test_row_sampling_and_dtype_paths_agree():
    rng = np.random.default_rng(11)
    B, H, Nq, Nk, d = 2, 3, 10, 21, 8
    Q, K, V = rand_bf16(rng, (B, H, Nq, d)), rand_bf16(rng, (B, H, Nk, d)), rand_bf16(rng, (B, H, Nk, d))
    vl = np.array([21, 9], dtype=np.int32)
    full = oracle.attention(Q, K, V, 0.2, valid_len=vl)["O"].reshape(-1, d)
    rows = np.array([0, 7, 10, 33, 59], dtype=np.int64)
    sub = oracle.attention(Q, K, V, 0.2, valid_len=vl, rows=rows, nthreads=2)["O"]
    assert np.array_equal(sub, full[rows])
    fullf = oracle.attention(f32(Q), f32(K), f32(V), 0.2, valid_len=vl)["O"].reshape(-1, d)
    assert np.array_equal(full, fullf)
    # thread count does not change anything
    assert np.array_equal(oracle.attention(Q, K, V, 0.2, valid_len=vl, nthreads=1)["O"].reshape(-1, d), full)


# P12 -- FLOP formula against the compute shares the paper prints.
def test_flop_formula_matches_printed_compute_share():
    D = 768  # BERT-base hidden size; per block: Q,K,V,O projections 8ND^2, two FCs (4x) 16ND^2, L+A 4N^2 D
    with open(os.path.join(GOLDEN, "la_compute_share.txt")) as f:
        rows = [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 3
    for n_s, pct_s in rows:
        N, pct = int(n_s), float(pct_s)
        w = inputs.Workload("x", 1, 12, N, N, 64)
        la = w.flops
        assert la == 4 * N * N * D
        share = la / (24 * N * D * D + la)
        assert abs(100 * share - pct) < 0.6, (N, share)


def test_bad_arguments_rejected():
    Q = np.zeros((1, 1, 2, 4), np.float32)
    with pytest.raises(ValueError):
        oracle.attention(Q, Q, Q, 1.0, valid_len=np.array([3], np.int32))
    with pytest.raises(ValueError):
        oracle.attention(Q, Q, Q, 1.0, rows=np.array([2], np.int64))


# ------------------------------------------------------------------------------------------------
# Additive bias of the logits (reading: added to the SCALED logit before the maximum; [B or 1, H or 1,
# Nq, Nk]; -inf switches a pair off).  Pinned by closed forms, invariances, mask equivalences and an
# independent numpy softmax.

def _rand_f32(rng, *shape):
    return rng.standard_normal(shape).astype(np.float32)


def test_bias_closed_form_and_not_scaled():
    # Q = 0: the weights are softmax(bias) whatever the scale; bias = log(1, 2, 3), V = (6, 12, 18) -> 14
    Q = np.zeros((1, 1, 2, 1), dtype=np.float32)
    K = np.array([0.3, -1.0, 2.0], dtype=np.float32).reshape(1, 1, 3, 1)
    V = np.array([6.0, 12.0, 18.0], dtype=np.float32).reshape(1, 1, 3, 1)
    bias = np.log(np.array([[1.0, 2.0, 3.0], [3.0, 2.0, 1.0]])).astype(np.float32).reshape(1, 1, 2, 3)
    r = oracle.attention(Q, K, V, 7.0, bias=bias, want_weights=True)
    assert np.abs(r["A"][0, 0, 0] - np.array([1, 2, 3]) / 6.0).max() < 1e-7       # (float32 logs)
    assert abs(r["O"][0, 0, 0, 0] - 14.0) < 1e-5 and abs(r["O"][0, 0, 1, 0] - 10.0) < 1e-5
    # scale = 0 with arbitrary Q: again softmax(bias) -- the bias is not multiplied by the scale
    Q2 = _rand_f32(np.random.default_rng(1), 1, 1, 2, 1)
    r0 = oracle.attention(Q2, K, V, 0.0, bias=bias, want_weights=True)
    assert np.abs(r0["A"] - r["A"]).max() < 1e-15
    # ... and with scale != 0 it differs from scaling the bias too
    r1 = oracle.attention(Q2, K, V, 2.0, bias=bias)["O"]
    r2 = oracle.attention(Q2, K, V, 2.0, bias=(2.0 * bias).astype(np.float32))["O"]
    assert np.abs(r1 - r2).max() > 1e-3


def test_bias_invariances_and_independent_softmax():
    rng = np.random.default_rng(12)
    B, H, Nq, Nk, d = 2, 3, 5, 9, 4
    Q, K, V = _rand_f32(rng, B, H, Nq, d), _rand_f32(rng, B, H, Nk, d), _rand_f32(rng, B, H, Nk, d)
    bias = _rand_f32(rng, B, H, Nq, Nk)
    s = np.float64(np.float32(0.6))
    got = oracle.attention(Q, K, V, 0.6, bias=bias, want_lse=True)
    S = s * np.einsum("bhid,bhjd->bhij", Q.astype(np.float64), K.astype(np.float64)) + bias
    A = np.exp(S - S.max(-1, keepdims=True)); A /= A.sum(-1, keepdims=True)
    assert np.abs(got["O"] - A @ V.astype(np.float64)).max() < 1e-13
    from scipy.special import logsumexp
    assert np.abs(got["LSE"] - logsumexp(S, axis=-1)).max() < 1e-12
    # a per-row constant added to the bias changes nothing (exactly representable shifts)
    shift = (np.round(rng.standard_normal((B, H, Nq, 1)) * 4) / 4).astype(np.float32)
    b16 = (np.round(bias * 16) / 16).astype(np.float32)
    o1 = oracle.attention(Q, K, V, 0.6, bias=b16)["O"]
    o2 = oracle.attention(Q, K, V, 0.6, bias=(b16 + shift).astype(np.float32))["O"]
    assert np.abs(o1 - o2).max() < 1e-13
    # zero bias = no bias, bit for bit
    assert np.array_equal(oracle.attention(Q, K, V, 0.6, bias=np.zeros_like(bias))["O"], oracle.attention(Q, K, V, 0.6)["O"])
    # broadcast over batch and / or head = the explicitly repeated tensor
    for shape in ((1, H), (B, 1), (1, 1)):
        small = _rand_f32(rng, shape[0], shape[1], Nq, Nk)
        full = np.ascontiguousarray(np.broadcast_to(small, (B, H, Nq, Nk)))
        assert np.array_equal(oracle.attention(Q, K, V, 0.6, bias=small)["O"], oracle.attention(Q, K, V, 0.6, bias=full)["O"])
    # bf16 bias bits = the widened values
    bits = inputs.f32_to_bf16_bits(bias).reshape(bias.shape)
    wide = inputs.bf16_bits_to_f32(bits).reshape(bias.shape)
    assert np.array_equal(oracle.attention(Q, K, V, 0.6, bias=bits)["O"], oracle.attention(Q, K, V, 0.6, bias=wide)["O"])


def test_bias_minus_infinity_is_a_mask():
    rng = np.random.default_rng(13)
    B, H, Nq, Nk, d = 2, 2, 6, 8, 4
    Q, K, V = _rand_f32(rng, B, H, Nq, d), _rand_f32(rng, B, H, Nk, d), _rand_f32(rng, B, H, Nk, d)
    # key padding: -inf on keys j >= valid_len[b]
    vl = np.array([5, 8], dtype=np.int32)
    bias = np.zeros((B, 1, Nq, Nk), dtype=np.float32)
    bias[0, :, :, 5:] = -np.inf
    a = oracle.attention(Q, K, V, 0.7, bias=bias, want_weights=True)
    b = oracle.attention(Q, K, V, 0.7, valid_len=vl, want_weights=True)
    assert np.abs(a["O"] - b["O"]).max() < 1e-15 and np.array_equal(a["A"] == 0, b["A"] == 0)
    # causal: -inf above the diagonal (offset Nk - Nq)
    cb = np.where(np.arange(Nk)[None, :] <= np.arange(Nq)[:, None] + (Nk - Nq), 0.0, -np.inf).astype(np.float32)
    a = oracle.attention(Q, K, V, 0.7, bias=cb.reshape(1, 1, Nq, Nk))["O"]
    assert np.abs(a - oracle.attention(Q, K, V, 0.7, causal=True)["O"]).max() < 1e-15
    # a row with every pair switched off: O = 0, lse = -inf, no NaN
    bias = np.zeros((1, 1, Nq, Nk), dtype=np.float32)
    bias[0, 0, 2, :] = -np.inf
    r = oracle.attention(Q, K, V, 0.7, bias=bias, want_lse=True)
    assert np.all(r["O"][:, :, 2] == 0) and np.all(np.isneginf(r["LSE"][:, :, 2])) and np.all(np.isfinite(r["O"]))


# ------------------------------------------------------------------------------------------------
# Pruned (block-sparse) attention: a byte map over blocks of the logit matrix; pruned pairs take no part.

def test_block_mask_is_a_minus_infinity_bias_on_the_pruned_blocks():
    rng = np.random.default_rng(21)
    B, H, Nq, Nk, d, blk = 2, 2, 10, 14, 4, 4
    Q, K, V = _rand_f32(rng, B, H, Nq, d), _rand_f32(rng, B, H, Nk, d), _rand_f32(rng, B, H, Nk, d)
    tq, tk = 3, 4
    for shape in ((B, H), (1, H), (B, 1), (1, 1)):
        m = (rng.random(shape + (tq, tk)) < 0.5).astype(np.uint8)
        m[..., 1, :] = 0                                   # a block row with nothing kept
        m[..., 0, 0] = 1
        # the same thing as an explicit bias tensor (the bias path has its own pins)
        full = np.repeat(np.repeat(m, blk, axis=2), blk, axis=3)[:, :, :Nq, :Nk]
        bias = np.where(full != 0, 0.0, -np.inf).astype(np.float32)
        a = oracle.attention(Q, K, V, 0.6, block_mask=m, block=blk, want_weights=True, want_lse=True)
        b = oracle.attention(Q, K, V, 0.6, bias=bias, want_weights=True, want_lse=True)
        assert np.array_equal(a["O"], b["O"]) and np.array_equal(a["A"], b["A"])
        assert np.array_equal(a["LSE"], b["LSE"])
        assert np.all(a["O"][:, :, 4:8] == 0) and np.all(np.isneginf(a["LSE"][:, :, 4:8]))   # rows of block row 1
        # an independent softmax over the kept columns only
        S = np.float64(np.float32(0.6)) * np.einsum("bhid,bhjd->bhij", Q.astype(np.float64), K.astype(np.float64))
        S = np.where(np.broadcast_to(full, S.shape) != 0, S, -np.inf)
        with np.errstate(invalid="ignore"):
            W = np.exp(S - S.max(-1, keepdims=True))
        W = np.nan_to_num(W)
        den = W.sum(-1, keepdims=True)
        ref = np.where(den > 0, W / np.where(den > 0, den, 1), 0) @ V.astype(np.float64)
        assert np.abs(a["O"] - ref).max() < 1e-13


def test_block_mask_special_cases():
    rng = np.random.default_rng(22)
    B, H, Nq, Nk, d, blk = 1, 2, 9, 12, 3, 4
    Q, K, V = _rand_f32(rng, B, H, Nq, d), _rand_f32(rng, B, H, Nk, d), _rand_f32(rng, B, H, Nk, d)
    ones = np.ones((1, 1, 3, 3), dtype=np.uint8)
    assert np.array_equal(oracle.attention(Q, K, V, 0.5, block_mask=ones, block=blk)["O"], oracle.attention(Q, K, V, 0.5)["O"])
    # pruning the trailing block column of every row = a key-padding mask at 8 keys = truncation
    m = ones.copy(); m[..., 2] = 0
    assert np.array_equal(oracle.attention(Q, K, V, 0.5, block_mask=m, block=blk)["O"],
                          oracle.attention(Q, K, V, 0.5, valid_len=np.array([8], dtype=np.int32))["O"])
    # the lower block triangle kept + the causal mask = the causal mask alone (Nq = Nk, blocks on the diagonal)
    Q2 = _rand_f32(rng, B, H, 12, d)
    tri = np.tril(np.ones((3, 3), dtype=np.uint8)).reshape(1, 1, 3, 3)
    assert np.array_equal(oracle.attention(Q2, K, V, 0.5, block_mask=tri, block=blk, causal=True)["O"],
                          oracle.attention(Q2, K, V, 0.5, causal=True)["O"])
    # one kept block: the row attends exactly those keys
    one = np.zeros((1, 1, 3, 3), dtype=np.uint8); one[0, 0, :, 1] = 1
    got = oracle.attention(Q, K, V, 0.5, block_mask=one, block=blk)["O"]
    assert np.abs(got - oracle.attention(Q, K[:, :, 4:8], V[:, :, 4:8], 0.5)["O"]).max() < 1e-15
    # sampled rows see the same map
    rows = np.array([0, 5, 13], dtype=np.int64)
    m = (rng.random((1, 2, 3, 3)) < 0.6).astype(np.uint8); m[..., 0] = 1
    allr = oracle.attention(Q, K, V, 0.5, block_mask=m, block=blk)["O"].reshape(-1, d)
    assert np.array_equal(oracle.attention(Q, K, V, 0.5, block_mask=m, block=blk, rows=rows)["O"], allr[rows])
