"""Pins of the backward oracle (oracle.attention_bwd) and of the forward oracle's log-sum-exp
output to things other than themselves: finite differences of the forward oracle, a long-double
brute force built from the explicit softmax Jacobian, invariances of the forward function that
translate into identities of the gradients, closed forms, and mask / causal equivalences with
truncation.  All CPU; all in float32 inputs so that the perturbations of the finite differences
are representable."""
import numpy as np
import pytest

import oracle


def _rand(rng, B, H, Nq, Nk, d, sigma=1.0):
    f = lambda *s: (rng.standard_normal(s) * sigma).astype(np.float32)
    return f(B, H, Nq, d), f(B, H, Nk, d), f(B, H, Nk, d), f(B, H, Nq, d)


def _loss(Q, K, V, dO, scale, **kw):
    """The scalar whose gradient attention_bwd returns: sum of O * dO."""
    return float(np.sum(oracle.attention(Q, K, V, scale, **kw)["O"] * dO.astype(np.float64)))


@pytest.mark.parametrize("kw", [dict(), dict(causal=True), dict(valid_len=[3, 5])])
def test_central_finite_differences_of_the_forward_oracle(kw):
    rng = np.random.default_rng(11)
    B, H, Nq, Nk, d = 2, 2, 4, 5, 3
    Q, K, V, dO = _rand(rng, B, H, Nq, Nk, d)
    scale = 0.7
    kw = dict(kw)
    if "valid_len" in kw:
        kw["valid_len"] = np.asarray(kw["valid_len"], dtype=np.int32)
    g = oracle.attention_bwd(Q, K, V, dO, scale, **kw)
    h = 2.0 ** -9                                      # exactly representable step; inputs are O(1) float32
    for name, X in (("dQ", Q), ("dK", K), ("dV", V)):
        num = np.zeros(X.shape, dtype=np.float64)
        it = np.nditer(X, flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            keep = X[idx]
            X[idx] = keep + np.float32(h)
            up = _loss(Q, K, V, dO, scale, **kw)
            X[idx] = keep - np.float32(h)
            dn = _loss(Q, K, V, dO, scale, **kw)
            X[idx] = keep
            num[idx] = (up - dn) / (2 * h)
        # the central difference is exact to O(h^2) = 4e-6 times third derivatives of order 1
        assert np.abs(num - g[name]).max() < 5e-5, (name, np.abs(num - g[name]).max())
        assert np.abs(g[name]).max() > 1e-2            # (the comparison is not between zeros)


def _brute_force(Q, K, V, dO, scale, n_valid):
    """Explicit weight matrix and explicit softmax Jacobian in long double, other loop order, no max
    subtraction.  n_valid[i] = number of keys row i sees.  One head: Q [Nq,d] ..."""
    ld = np.longdouble
    Q, K, V, dO = (x.astype(ld) for x in (Q, K, V, dO))
    Nq, d = Q.shape
    Nk = K.shape[0]
    A = np.zeros((Nq, Nk), dtype=ld)
    for i in range(Nq):
        e = np.exp(ld(scale) * (K[:n_valid[i]] @ Q[i]))
        if n_valid[i] > 0:
            A[i, :n_valid[i]] = e / e.sum()
    dA = dO @ V.T
    dS = np.zeros_like(A)
    for i in range(Nq):
        # J[j,k] = dA_k/dS_j = A_k (delta_jk - A_j): dS_j = sum_k J[j,k] dA_k
        J = np.diag(A[i]) - np.outer(A[i], A[i])
        dS[i] = J @ dA[i]
    return (ld(scale) * dS @ K).astype(np.float64), (ld(scale) * dS.T @ Q).astype(np.float64), (A.T @ dO).astype(np.float64)


@pytest.mark.parametrize("shape", [(1, 1, 1, 1, 1), (1, 2, 3, 2, 4), (2, 1, 17, 9, 5), (1, 1, 5, 129, 8), (1, 1, 6, 6, 64)])
@pytest.mark.parametrize("causal", [False, True])
def test_long_double_brute_force_with_the_explicit_jacobian(shape, causal):
    rng = np.random.default_rng(sum(shape) + causal)
    B, H, Nq, Nk, d = shape
    Q, K, V, dO = _rand(rng, *shape)
    scale = 0.37
    g = oracle.attention_bwd(Q, K, V, dO, scale, causal=causal)
    for b in range(B):
        for h in range(H):
            nv = [max(0, min(Nk, i + 1 + Nk - Nq)) if causal else Nk for i in range(Nq)]
            dq, dk, dv = _brute_force(Q[b, h], K[b, h], V[b, h], dO[b, h], np.float32(scale), nv)
            assert np.abs(dq - g["dQ"][b, h]).max() < 1e-12
            assert np.abs(dk - g["dK"][b, h]).max() < 1e-12
            assert np.abs(dv - g["dV"][b, h]).max() < 1e-12


def test_gradient_identities_from_invariances_of_the_forward():
    rng = np.random.default_rng(5)
    Q, K, V, dO = _rand(rng, 2, 3, 7, 11, 6)
    g = oracle.attention_bwd(Q, K, V, dO, 0.5)
    # shifting every key by the same vector adds a per-row constant to the logits and leaves O alone,
    # so the key gradients sum to zero over the keys (this is what the subtracted row term buys)
    assert np.abs(g["dK"].sum(axis=2)).max() < 1e-13
    assert np.abs(g["dK"]).max() > 1e-2
    # O is linear in V with weights that sum to one: sum_j dV[j] = sum_i dO[i]
    assert np.abs(g["dV"].sum(axis=2) - dO.astype(np.float64).sum(axis=2)).max() < 1e-12
    # scaling Q by c and K by 1/c leaves the logits alone: <Q, dQ> = <K, dK> (per head)
    lhs = np.sum(Q.astype(np.float64) * g["dQ"], axis=(2, 3))
    rhs = np.sum(K.astype(np.float64) * g["dK"], axis=(2, 3))
    assert np.abs(lhs - rhs).max() < 1e-12 and np.abs(lhs).max() > 1e-3


def test_linear_in_dO_and_zero_for_zero():
    rng = np.random.default_rng(6)
    Q, K, V, dO1 = _rand(rng, 1, 2, 5, 8, 4)
    # multiples of 1/64, so that the combination below is exact in float32
    dO1 = (np.round(dO1 * 64) / 64).astype(np.float32)
    dO2 = (np.round(rng.standard_normal(dO1.shape) * 64) / 64).astype(np.float32)
    g1 = oracle.attention_bwd(Q, K, V, dO1, 0.9)
    g2 = oracle.attention_bwd(Q, K, V, dO2, 0.9)
    g3 = oracle.attention_bwd(Q, K, V, (2 * dO1 - 4 * dO2).astype(np.float32), 0.9)
    for n in ("dQ", "dK", "dV"):
        assert np.abs(g3[n] - (2 * g1[n] - 4 * g2[n])).max() < 1e-12
    g0 = oracle.attention_bwd(Q, K, V, np.zeros_like(dO1), 0.9)
    assert all(np.all(g0[n] == 0) for n in ("dQ", "dK", "dV"))


def test_closed_forms_one_key_and_zero_queries():
    rng = np.random.default_rng(7)
    # one key: the weight is 1 whatever Q and K are -> dQ = dK = 0, dV = sum of dO over the rows
    Q, K, V, dO = _rand(rng, 1, 2, 6, 1, 5)
    g = oracle.attention_bwd(Q, K, V, dO, 1.3)
    assert np.abs(g["dQ"]).max() < 1e-15 and np.abs(g["dK"]).max() < 1e-15
    assert np.abs(g["dV"][:, :, 0] - dO.astype(np.float64).sum(axis=2)).max() < 1e-13
    # Q = 0: uniform weights 1/n -> dV[j] = mean-weight * sum_i dO[i]; dK = 0 (multiplied by Q);
    # dQ[i] = scale/n * sum_j (dA[i,j] - mean_j dA[i,:]) K[j]
    Q, K, V, dO = _rand(rng, 1, 1, 4, 7, 3)
    Q[:] = 0
    s = 0.8
    g = oracle.attention_bwd(Q, K, V, dO, s)
    n = 7
    assert np.abs(g["dV"][0, 0] - dO[0, 0].astype(np.float64).sum(axis=0)[None, :] / n).max() < 1e-14
    assert np.abs(g["dK"]).max() < 1e-15
    dA = dO[0, 0].astype(np.float64) @ V[0, 0].astype(np.float64).T
    want = np.float64(np.float32(s)) / n * (dA - dA.mean(axis=1, keepdims=True)) @ K[0, 0].astype(np.float64)
    assert np.abs(g["dQ"][0, 0] - want).max() < 1e-14


def test_masks_equal_truncation_and_rows_without_keys_give_nothing():
    rng = np.random.default_rng(8)
    B, H, Nq, Nk, d = 2, 2, 5, 9, 4
    Q, K, V, dO = _rand(rng, B, H, Nq, Nk, d)
    vl = np.array([4, 0], dtype=np.int32)
    g = oracle.attention_bwd(Q, K, V, dO, 0.6, valid_len=vl)
    # batch 0: identical to the unmasked call on the first 4 keys; masked keys get zero gradients
    t = oracle.attention_bwd(Q[:1], K[:1, :, :4], V[:1, :, :4], dO[:1], 0.6)
    assert np.abs(g["dQ"][0] - t["dQ"][0]).max() < 1e-14
    assert np.abs(g["dK"][0, :, :4] - t["dK"][0]).max() < 1e-14 and np.abs(g["dV"][0, :, :4] - t["dV"][0]).max() < 1e-14
    assert np.all(g["dK"][0, :, 4:] == 0) and np.all(g["dV"][0, :, 4:] == 0)
    # garbage in masked keys changes nothing
    K2, V2 = K.copy(), V.copy()
    K2[0, :, 4:] = 1e6; V2[0, :, 4:] = -1e6
    g2 = oracle.attention_bwd(Q, K2, V2, dO, 0.6, valid_len=vl)
    assert all(np.array_equal(g[n], g2[n]) for n in ("dQ", "dK", "dV"))
    # batch 1 has no valid key: nothing flows, lse is the empty sum
    assert all(np.all(g[n][1] == 0) for n in ("dQ", "dK", "dV"))
    assert np.all(np.isneginf(g["LSE"][1]))
    # causal: row i is the unmasked problem on keys 0 .. i + (Nk - Nq); sum the per-row problems
    c = oracle.attention_bwd(Q, K, V, dO, 0.6, causal=True)
    dK = np.zeros_like(c["dK"]); dV = np.zeros_like(c["dV"])
    for i in range(Nq):
        n = i + 1 + Nk - Nq
        r = oracle.attention_bwd(Q[:, :, i:i + 1], K[:, :, :n], V[:, :, :n], dO[:, :, i:i + 1], 0.6)
        assert np.abs(c["dQ"][:, :, i] - r["dQ"][:, :, 0]).max() < 1e-14
        dK[:, :, :n] += r["dK"]; dV[:, :, :n] += r["dV"]
    assert np.abs(c["dK"] - dK).max() < 1e-13 and np.abs(c["dV"] - dV).max() < 1e-13
    # Nq > Nk under the causal mask: the first Nq - Nk rows see no key
    Q3, K3, V3, dO3 = _rand(rng, 1, 1, 6, 3, 4)
    c3 = oracle.attention_bwd(Q3, K3, V3, dO3, 0.6, causal=True)
    assert np.all(c3["dQ"][0, 0, :3] == 0) and np.all(np.isneginf(c3["LSE"][0, 0, :3])) and np.abs(c3["dQ"][0, 0, 3:]).max() > 0


def test_head_subset_and_bf16_inputs_and_threads():
    rng = np.random.default_rng(9)
    from paper_2107_06419_b200 import inputs
    f = lambda *s: inputs.f32_to_bf16_bits(rng.standard_normal(s).astype(np.float32)).reshape(s)
    Q, K, V, dO = f(2, 3, 6, 8), f(2, 3, 10, 8), f(2, 3, 10, 8), f(2, 3, 6, 8)
    full = oracle.attention_bwd(Q, K, V, dO, 0.35, causal=True, nthreads=3)
    sub = oracle.attention_bwd(Q, K, V, dO, 0.35, causal=True, heads=[4, 1], nthreads=1)
    for n in ("dQ", "dK", "dV", "LSE"):
        assert np.array_equal(sub[n][0], full[n][1, 1]) and np.array_equal(sub[n][1], full[n][0, 1])
    # the bf16 path is the float32 path on the widened values
    w = lambda b: inputs.bf16_bits_to_f32(b).reshape(b.shape)
    g32 = oracle.attention_bwd(w(Q), w(K), w(V), w(dO), 0.35, causal=True)
    assert all(np.array_equal(g32[n], full[n]) for n in ("dQ", "dK", "dV"))


def test_lse_against_an_independent_log_sum_exp():
    from scipy.special import logsumexp
    rng = np.random.default_rng(10)
    Q, K, V, dO = _rand(rng, 2, 2, 9, 13, 5, sigma=3.0)
    vl = np.array([13, 6], dtype=np.int32)
    s = np.float64(np.float32(0.45))
    for causal in (False, True):
        fwd = oracle.attention(Q, K, V, 0.45, valid_len=vl, causal=causal, want_lse=True, want_logits=True)
        bwd = oracle.attention_bwd(Q, K, V, dO, 0.45, valid_len=vl, causal=causal)
        logits = s * np.einsum("bhid,bhjd->bhij", Q.astype(np.float64), K.astype(np.float64))
        for b in range(2):
            for i in range(9):
                n = min(int(vl[b]), i + 1 + 13 - 9) if causal else int(vl[b])
                want = logsumexp(logits[b, :, i, :n], axis=-1)
                assert np.abs(fwd["LSE"][b, :, i] - want).max() < 1e-12
                assert np.abs(bwd["LSE"][b, :, i] - want).max() < 1e-12
        # exp(logit - lse) reproduces the weights
        A = oracle.attention(Q, K, V, 0.45, valid_len=vl, causal=causal, want_weights=True)["A"]
        with np.errstate(invalid="ignore"):
            rebuilt = np.exp(fwd["L"] - fwd["LSE"][..., None])
        assert np.abs(np.nan_to_num(rebuilt) - A).max() < 1e-13
    # sampled rows return their own lse
    rows = np.array([0, 17, 35], dtype=np.int64)
    part = oracle.attention(Q, K, V, 0.45, valid_len=vl, rows=rows, want_lse=True)["LSE"]
    allr = oracle.attention(Q, K, V, 0.45, valid_len=vl, want_lse=True)["LSE"].reshape(-1)
    assert np.array_equal(part, allr[rows])
