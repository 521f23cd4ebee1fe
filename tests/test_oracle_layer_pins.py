"""Pins for the attention-layer oracle (Section 2, steps 1-5), independent of the oracle's code.

A plausible mistake -- Key and Value blocks of the stacked weights swapped, heads interleaved
instead of blocked, a transposed weight, the concatenation order of the heads, rounding at the
wrong place -- fails at least one of these.
"""
import numpy as np
import pytest

import oracle
from paper_2107_06419_b200 import inputs


def bits(x):
    x = np.asarray(x, dtype=np.float32)
    return inputs.f32_to_bf16_bits(x).reshape(x.shape)


def f64(b):
    return inputs.bf16_bits_to_f32(b).reshape(b.shape).astype(np.float64)


def test_bf16_rounding_helpers_against_exact_cases():
    # 1 + 2^-8 is a tie between 1 and 1 + 2^-7: ties go to the even mantissa (1.0); 1 + 3*2^-8 ties up to 1 + 2^-6
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20, -2.5, 0.0, 3.0e38])
    got = oracle.bf16_bits_to_f64(oracle.round_to_bf16_bits(x))
    want = np.array([1.0, 1.0, 1.0 + 2.0 ** -6, 1.0 + 2.0 ** -7, -2.5, 0.0, float(np.float32(2.0 ** 127 * 1.7578125))])
    assert np.array_equal(got[:6], want[:6])
    assert abs(got[6] - 3.0e38) <= 3.0e38 * 2.0 ** -8
    # every bf16 value is a fixed point of the round trip
    allbits = np.arange(0, 0x7F80, dtype=np.uint16)
    assert np.array_equal(oracle.round_to_bf16_bits(oracle.bf16_bits_to_f64(allbits)), allbits)


def test_projection_by_hand_worked_example():
    # B = 1, N = 2 tokens, Dm = 2, H = 2 heads of d = 1.  Stacked weights: rows Q(h0), Q(h1), K(h0), K(h1), V(h0), V(h1).
    X = bits([[[1.0, 2.0], [3.0, -1.0]]])
    W = bits([[1, 0], [0, 1], [1, 1], [2, 0], [0, -1], [1, -1]])
    q, k, v = oracle.qkv_projection(X, W, H=2, d=1)
    assert q.shape == (1, 2, 2, 1)
    assert np.array_equal(q[0, :, :, 0], [[1.0, 3.0], [2.0, -1.0]])      # head 0 takes x0, head 1 takes x1
    assert np.array_equal(k[0, :, :, 0], [[3.0, 2.0], [2.0, 6.0]])       # x0 + x1 ; 2 x0
    assert np.array_equal(v[0, :, :, 0], [[-2.0, 1.0], [-1.0, 4.0]])     # -x1 ; x0 - x1
    # output projection: Y[n, j] = sum over (h, c) of O[h, n, c] Wo[j, h*d + c]
    O = np.array([[[[1.0], [2.0]], [[10.0], [20.0]]]])                   # [1, H=2, N=2, d=1]
    Wo = bits([[1, 0], [0, 1], [1, 1]])                                  # Dm = 3
    Y = oracle.out_projection(O, Wo)
    assert np.array_equal(Y[0], [[1.0, 10.0, 11.0], [2.0, 20.0, 22.0]])


def test_one_hot_weights_reduce_the_layer_to_plain_attention():
    rng = np.random.default_rng(3)
    B, N, H, d = 2, 9, 2, 4
    Dm = 3 * H * d
    X = bits(rng.standard_normal((B, N, Dm)))
    Wqkv = bits(np.eye(3 * H * d, Dm))                                   # feature f of the stack = input column f
    Wo = bits(np.eye(H * d, H * d))
    out = oracle.attention_layer(X, Wqkv, Wo, H, d, 0.5)
    x = f64(X)
    Q = x[:, :, 0:H * d].reshape(B, N, H, d).transpose(0, 2, 1, 3)
    K = x[:, :, H * d:2 * H * d].reshape(B, N, H, d).transpose(0, 2, 1, 3)
    V = x[:, :, 2 * H * d:].reshape(B, N, H, d).transpose(0, 2, 1, 3)
    assert np.array_equal(f64(out["Q"]), Q) and np.array_equal(f64(out["K"]), K) and np.array_equal(f64(out["V"]), V)
    ref = oracle.attention(bits(Q), bits(K), bits(V), 0.5)["O"]
    assert np.array_equal(out["O"], oracle.round_to_bf16_bits(ref))
    # identity output weights: Y is the concatenation of the heads of the stored (rounded) O
    Ocat = f64(out["O"]).transpose(0, 2, 1, 3).reshape(B, N, H * d)
    assert np.array_equal(out["Y"], Ocat)


def test_brute_force_loops_on_a_tiny_layer():
    rng = np.random.default_rng(11)
    B, N, H, d, Dm = 1, 5, 2, 2, 3
    X = bits(rng.standard_normal((B, N, Dm)))
    Wqkv = bits(rng.standard_normal((3 * H * d, Dm)))
    Wo = bits(rng.standard_normal((Dm, H * d)))
    out = oracle.attention_layer(X, Wqkv, Wo, H, d, 0.7, causal=True)
    x, w, wo = f64(X), f64(Wqkv), f64(Wo)
    rb = lambda a: f64(bits(np.float32(a)))                              # storage rounding, by another route
    Q = np.zeros((H, N, d)); K = np.zeros((H, N, d)); V = np.zeros((H, N, d))
    for h in range(H):
        for n in range(N):
            for c in range(d):
                Q[h, n, c] = rb(sum(x[0, n, k] * w[h * d + c, k] for k in range(Dm)))
                K[h, n, c] = rb(sum(x[0, n, k] * w[H * d + h * d + c, k] for k in range(Dm)))
                V[h, n, c] = rb(sum(x[0, n, k] * w[2 * H * d + h * d + c, k] for k in range(Dm)))
    sc = float(np.float32(0.7))
    O = np.zeros((H, N, d))
    for h in range(H):
        for i in range(N):
            e = [np.exp(sc * sum(Q[h, i, c] * K[h, j, c] for c in range(d))) for j in range(i + 1)]   # causal: j <= i
            for c in range(d):
                O[h, i, c] = rb(sum(e[j] * V[h, j, c] for j in range(i + 1)) / sum(e))
    for n in range(N):
        for j in range(Dm):
            y = sum(O[h, n, c] * wo[j, h * d + c] for h in range(H) for c in range(d))
            assert abs(out["Y"][0, n, j] - y) <= 1e-12 * max(1.0, abs(y))
    assert np.array_equal(f64(out["O"])[0], O)


def test_output_projection_is_linear_in_its_weights():
    rng = np.random.default_rng(5)
    O = rng.standard_normal((2, 3, 4, 2))
    W1 = bits(rng.standard_normal((5, 6))); W2 = bits(rng.standard_normal((5, 6)))
    # W1 + W2 is taken in double (not re-rounded): build it as bf16-exact sums of small integers
    W1 = bits(np.round(f64(W1) * 4) / 4); W2 = bits(np.round(f64(W2) * 4) / 4)
    Ws = bits(f64(W1) + f64(W2))
    assert np.array_equal(f64(Ws), f64(W1) + f64(W2))
    y = oracle.out_projection(O, W1) + oracle.out_projection(O, W2)
    assert np.allclose(oracle.out_projection(O, Ws), y, rtol=0, atol=1e-12)


def test_fully_connected_by_hand():
    X = bits([[1.0, 2.0, 3.0], [0.5, -1.0, 0.0]])
    W = bits([[1, 0, 0], [0, 1, 1], [2, 2, 2], [-1, 0, 1]])              # [Nout = 4, K = 3]
    Y = oracle.fully_connected(X, W)
    assert np.array_equal(Y, [[1.0, 5.0, 12.0, 2.0], [0.5, -1.0, -1.0, -0.5]])
    # leading dimensions are kept
    assert oracle.fully_connected(X.reshape(1, 2, 3), W).shape == (1, 2, 4)


# ------------------------------------------------------------------------------------------------
# The block's normalisation layer (reading: layer normalisation over the features, after the residual add)

def _bits(a):
    return inputs.f32_to_bf16_bits(np.asarray(a, dtype=np.float32)).reshape(np.shape(a))


def test_layer_norm_hand_example_and_moments():
    # z = (1, 2, 3, 4): mean 2.5, biased variance 1.25 -> (z - 2.5) / sqrt(1.25); eps = 0
    X = _bits([[1.0, 2.0, 3.0, 4.0]])
    one, zero = _bits(np.ones(4)), _bits(np.zeros(4))
    y = oracle.layer_norm(X, one, zero, 0.0)
    assert np.abs(y[0] - np.array([-1.5, -0.5, 0.5, 1.5]) / np.sqrt(1.25)).max() < 1e-15
    # gamma scales and beta shifts feature by feature
    y2 = oracle.layer_norm(X, _bits([2.0, 1.0, 0.5, -1.0]), _bits([0.0, 1.0, 2.0, 3.0]), 0.0)
    assert np.abs(y2[0] - (np.array([2.0, 1.0, 0.5, -1.0]) * y[0] + np.array([0.0, 1.0, 2.0, 3.0]))).max() < 1e-15
    # random rows: zero mean and unit (biased) variance of the output when gamma = 1, beta = 0, eps = 0
    rng = np.random.default_rng(3)
    X = _bits(rng.standard_normal((5, 7, 64)) * 3 + 1)
    y = oracle.layer_norm(X, _bits(np.ones(64)), _bits(np.zeros(64)), 0.0)
    assert np.abs(y.mean(-1)).max() < 1e-14 and np.abs((y ** 2).mean(-1) - 1).max() < 1e-13


def test_layer_norm_invariances_residual_and_eps():
    rng = np.random.default_rng(4)
    x = np.round(rng.standard_normal((6, 32)) * 8) / 8           # exactly representable, also after the maps below
    g, b = _bits(rng.standard_normal(32)), _bits(rng.standard_normal(32))
    y = oracle.layer_norm(_bits(x), g, b, 0.0)
    # shifting a row by a constant and scaling it by a positive constant change nothing (eps = 0)
    assert np.abs(oracle.layer_norm(_bits(4 * x + 2), g, b, 0.0) - y).max() < 1e-13
    # a negative scale flips the normalised row: y -> 2 beta - y
    assert np.abs(oracle.layer_norm(_bits(-x), g, b, 0.0) - (2 * oracle.bf16_bits_to_f64(b) - y)).max() < 1e-13
    # the residual is added before the statistics: LN(x, residual = r) = LN(x + r)
    r = np.round(rng.standard_normal((6, 32)) * 8) / 8
    assert np.array_equal(oracle.layer_norm(_bits(x), g, b, 1e-5, residual=_bits(r)), oracle.layer_norm(_bits(x + r), g, b, 1e-5))
    # eps enters under the root, next to the variance: a constant row gives exactly beta, and a row of
    # variance v is scaled by sqrt(v / (v + eps))
    c = oracle.layer_norm(_bits(np.full((1, 32), 3.0)), g, b, 1e-5)
    assert np.array_equal(c[0], oracle.bf16_bits_to_f64(b))
    v = x[0].var()
    e = np.float64(np.float32(0.5))
    lhs = oracle.layer_norm(_bits(x[:1]), _bits(np.ones(32)), _bits(np.zeros(32)), 0.5)
    rhs = oracle.layer_norm(_bits(x[:1]), _bits(np.ones(32)), _bits(np.zeros(32)), 0.0) * np.sqrt(v / (v + e))
    assert np.abs(lhs - rhs).max() < 1e-14


def test_layer_norm_against_an_independent_library_routine():
    import torch
    rng = np.random.default_rng(5)
    X, R = _bits(rng.standard_normal((3, 9, 128))), _bits(rng.standard_normal((3, 9, 128)))
    g, b = _bits(rng.standard_normal(128)), _bits(rng.standard_normal(128))
    f = lambda bits: torch.from_numpy(oracle.bf16_bits_to_f64(bits))
    want = torch.nn.functional.layer_norm(f(X) + f(R), (128,), f(g), f(b), eps=float(np.float32(1e-5))).numpy()
    assert np.abs(oracle.layer_norm(X, g, b, 1e-5, residual=R) - want).max() < 1e-12
