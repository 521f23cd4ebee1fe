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
