"""GPU parity of the attention layer (Section 2, steps 1-5) against the oracle, through the C ABI.

The projections accumulate in fp32 where the oracle uses double, so a stored bf16 intermediate may
land on the neighbouring bf16 value when the exact result sits next to a rounding boundary: Q, K, V
are compared within one bf16 step, the layer output with the bars of the attention path.
"""
import numpy as np
import pytest
import torch

import oracle
from helpers import BF16_MAX, BF16_MEAN, BF16_REL_MAX, bf16_tensor, bf16_to_f64, rand_bits

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def api():
    from paper_2107_06419_b200 import api as _api
    return _api


def make_layer(rng, B, N, H, d, Dm):
    X = rand_bits(rng, (B, N, Dm))
    Wqkv = rand_bits(rng, (3 * H * d, Dm), sigma=Dm ** -0.5)
    Wo = rand_bits(rng, (Dm, H * d), sigma=(H * d) ** -0.5)
    return X, Wqkv, Wo


def within_one_bf16_step(got, ref):
    """|got - ref| <= one bf16 step of the reference (2^-7 relative, one sided bound)."""
    return np.all(np.abs(got - ref) <= np.maximum(np.abs(ref), 2.0 ** -120) * 2.0 ** -7)


# (B, N, H, d, Dm): several row tiles and column tiles, a ragged row tail, both head sizes
QKV_SHAPES = [(2, 256, 4, 64, 256), (1, 200, 4, 64, 320), (3, 129, 8, 64, 64), (1, 384, 2, 128, 512), (2, 77, 4, 128, 192)]


@pytest.mark.parametrize("shape", QKV_SHAPES)
def test_qkv_projection(api, shape):
    B, N, H, d, Dm = shape
    rng = np.random.default_rng(hash(shape) & 0xFFFF)
    X, Wqkv, _ = make_layer(rng, B, N, H, d, Dm)
    dev = "cuda"
    Q = torch.full((B, H, N, d), 7.0, device=dev, dtype=torch.bfloat16); K = Q.clone(); V = Q.clone()
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    api.flat_qkv_proj_fwd(bf16_tensor(X), bf16_tensor(Wqkv), Q, K, V, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    q, k, v = oracle.qkv_projection(X, Wqkv, H, d)
    for name, got, ref in (("Q", Q, q), ("K", K, k), ("V", V, v)):
        g = bf16_to_f64(got)
        r = oracle.bf16_bits_to_f64(oracle.round_to_bf16_bits(ref))
        assert within_one_bf16_step(g, r) or np.abs(g - ref).max() <= 2e-2, name
        # (tiny values: the absolute bar; everything else: one bf16 step of the rounded reference)
        assert np.abs(g - ref).max() <= np.abs(ref).max() * 2.0 ** -7
        assert np.mean(g == r) > 0.98, name + ": more than 2 % of the stored values differ from the rounded reference"


LAYER_SHAPES = [(2, 256, 4, 64, 256, False), (1, 384, 2, 128, 512, True), (2, 512, 8, 64, 512, True), (1, 1280, 4, 64, 256, False)]


@pytest.mark.parametrize("shape", LAYER_SHAPES)
def test_layer_against_oracle(api, shape):
    B, N, H, d, Dm, causal = shape
    rng = np.random.default_rng(hash(shape) & 0xFFFF)
    X, Wqkv, Wo = make_layer(rng, B, N, H, d, Dm)
    dev = "cuda"
    Q = torch.empty((B, H, N, d), device=dev, dtype=torch.bfloat16); K = torch.empty_like(Q); V = torch.empty_like(Q)
    O = torch.empty_like(Q)
    Y = torch.full((B, N, Dm), 9.0, device=dev, dtype=torch.bfloat16)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    scale = d ** -0.5
    api.flat_attn_layer_fwd(bf16_tensor(X), bf16_tensor(Wqkv), bf16_tensor(Wo), Y, Q, K, V, O, scale, causal=causal,
                            status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and api.flat_attn_last_launch_count() == 3
    ref = oracle.attention_layer(X, Wqkv, Wo, H, d, scale, causal=causal)
    # the stored intermediates
    for name, got in (("Q", Q), ("K", K), ("V", V)):
        g, r = bf16_to_f64(got), oracle.bf16_bits_to_f64(ref[name])
        assert np.abs(g - r).max() <= np.abs(r).max() * 2.0 ** -7, name
    go, ro = bf16_to_f64(O), oracle.bf16_bits_to_f64(ref["O"])
    assert np.abs(go - ro).max() <= BF16_MAX and np.abs(go - ro).mean() <= BF16_MEAN
    # the layer output
    gy, ry = bf16_to_f64(Y), ref["Y"]
    err = np.abs(gy - ry)
    assert np.all(np.isfinite(gy))
    assert err.max() <= BF16_MAX and err.mean() <= BF16_MEAN, (err.max(), err.mean())
    assert err.max() / np.abs(ry).max() <= 2 * BF16_REL_MAX, err.max() / np.abs(ry).max()


def test_output_projection_alone_with_planted_heads(api):
    """Every head of O carries its own constant; Wo picks single (head, column) features: a wrong
    head order, a transposed tile or a wrong slice of the contraction shows up exactly."""
    B, N, H, d, Dm = 2, 256, 4, 64, 256
    dev = "cuda"
    O = torch.zeros((B, H, N, d), device=dev, dtype=torch.bfloat16)
    for h in range(H):
        O[:, h] = float(h + 1)
    O[:, :, :, 5] *= 2
    O[1] *= -1
    Wo = torch.zeros((Dm, H * d), device=dev, dtype=torch.bfloat16)
    for j in range(Dm):
        Wo[j, j % (H * d)] = 1.0                                     # output j copies feature j (= head j // d, column j % d)
    Y = torch.empty((B, N, Dm), device=dev, dtype=torch.bfloat16)
    api.flat_out_proj_fwd(O, Wo, Y)
    torch.cuda.synchronize()
    want = O.permute(0, 2, 1, 3).reshape(B, N, H * d)
    assert torch.equal(Y, want)


def test_full_size_layer_sampled_rows(api):
    """The block of the headline workload (B16 H16 N4096 d64, model width 1024): one batch and a
    sample of its rows are checked against the oracle (rows are independent given K and V)."""
    B, N, H, d, Dm = 16, 4096, 16, 64, 1024
    rng = np.random.default_rng(2107)
    X, Wqkv, Wo = make_layer(rng, B, N, H, d, Dm)
    dev = "cuda"
    Q = torch.empty((B, H, N, d), device=dev, dtype=torch.bfloat16); K = torch.empty_like(Q); V = torch.empty_like(Q)
    O = torch.empty_like(Q)
    Y = torch.empty((B, N, Dm), device=dev, dtype=torch.bfloat16)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    scale = d ** -0.5
    api.flat_attn_layer_fwd(bf16_tensor(X), bf16_tensor(Wqkv), bf16_tensor(Wo), Y, Q, K, V, O, scale, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    b = 11
    q, k, v = oracle.qkv_projection(X[b:b + 1], Wqkv, H, d)
    Qb, Kb, Vb = (oracle.round_to_bf16_bits(t) for t in (q, k, v))
    for name, got, r in (("Q", Q, Qb), ("K", K, Kb), ("V", V, Vb)):
        g, rr = bf16_to_f64(got[b:b + 1]), oracle.bf16_bits_to_f64(r)
        assert np.abs(g - rr).max() <= np.abs(rr).max() * 2.0 ** -7, name
        assert np.mean(g == rr) > 0.98, name
    toks = np.array([0, 1, 127, 128, 2047, 2048, 3000, 4095], dtype=np.int64)
    rows = np.concatenate([h * N + toks for h in range(H)])             # flat row ids (b*H + h)*N + i with b = 0
    o = oracle.attention(Qb, Kb, Vb, scale, rows=rows)["O"].reshape(H, len(toks), d)
    ob = oracle.bf16_bits_to_f64(oracle.round_to_bf16_bits(o))
    go = bf16_to_f64(O[b][:, torch.from_numpy(toks).to(dev)])
    assert np.abs(go - ob).max() <= BF16_MAX and np.abs(go - ob).mean() <= BF16_MEAN
    y = oracle.out_projection(ob[None], Wo)[0]                        # [len(toks), Dm]
    gy = bf16_to_f64(Y[b][torch.from_numpy(toks).to(dev)])
    err = np.abs(gy - y)
    assert err.max() <= BF16_MAX and err.mean() <= BF16_MEAN
    assert err.max() / np.abs(y).max() <= 2 * BF16_REL_MAX


@pytest.mark.parametrize("shape", [(300, 64, 256), (1024, 256, 1024), (77, 192, 512)])
def test_fully_connected(api, shape):
    M, K, Nout = shape
    rng = np.random.default_rng(M + K)
    X = rand_bits(rng, (M, K)); W = rand_bits(rng, (Nout, K), sigma=K ** -0.5)
    Y = torch.full((M, Nout), 5.0, device="cuda", dtype=torch.bfloat16)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.flat_fc_fwd(bf16_tensor(X), bf16_tensor(W), Y, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = oracle.fully_connected(X, W)
    g = bf16_to_f64(Y)
    assert np.abs(g - ref).max() <= np.abs(ref).max() * 2.0 ** -7
    assert np.mean(g == oracle.bf16_bits_to_f64(oracle.round_to_bf16_bits(ref))) > 0.98


def test_layer_and_packed_calls_in_a_cuda_graph_on_two_streams(api):
    """The widened entry points also only enqueue work: a layer call and a packed variable-length call are
    captured on two streams of one graph (they run concurrently) and the replays reproduce the direct launches
    bit for bit."""
    rng = np.random.default_rng(404)
    B, N, H, d, Dm = 2, 512, 8, 64, 512
    X, Wqkv, Wo = (bf16_tensor(t) for t in make_layer(rng, B, N, H, d, Dm))
    mk = lambda: torch.empty((B, H, N, d), device="cuda", dtype=torch.bfloat16)
    Q, K, V, O = mk(), mk(), mk(), mk()
    Y_direct = torch.empty((B, N, Dm), device="cuda", dtype=torch.bfloat16)
    api.flat_attn_layer_fwd(X, Wqkv, Wo, Y_direct, Q, K, V, O, d ** -0.5, causal=True)
    lens = np.array([300, 1, 700, 129, 64], dtype=np.int64)
    cu = torch.from_numpy(np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)).cuda()
    Qp, Kp, Vp = (bf16_tensor(rand_bits(rng, (int(lens.sum()), H, d))) for _ in range(3))
    Op_direct = torch.empty_like(Qp)
    api.flat_attn_varlen_fwd(Qp, Kp, Vp, Op_direct, cu, cu, int(lens.max()), d ** -0.5)
    torch.cuda.synchronize()
    Y, Op = torch.zeros_like(Y_direct), torch.zeros_like(Op_direct)
    g = torch.cuda.CUDAGraph()
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    s1.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s1):
        with torch.cuda.graph(g, stream=s1):
            s2.wait_stream(s1)
            api.flat_attn_layer_fwd(X, Wqkv, Wo, Y, Q, K, V, O, d ** -0.5, causal=True, stream=s1)
            with torch.cuda.stream(s2):
                api.flat_attn_varlen_fwd(Qp, Kp, Vp, Op, cu, cu, int(lens.max()), d ** -0.5, stream=s2)
            s1.wait_stream(s2)
    torch.cuda.current_stream().wait_stream(s1)
    for _ in range(3):
        Y.zero_(); Op.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(Y.view(torch.int16), Y_direct.view(torch.int16))
        assert torch.equal(Op.view(torch.int16), Op_direct.view(torch.int16))
