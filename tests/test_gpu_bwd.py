"""Backward pass and the forward's log-sum-exp output: CUDA path vs CPU oracle, element by element on
the same seeded inputs, through the C ABI.  Bars (stated before the kernels ran): per gradient tensor
max |dg| <= 2e-2 max |g_ref| and mean |dg| <= 1e-2 mean |g_ref|; lse within 1e-3."""
import numpy as np
import pytest
import torch

import oracle
from paper_2107_06419_b200 import inputs
from helpers import bf16_tensor, bf16_to_f64, check_bf16, rand_bits

pytestmark = pytest.mark.gpu

GRAD_MAX_REL, GRAD_MEAN_REL, LSE_MAX = 2e-2, 1e-2, 1e-3


@pytest.fixture(scope="module")
def api():
    from paper_2107_06419_b200 import api as _api
    return _api


def check_grad(got, ref, what):
    assert np.all(np.isfinite(got)), what + ": non-finite gradient"
    err = np.abs(got - ref)
    mx, mean = float(err.max()), float(err.mean())
    ref_max, ref_mean = float(np.abs(ref).max()), float(np.abs(ref).mean())
    assert mx <= GRAD_MAX_REL * max(ref_max, 1e-30), "%s: max |dg| = %.3e against max |g| = %.3e" % (what, mx, ref_max)
    assert mean <= GRAD_MEAN_REL * max(ref_mean, 1e-30), "%s: mean |dg| = %.3e against mean |g| = %.3e" % (what, mean, ref_mean)
    return mx / max(ref_max, 1e-30), mean / max(ref_mean, 1e-30)


def check_lse(got, ref, what):
    got = got.astype(np.float64)
    empty = np.isneginf(ref)
    assert np.array_equal(np.isneginf(got), empty), what + ": rows without keys"
    assert np.all(np.isfinite(got[~empty])), what + ": non-finite lse"
    if (~empty).any():
        assert np.abs(got[~empty] - ref[~empty]).max() <= LSE_MAX, "%s: max |dlse| = %.3e" % (what, np.abs(got[~empty] - ref[~empty]).max())


def run_fwd_bwd(api, Qb, Kb, Vb, dOb, scale, vl=None, causal=False, variant=0):
    Q, K, V, dO = bf16_tensor(Qb), bf16_tensor(Kb), bf16_tensor(Vb), bf16_tensor(dOb)
    B, H, Nq, d = Q.shape
    O = torch.full(Q.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((B, H, Nq), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    vlt = None if vl is None else torch.from_numpy(vl).cuda()
    api.flat_attn_fwd_ex(Q, K, V, O, scale, k_valid_len=vlt, status=status, variant=variant, causal=causal, lse=lse)
    dQ = torch.full(Q.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    dK = torch.full(K.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    dV = torch.full(K.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    delta = torch.full((B, H, Nq), float("nan"), dtype=torch.float32, device="cuda")
    api.flat_attn_bwd_ex(Q, K, V, O, dO, lse, dQ, dK, dV, delta, scale, k_valid_len=vlt, status=status, causal=causal)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, "device status 0x%x" % int(status.item())
    assert api.flat_attn_last_launch_count() == 2
    return bf16_to_f64(O), lse.cpu().numpy(), bf16_to_f64(dQ), bf16_to_f64(dK), bf16_to_f64(dV)


SHAPES = [
    # B, H, Nq, Nk, d -- one tile, several tiles, ragged tails on both sides, one key, one query
    (1, 1, 128, 128, 64),
    (2, 3, 300, 517, 64),
    (1, 2, 129, 1, 64),
    (1, 1, 1, 700, 64),
    (1, 2, 700, 900, 64),
    (2, 2, 200, 333, 128),
    (1, 1, 384, 256, 128),
]


@pytest.mark.parametrize("shape", SHAPES)
def test_backward_small(api, shape):
    B, H, Nq, Nk, d = shape
    rng = np.random.default_rng(sum(shape))
    Qb, Kb, Vb, dOb = (rand_bits(rng, s) for s in ((B, H, Nq, d), (B, H, Nk, d), (B, H, Nk, d), (B, H, Nq, d)))
    scale = d ** -0.5
    O, lse, dQ, dK, dV = run_fwd_bwd(api, Qb, Kb, Vb, dOb, scale)
    ref = oracle.attention_bwd(Qb, Kb, Vb, dOb, scale)
    check_bf16(O, oracle.attention(Qb, Kb, Vb, scale)["O"], "O %s" % (shape,))
    check_lse(lse, ref["LSE"], "lse %s" % (shape,))
    if Nk > 1:                                           # (one key: dQ = dK = 0 exactly, nothing to scale the bar by)
        check_grad(dQ, ref["dQ"], "dQ %s" % (shape,))
        check_grad(dK, ref["dK"], "dK %s" % (shape,))
    else:
        assert np.abs(dQ).max() <= 1e-2 and np.abs(dK).max() <= 1e-2
    check_grad(dV, ref["dV"], "dV %s" % (shape,))


@pytest.mark.parametrize("shape", [(2, 2, 300, 517, 64), (1, 2, 517, 300, 64), (1, 2, 256, 256, 128), (2, 1, 130, 400, 128)])
def test_backward_causal(api, shape):
    B, H, Nq, Nk, d = shape
    rng = np.random.default_rng(7 + sum(shape))
    Qb, Kb, Vb, dOb = (rand_bits(rng, s) for s in ((B, H, Nq, d), (B, H, Nk, d), (B, H, Nk, d), (B, H, Nq, d)))
    scale = d ** -0.5
    O, lse, dQ, dK, dV = run_fwd_bwd(api, Qb, Kb, Vb, dOb, scale, causal=True)
    ref = oracle.attention_bwd(Qb, Kb, Vb, dOb, scale, causal=True)
    check_lse(lse, ref["LSE"], "lse causal %s" % (shape,))
    for name, got in (("dQ", dQ), ("dK", dK), ("dV", dV)):
        check_grad(got, ref[name], "%s causal %s" % (name, shape))
    if Nq > Nk:                                          # the first Nq - Nk queries see no key
        assert np.all(dQ[:, :, :Nq - Nk] == 0)


@pytest.mark.parametrize("d", [64, 128])
def test_backward_key_padding(api, d):
    B, H, Nq, Nk = 3, 2, 260, 600
    rng = np.random.default_rng(d)
    Qb, Kb, Vb, dOb = (rand_bits(rng, s) for s in ((B, H, Nq, d), (B, H, Nk, d), (B, H, Nk, d), (B, H, Nq, d)))
    vl = np.array([600, 257, 0], dtype=np.int32)         # all keys, a ragged cut inside a tile, none
    scale = d ** -0.5
    for causal in (False, True):
        O, lse, dQ, dK, dV = run_fwd_bwd(api, Qb, Kb, Vb, dOb, scale, vl=vl, causal=causal)
        ref = oracle.attention_bwd(Qb, Kb, Vb, dOb, scale, valid_len=vl, causal=causal)
        check_lse(lse, ref["LSE"], "lse masked")
        for name, got in (("dQ", dQ), ("dK", dK), ("dV", dV)):
            check_grad(got[:2], ref[name][:2], "%s masked d=%d causal=%d" % (name, d, causal))
            assert np.all(got[2] == 0), name + ": a batch without keys has zero gradients"
        assert np.all(dK[1, :, 257:] == 0) and np.all(dV[1, :, 257:] == 0)


@pytest.mark.parametrize("variant,shape", [(1, (1, 2, 200, 333, 32)), (1, (1, 1, 150, 150, 64)), (3, (1, 2, 300, 517, 64)),
                                           (4, (2, 2, 300, 517, 64)), (5, (1, 2, 600, 1300, 64)), (3, (1, 2, 300, 517, 128))],
                         ids=["simt32", "simt64", "tc2", "tc2single", "tc3", "tc2_d128"])
def test_forward_lse_of_every_kernel_that_writes_it(api, variant, shape):
    B, H, Nq, Nk, d = shape
    rng = np.random.default_rng(100 + variant + d)
    Qb, Kb, Vb = (rand_bits(rng, s) for s in ((B, H, Nq, d), (B, H, Nk, d), (B, H, Nk, d)))
    vl = np.array([Nk - 77] + [Nk] * (B - 1), dtype=np.int32)
    for causal in (False, True):
        Q, K, V = bf16_tensor(Qb), bf16_tensor(Kb), bf16_tensor(Vb)
        O = torch.empty_like(Q)
        lse = torch.full((B, H, Nq), float("nan"), dtype=torch.float32, device="cuda")
        api.flat_attn_fwd_ex(Q, K, V, O, d ** -0.5, k_valid_len=torch.from_numpy(vl).cuda(), variant=variant,
                             causal=causal, lse=lse)
        torch.cuda.synchronize()
        ref = oracle.attention(Qb, Kb, Vb, d ** -0.5, valid_len=vl, causal=causal, want_lse=True)
        check_bf16(bf16_to_f64(O), ref["O"], "O v%d" % variant)
        check_lse(lse.cpu().numpy(), ref["LSE"], "lse v%d causal=%d" % (variant, causal))


def test_lse_is_refused_where_no_kernel_writes_it(api):
    q = torch.zeros(1, 1, 128, 64, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(1, 1, 128, dtype=torch.float32, device="cuda")
    for variant in (2, 6):
        with pytest.raises(api.FlatAttnError) as e:
            api.flat_attn_fwd_ex(q, q, q, torch.empty_like(q), 1.0, variant=variant, lse=lse)
        assert e.value.code == 3


def test_backward_large_logits_and_reproducible(api):
    """Logits of tens (sigma 3 inputs): the weights are rebuilt from lse alone, so a wrong or stale lse
    would overflow or vanish here; and two runs give identical bits (no atomics)."""
    rng = np.random.default_rng(77)
    B, H, Nq, Nk, d = 1, 2, 384, 640, 64
    Qb, Kb, Vb, dOb = (rand_bits(rng, s, sigma=sg) for s, sg in (((B, H, Nq, d), 3.0), ((B, H, Nk, d), 3.0),
                                                                  ((B, H, Nk, d), 1.0), ((B, H, Nq, d), 1.0)))
    r1 = run_fwd_bwd(api, Qb, Kb, Vb, dOb, 0.125)
    r2 = run_fwd_bwd(api, Qb, Kb, Vb, dOb, 0.125)
    assert all(np.array_equal(a, b) for a, b in zip(r1, r2))
    ref = oracle.attention_bwd(Qb, Kb, Vb, dOb, 0.125)
    check_lse(r1[1], ref["LSE"], "lse sigma 3")
    for name, got in zip(("dQ", "dK", "dV"), r1[2:]):
        check_grad(got, ref[name], name + " sigma 3")


def test_backward_argument_errors(api):
    q = torch.zeros(1, 1, 128, 32, dtype=torch.bfloat16, device="cuda")
    f = torch.zeros(1, 1, 128, dtype=torch.float32, device="cuda")
    with pytest.raises(api.FlatAttnError) as e:
        api.flat_attn_bwd(q, q, q, q, q, f, torch.empty_like(q), torch.empty_like(q), torch.empty_like(q), f.clone(), 1.0)
    assert e.value.code == 3                             # d = 32: no backward kernel, no fallback


def test_backward_c2_sampled_heads(api):
    """Full-size c2: all of dQ, dK, dV of a few (batch, head) pairs against the oracle."""
    w = inputs.WORKLOADS["c2_bert_large_4k"]
    Qb, Kb, Vb = inputs.make_qkv_bf16(w)
    n = w.B * w.H * w.Nq * w.d
    dOb = inputs.f32_to_bf16_bits(inputs.normal_f32(inputs.DEFAULT_SEED, 5, 0, n)).reshape(Qb.shape)
    O, lse, dQ, dK, dV = run_fwd_bwd(api, Qb, Kb, Vb, dOb, w.scale)
    heads = np.array([0, 37, 130, 255], dtype=np.int64)
    ref = oracle.attention_bwd(Qb, Kb, Vb, dOb, w.scale, heads=heads)
    pick = lambda x: x.reshape(w.B * w.H, -1, w.d)[heads]
    check_lse(lse.reshape(w.B * w.H, -1)[heads], ref["LSE"], "lse c2")
    for name, got in (("dQ", dQ), ("dK", dK), ("dV", dV)):
        rel = check_grad(pick(got), ref[name], name + " c2")
        print(name, "c2: max/max %.2e mean/mean %.2e" % rel)
