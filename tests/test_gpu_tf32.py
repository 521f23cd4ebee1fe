"""The fp32 tensor-core kernel (split-tf32 products, d = 64) against the oracle: shapes that span one key step,
two, odd and even counts and ragged tails; the masks; the row log-sum-exp; rows whose weight sits on one or two
keys; and the same inputs through the FFMA kernel, which must agree with it far inside the fp32 bar."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2107_06419_b200 import inputs
from helpers import check_f32

pytestmark = pytest.mark.gpu

D = 64


@pytest.fixture(scope="module")
def api():
    from paper_2107_06419_b200 import api as _api
    return _api


def run(api, Q, K, V, scale, variant, vl=None, causal=False, want_lse=False):
    Qt, Kt, Vt = (torch.from_numpy(np.ascontiguousarray(x)).cuda() for x in (Q, K, V))
    O = torch.full(Qt.shape, float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    lse = torch.full(Qt.shape[:3], float("nan"), dtype=torch.float32, device="cuda") if want_lse else None
    api.flat_attn_fwd_ex(Qt, Kt, Vt, O, scale, k_valid_len=None if vl is None else torch.from_numpy(vl).cuda(),
                         status=status, variant=variant, causal=causal, lse=lse)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return O.double().cpu().numpy(), None if lse is None else lse.double().cpu().numpy()


def normal(rng, *shape):
    return rng.standard_normal(shape).astype(np.float32)


# (B, H, Nq, Nk): one step, one step ragged, two steps, three, an odd and an even count with ragged tails, several query tiles
SHAPES = [(1, 1, 128, 64), (1, 2, 128, 40), (1, 2, 128, 128), (2, 1, 100, 192), (1, 2, 200, 333), (2, 2, 384, 1000),
          (1, 1, 512, 2048), (1, 3, 1, 77), (1, 1, 129, 4160)]


@pytest.mark.parametrize("shape", SHAPES)
def test_dense(api, shape):
    B, H, Nq, Nk = shape
    rng = np.random.default_rng(Nq * 7 + Nk)
    Q, K, V = normal(rng, B, H, Nq, D), normal(rng, B, H, Nk, D), normal(rng, B, H, Nk, D)
    scale = 1 / math.sqrt(D)
    ref = oracle.attention(Q, K, V, scale, want_lse=True)
    O, lse = run(api, Q, K, V, scale, api.FLAT_VARIANT_TF32, want_lse=True)
    assert api.flat_attn_last_variant() == api.FLAT_VARIANT_TF32
    mx = check_f32(O, ref["O"], "tf32 %s" % (shape,))
    assert mx < 2e-5                                   # (iid rows: far inside the bar)
    assert np.max(np.abs(lse - ref["LSE"])) < 2e-5
    # AUTO takes the same kernel for fp32, d = 64
    O2, _ = run(api, Q, K, V, scale, api.FLAT_VARIANT_AUTO)
    assert api.flat_attn_last_variant() == api.FLAT_VARIANT_TF32
    assert np.array_equal(O, O2)
    # and the FFMA kernel agrees
    O3, _ = run(api, Q, K, V, scale, api.FLAT_VARIANT_SIMT)
    assert np.max(np.abs(O3 - O)) < 2e-5


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("shape", [(2, 3, 130, 777), (2, 2, 384, 384), (2, 1, 64, 300), (2, 2, 300, 64)])
def test_masks(api, shape, causal):
    B, H, Nq, Nk = shape
    rng = np.random.default_rng(Nq + 3 * Nk + causal)
    Q, K, V = normal(rng, B, H, Nq, D), normal(rng, B, H, Nk, D), normal(rng, B, H, Nk, D)
    vl = np.array([max(1, Nk * 2 // 3), 0], dtype=np.int32)    # (the second batch sees no key at all)
    ref = oracle.attention(Q, K, V, 0.2, valid_len=vl, causal=causal, want_lse=True)
    O, lse = run(api, Q, K, V, 0.2, api.FLAT_VARIANT_TF32, vl=vl, causal=causal, want_lse=True)
    check_f32(O, ref["O"], "tf32 masks %s causal=%d" % (shape, causal))
    assert np.all(O[1] == 0.0)
    fin = np.isfinite(ref["LSE"])
    assert np.array_equal(np.isneginf(lse), np.isneginf(ref["LSE"]))     # rows without a key: -inf on both sides
    assert np.max(np.abs(lse[fin] - ref["LSE"][fin])) < 2e-5


@pytest.mark.parametrize("scale", [-0.3, 0.0, 2.0])
def test_scales(api, scale):
    rng = np.random.default_rng(17)
    Q, K, V = normal(rng, 1, 2, 150, D), normal(rng, 1, 2, 260, D), normal(rng, 1, 2, 260, D)
    ref = oracle.attention(Q, K, V, scale)["O"]
    O, _ = run(api, Q, K, V, scale, api.FLAT_VARIANT_TF32)
    check_f32(O, ref, "tf32 scale %g" % scale)


def test_planted_and_tied_keys(api):
    """Rows whose weight sits on one planted key, and rows split evenly between two identical keys with different
    values: a dropped or misplaced tile moves the output by O(1); a weight rounded to tf32 without its remainder
    would move the tied rows by about 1e-3 |v|."""
    rng = np.random.default_rng(23)
    Nq, Nk = 256, 1024
    K = normal(rng, 1, 1, Nk, D)
    V = normal(rng, 1, 1, Nk, D) * 4
    planted = rng.integers(0, Nk, size=Nq)
    Q = (K[0, 0, planted] * 1.5 + 0.05 * normal(rng, Nq, D))[None, None].astype(np.float32)
    ref = oracle.attention(Q, K, V, 1.0)["O"]
    assert np.median(np.abs(ref[0, 0] - V[0, 0, planted]).max(axis=1)) < 1e-3
    O, _ = run(api, Q, K, V, 1.0, api.FLAT_VARIANT_TF32)
    check_f32(O, ref, "tf32 planted")
    K2 = K.copy()
    K2[0, 0, 900] = K2[0, 0, 37]                        # two keys with the same logits for every query
    Q2 = (K2[0, 0, 37] * 1.2 + 0.05 * normal(rng, Nq, D))[None, None].astype(np.float32)
    ref2 = oracle.attention(Q2, K2, V, 1.0)["O"]
    assert np.median(np.abs(ref2[0, 0] - 0.5 * (V[0, 0, 37] + V[0, 0, 900])).max(axis=1)) < 1e-2
    O2, _ = run(api, Q2, K2, V, 1.0, api.FLAT_VARIANT_TF32)
    check_f32(O2, ref2, "tf32 tied keys")


def test_values_that_need_every_mantissa_bit(api):
    """Operands whose low mantissa bits carry the signal: K = c + tiny differences.  A logit computed from the tf32
    heads alone would lose the differences (and the ranking of the keys with them)."""
    rng = np.random.default_rng(29)
    Nq, Nk = 128, 256
    base = normal(rng, 1, D)
    K = (base + 1e-3 * normal(rng, Nk, D)).astype(np.float32)[None, None]
    Q = (40.0 * normal(rng, Nq, D)).astype(np.float32)[None, None]
    V = normal(rng, 1, 1, Nk, D)
    ref = oracle.attention(Q, K, V, 1.0)["O"]
    O, _ = run(api, Q, K, V, 1.0, api.FLAT_VARIANT_TF32)
    check_f32(O, ref, "tf32 low bits")
    # sanity of the case itself: with K rounded to tf32 the oracle's answer moves by far more than the bar
    Kt = (K.view(np.uint32) & np.uint32(0xffffe000)).view(np.float32)
    assert np.max(np.abs(oracle.attention(Q, Kt, V, 1.0)["O"] - ref)) > 1e-2


def test_refusals(api):
    Q = torch.zeros(1, 1, 128, 128, device="cuda")
    O = torch.empty_like(Q)
    with pytest.raises(api.FlatAttnError):               # d = 128
        api.flat_attn_fwd_ex(Q, Q, Q, O, 1.0, variant=api.FLAT_VARIANT_TF32)
    Qb = torch.zeros(1, 1, 128, 64, device="cuda", dtype=torch.bfloat16)
    with pytest.raises(api.FlatAttnError):               # bf16 tensors
        api.flat_attn_fwd_ex(Qb, Qb, Qb, torch.empty_like(Qb), 1.0, variant=api.FLAT_VARIANT_TF32)
    Qf = torch.zeros(1, 1, 128, 64, device="cuda")
    bias = torch.zeros(1, 1, 128, 128, device="cuda")
    with pytest.raises(api.FlatAttnError):               # a bias goes to the FFMA kernel, not here
        api.flat_attn_fwd_ex(Qf, Qf, Qf, torch.empty_like(Qf), 1.0, variant=api.FLAT_VARIANT_TF32, bias=bias)
    Of = torch.empty_like(Qf)
    api.flat_attn_fwd_ex(Qf, Qf, Qf, Of, 1.0, bias=bias)    # AUTO with a bias: the FFMA kernel
    torch.cuda.synchronize()
    assert api.flat_attn_last_variant() == api.FLAT_VARIANT_SIMT


def test_full_size_sampled_rows_c3(api):
    """c3 widened to fp32, in the launch configuration the bench's fp32 line times."""
    w = inputs.WORKLOADS["c3_16k"]
    Qb, Kb, Vb = inputs.make_qkv_bf16(w)
    rows = inputs.sample_rows(w, 8)
    ref = oracle.attention(Qb, Kb, Vb, w.scale, rows=rows)["O"]
    f = lambda bits: torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).cuda().float()
    Q, K, V = f(Qb), f(Kb), f(Vb)
    O = torch.full(Q.shape, float("nan"), device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.flat_attn_fwd_ex(Q, K, V, O, w.scale, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and api.flat_attn_last_variant() == api.FLAT_VARIANT_TF32
    got = O.view(-1, w.d)[torch.from_numpy(rows).cuda()].double().cpu().numpy()
    check_f32(got, ref, "c3 fp32")
    assert bool(torch.isfinite(O).all())
