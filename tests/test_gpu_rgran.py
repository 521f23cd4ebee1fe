"""GPU parity of the literal row-granularity kernel (whole logit rows on chip, two-pass softmax)
against the oracle, through the C ABI with variant = FLAT_VARIANT_RGRAN."""
import numpy as np
import pytest
import torch

import oracle
from helpers import bf16_tensor, bf16_to_f64, check_bf16, rand_bits

pytestmark = pytest.mark.gpu

# B, H, Nq, Nk (<= 512), masked, causal
SHAPES = [
    (1, 12, 512, 512, False, False),     # the shortest workload of the paper's set
    (2, 3, 300, 517 - 5, True, False),   # ragged rows and keys, key-padding mask
    (1, 2, 129, 1, False, False),        # one key
    (2, 2, 128, 128, False, True),       # square causal
    (1, 2, 77, 400, True, True),         # causal with more keys than queries, masked
    (1, 1, 400, 70, False, True),        # fewer keys than queries: the first rows see no key
    (3, 2, 640, 384, True, False),       # three key tiles, five row tiles
]


@pytest.fixture(scope="module")
def api():
    from paper_2107_06419_b200 import api as _api
    return _api


def run(api, Qb, Kb, Vb, scale, vl=None, causal=False):
    Q, K, V = bf16_tensor(Qb), bf16_tensor(Kb), bf16_tensor(Vb)
    O = torch.full(Q.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    vlt = None if vl is None else torch.from_numpy(vl).cuda()
    api.flat_attn_fwd_ex(Q, K, V, O, scale, k_valid_len=vlt, status=status, variant=api.FLAT_VARIANT_RGRAN, causal=causal)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return bf16_to_f64(O)


@pytest.mark.parametrize("shape", SHAPES)
def test_rgran_against_oracle(api, shape):
    B, H, Nq, Nk, masked, causal = shape
    d = 64
    rng = np.random.default_rng(Nq * 7 + Nk)
    Qb, Kb, Vb = rand_bits(rng, (B, H, Nq, d)), rand_bits(rng, (B, H, Nk, d)), rand_bits(rng, (B, H, Nk, d))
    vl = None
    if masked:
        vl = rng.integers(0, Nk + 1, size=B).astype(np.int32)
        vl[0] = Nk // 2 + 1
    scale = d ** -0.5
    ref = oracle.attention(Qb, Kb, Vb, scale, valid_len=vl, causal=causal)["O"]
    check_bf16(run(api, Qb, Kb, Vb, scale, vl=vl, causal=causal), ref, "rgran %s" % (shape,))


def test_rgran_peaked_and_negative_scale(api):
    """Exact two-pass softmax: logits of hundreds (no overflow), a negative scale (the maximum is taken
    after scaling), and scale 0 (uniform weights)."""
    B, H, Nq, Nk, d = 1, 2, 256, 512, 64
    rng = np.random.default_rng(9)
    Qb, Kb, Vb = rand_bits(rng, (B, H, Nq, d), 3.0), rand_bits(rng, (B, H, Nk, d), 3.0), rand_bits(rng, (B, H, Nk, d), 0.25)
    for scale in (2.0, -1.5, 0.0):
        ref = oracle.attention(Qb, Kb, Vb, scale)["O"]
        check_bf16(run(api, Qb, Kb, Vb, scale), ref, "rgran scale %g" % scale)


def test_rgran_rejects_what_it_cannot_hold(api):
    Q = torch.zeros((1, 1, 128, 64), dtype=torch.bfloat16, device="cuda")
    K = torch.zeros((1, 1, 513, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(api.FlatAttnError) as e:
        api.flat_attn_fwd_ex(Q, K, K.clone(), Q.clone(), 1.0, variant=api.FLAT_VARIANT_RGRAN)
    assert e.value.code == 3
