"""The block's normalisation layer: CUDA kernel against the oracle, element by element."""
import numpy as np
import pytest
import torch

import oracle
from helpers import bf16_tensor, bf16_to_f64, rand_bits

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def api():
    from paper_2107_06419_b200 import api as _api
    return _api


@pytest.mark.parametrize("M,D", [(1, 8), (37, 64), (300, 768), (129, 1024), (17, 1032), (5, 4096), (3, 8192), (1000, 256)])
@pytest.mark.parametrize("res", [False, True])
def test_layernorm_matches_oracle(api, M, D, res):
    rng = np.random.default_rng(M + D + res)
    Xb = rand_bits(rng, (M, D), sigma=2.0)
    Rb = rand_bits(rng, (M, D)) if res else None
    gb, bb = rand_bits(rng, (D,)), rand_bits(rng, (D,))
    X = bf16_tensor(Xb)
    Y = torch.full(X.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    api.flat_layernorm_fwd(X, bf16_tensor(gb), bf16_tensor(bb), Y, eps=1e-5, residual=None if Rb is None else bf16_tensor(Rb))
    torch.cuda.synchronize()
    ref = oracle.layer_norm(Xb, gb, bb, 1e-5, residual=Rb)
    # |y| reaches a few units, so the bf16 rounding of the output alone is up to 2^-8 * |y|
    err = np.abs(bf16_to_f64(Y) - ref)
    assert np.all(np.isfinite(bf16_to_f64(Y)))
    assert np.all(err <= 2.0 ** -8 * np.abs(ref) + 1e-3), float(err.max())
    # (on average the rounding of the output costs a quarter of a bf16 step of |y|)
    assert err.mean() <= 2.0 ** -9 * np.abs(ref).mean() + 1e-4


def test_layernorm_in_place_constant_rows_and_padding(api):
    rng = np.random.default_rng(9)
    M, D = 64, 512
    Xb = rand_bits(rng, (M, D))
    Xb[3] = Xb[3, 0]                                     # a constant row: variance 0 -> y = beta
    gb, bb = rand_bits(rng, (D,)), rand_bits(rng, (D,))
    buf = torch.full((M + 2, D), 7.0, dtype=torch.bfloat16, device="cuda")
    buf[1:M + 1] = bf16_tensor(Xb)
    X = buf[1:M + 1]
    api.flat_layernorm_fwd(X, bf16_tensor(gb), bf16_tensor(bb), X, eps=1e-5)      # Y aliases X
    torch.cuda.synchronize()
    assert torch.all(buf[0] == 7.0) and torch.all(buf[M + 1] == 7.0)
    ref = oracle.layer_norm(Xb, gb, bb, 1e-5)
    err = np.abs(bf16_to_f64(X) - ref)
    assert np.all(err <= 2.0 ** -8 * np.abs(ref) + 1e-3), float(err.max())
    assert np.array_equal(bf16_to_f64(X)[3], oracle.bf16_bits_to_f64(bb))
