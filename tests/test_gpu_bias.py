"""Additive bias of the scaled logits: CUDA path (two-tile tensor-core kernel and FFMA kernel) against
the oracle, element by element, on ragged shapes at both head sizes, with every broadcast form, both
storage types, the masks, and -inf entries."""
import numpy as np
import pytest
import torch

import oracle
from paper_2107_06419_b200 import inputs
from helpers import bf16_tensor, bf16_to_f64, check_bf16, check_f32, rand_bits

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def api():
    from paper_2107_06419_b200 import api as _api
    return _api


def run(api, Qb, Kb, Vb, scale, bias, vl=None, causal=False, variant=0, want_lse=False):
    Q, K, V = bf16_tensor(Qb), bf16_tensor(Kb), bf16_tensor(Vb)
    O = torch.full(Q.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    lse = torch.full(Q.shape[:3], float("nan"), dtype=torch.float32, device="cuda") if want_lse else None
    bt = bf16_tensor(bias) if bias.dtype == np.uint16 else torch.from_numpy(bias).cuda()
    api.flat_attn_fwd_ex(Q, K, V, O, scale, k_valid_len=None if vl is None else torch.from_numpy(vl).cuda(),
                         status=status, variant=variant, causal=causal, bias=bt, lse=lse)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return bf16_to_f64(O), (None if lse is None else lse.cpu().numpy())


@pytest.mark.parametrize("shape", [(2, 3, 300, 517, 64), (1, 2, 256, 384, 64), (2, 2, 200, 333, 128), (1, 2, 128, 1024, 128)])
@pytest.mark.parametrize("bshape", ["full", "per_head", "per_batch", "one"])
def test_bias_tc2(api, shape, bshape):
    B, H, Nq, Nk, d = shape
    rng = np.random.default_rng(sum(shape) + len(bshape))
    Qb, Kb, Vb = (rand_bits(rng, s) for s in ((B, H, Nq, d), (B, H, Nk, d), (B, H, Nk, d)))
    bs = {"full": (B, H), "per_head": (1, H), "per_batch": (B, 1), "one": (1, 1)}[bshape]
    bias = rand_bits(rng, bs + (Nq, Nk), sigma=2.0)      # bf16; of the size of the logits themselves
    got, lse = run(api, Qb, Kb, Vb, d ** -0.5, bias, want_lse=True)
    assert api.flat_attn_last_variant() == api.FLAT_VARIANT_TC2
    ref = oracle.attention(Qb, Kb, Vb, d ** -0.5, bias=bias, want_lse=True)
    check_bf16(got, ref["O"], "bias %s %s" % (shape, bshape))
    assert np.abs(lse - ref["LSE"]).max() <= 1e-3
    # and the bias matters: without it the answer is far away
    assert np.abs(ref["O"] - oracle.attention(Qb, Kb, Vb, d ** -0.5)["O"]).max() > 0.1


def test_bias_f32_storage_masks_and_minus_infinity(api):
    B, H, Nq, Nk, d = 2, 2, 260, 520, 64
    rng = np.random.default_rng(3)
    Qb, Kb, Vb = (rand_bits(rng, s) for s in ((B, H, Nq, d), (B, H, Nk, d), (B, H, Nk, d)))
    bias = rng.standard_normal((1, H, Nq, Nk)).astype(np.float32)
    bias[0, 0, :, 100:300] = -np.inf                     # a block of keys switched off for head 0
    bias[0, 1, 7, :] = -np.inf                           # a whole row switched off
    bias[0, 1, 200, :519] = -np.inf                      # a row with a single live pair, in the last tile
    vl = np.array([520, 391], dtype=np.int32)
    for causal in (False, True):
        got, lse = run(api, Qb, Kb, Vb, 0.125, bias, vl=vl, causal=causal, want_lse=True)
        ref = oracle.attention(Qb, Kb, Vb, 0.125, bias=bias, valid_len=vl, causal=causal, want_lse=True)
        check_bf16(got, ref["O"], "bias f32 causal=%d" % causal)
        assert np.all(got[:, 1, 7] == 0)
        dead = np.isneginf(ref["LSE"])
        assert np.array_equal(np.isneginf(lse), dead) and np.abs(lse[~dead] - ref["LSE"][~dead]).max() <= 1e-3


@pytest.mark.parametrize("bshape", ["full", "per_head", "per_batch", "one"])
@pytest.mark.parametrize("causal", [False, True])
def test_bias_bf16_tiles_staged_in_shared_memory(api, bshape, causal):
    """d = 64 with a bf16 bias whose rows are 16-byte aligned: the tiles come through shared memory, the batches of a
    head run next to each other when the bias is shared by the batches (a different order of the CTAs, the same
    results), ragged last key tile, a key-padding mask, -inf entries."""
    B, H, Nq, Nk, d = 3, 2, 300, 520, 64
    rng = np.random.default_rng(11 + len(bshape) + causal)
    Qb, Kb, Vb = (rand_bits(rng, s) for s in ((B, H, Nq, d), (B, H, Nk, d), (B, H, Nk, d)))
    bs = {"full": (B, H), "per_head": (1, H), "per_batch": (B, 1), "one": (1, 1)}[bshape]
    bf = (rng.standard_normal(bs + (Nq, Nk)) * 2.0).astype(np.float32)
    bf[0, 0, :, 130:260] = -np.inf                       # a block of keys switched off
    bf[0, -1, 9, :] = -np.inf                            # a whole row switched off
    bias = inputs.f32_to_bf16_bits(bf).reshape(bf.shape)
    vl = np.array([520, 391, 77], dtype=np.int32)
    got, lse = run(api, Qb, Kb, Vb, 0.125, bias, vl=vl, causal=causal, want_lse=True)
    assert api.flat_attn_last_variant() == api.FLAT_VARIANT_TC2
    ref = oracle.attention(Qb, Kb, Vb, 0.125, bias=bias, valid_len=vl, causal=causal, want_lse=True)
    check_bf16(got, ref["O"], "staged bias %s causal=%d" % (bshape, causal))
    dead = np.isneginf(ref["LSE"])
    assert np.array_equal(np.isneginf(lse), dead) and np.abs(lse[~dead] - ref["LSE"][~dead]).max() <= 1e-3


def test_bias_unaligned_rows_take_the_scalar_loads(api):
    B, H, Nq, Nk, d = 1, 2, 130, 263, 64                 # Nk odd: no 16-byte loads
    rng = np.random.default_rng(4)
    Qb, Kb, Vb = (rand_bits(rng, s) for s in ((B, H, Nq, d), (B, H, Nk, d), (B, H, Nk, d)))
    bias = rand_bits(rng, (B, H, Nq, Nk), sigma=1.5)
    got, _ = run(api, Qb, Kb, Vb, 0.125, bias)
    check_bf16(got, oracle.attention(Qb, Kb, Vb, 0.125, bias=bias)["O"], "bias odd Nk")


@pytest.mark.parametrize("d", [32, 64])
def test_bias_ffma_kernel_bf16_and_f32_inputs(api, d):
    B, H, Nq, Nk = 2, 2, 150, 210
    rng = np.random.default_rng(5 + d)
    Qb, Kb, Vb = (rand_bits(rng, s) for s in ((B, H, Nq, d), (B, H, Nk, d), (B, H, Nk, d)))
    bias = rng.standard_normal((B, 1, Nq, Nk)).astype(np.float32)
    bias[1, 0, 3, :] = -np.inf
    got, _ = run(api, Qb, Kb, Vb, 0.2, bias, variant=1, causal=True)
    check_bf16(got, oracle.attention(Qb, Kb, Vb, 0.2, bias=bias, causal=True)["O"], "bias simt d=%d" % d)
    # float32 tensors
    w = lambda b: torch.from_numpy(inputs.bf16_bits_to_f32(b).reshape(b.shape)).cuda()
    Q, K, V = w(Qb), w(Kb), w(Vb)
    O = torch.empty_like(Q)
    api.flat_attn_fwd_ex(Q, K, V, O, 0.2, bias=torch.from_numpy(bias).cuda())
    torch.cuda.synchronize()
    check_f32(O.cpu().numpy().astype(np.float64), oracle.attention(Qb, Kb, Vb, 0.2, bias=bias)["O"], "bias simt f32")


def test_bias_is_refused_by_the_kernels_that_do_not_read_it(api):
    q = torch.zeros(1, 1, 128, 64, dtype=torch.bfloat16, device="cuda")
    b = torch.zeros(1, 1, 128, 128, dtype=torch.bfloat16, device="cuda")
    for variant in (2, 4, 5, 6):
        with pytest.raises(api.FlatAttnError) as e:
            api.flat_attn_fwd_ex(q, q, q, torch.empty_like(q), 1.0, variant=variant, bias=b)
        assert e.value.code == 3
    L = torch.empty(1, 1, 128, 128, dtype=torch.float32, device="cuda")
    A = torch.empty(1, 1, 128, 128, dtype=torch.bfloat16, device="cuda")
    p = api._params(q, q, q, torch.empty_like(q), 1.0, None, None, 0, bias=b)
    import ctypes
    assert api._lib.flat_attn_naive_fwd_ex(ctypes.byref(p), L.data_ptr(), A.data_ptr(), None) == 3
