"""CUDA path vs CPU oracle, element by element on the same seeded inputs, through the C ABI."""
import math

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


def run_fused_bf16(api, Qb, Kb, Vb, scale, vl=None, variant=0, causal=False):
    Q, K, V = bf16_tensor(Qb), bf16_tensor(Kb), bf16_tensor(Vb)
    O = torch.full(Q.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    vlt = None if vl is None else torch.from_numpy(vl).cuda()
    api.flat_attn_fwd_ex(Q, K, V, O, scale, k_valid_len=vlt, status=status, variant=variant, causal=causal)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, "device status 0x%x" % int(status.item())
    return bf16_to_f64(O)


SMALL = [
    # B, H, Nq, Nk, d  -- several 128-tiles plus ragged tails in both Nq and Nk
    (1, 1, 128, 128, 64),
    (1, 2, 256, 384, 64),
    (2, 3, 300, 517, 64),
    (1, 2, 129, 1, 64),
    (1, 1, 1, 700, 64),
    (2, 2, 200, 333, 128),
    (1, 1, 128, 256, 128),
]


@pytest.mark.parametrize("shape", SMALL)
@pytest.mark.parametrize("variant", [1, 2, 3, 4, 5], ids=["simt", "tc", "tc2", "tc2single", "tc3"])
def test_fused_bf16_small(api, shape, variant):
    B, H, Nq, Nk, d = shape
    if variant in (4, 5) and d != 64:
        pytest.skip("single-tile TC2 CTAs exist for d = 64 only")
    rng = np.random.default_rng(abs(hash(shape)) % (2 ** 31))
    Qb, Kb, Vb = rand_bits(rng, (B, H, Nq, d)), rand_bits(rng, (B, H, Nk, d)), rand_bits(rng, (B, H, Nk, d))
    scale = 1 / math.sqrt(d)
    ref = oracle.attention(Qb, Kb, Vb, scale)["O"]
    got = run_fused_bf16(api, Qb, Kb, Vb, scale, variant=variant)
    check_bf16(got, ref, "fused bf16 %s v%d" % (shape, variant))


@pytest.mark.parametrize("variant", [1, 2, 3, 4, 5], ids=["simt", "tc", "tc2", "tc2single", "tc3"])
@pytest.mark.parametrize("d", [64, 128])
def test_fused_bf16_masked(api, variant, d):
    if variant in (4, 5) and d != 64:
        pytest.skip("single-tile TC2 CTAs exist for d = 64 only")
    B, H, Nq, Nk = 5, 2, 200, 600
    rng = np.random.default_rng(77 + d)
    Qb, Kb, Vb = rand_bits(rng, (B, H, Nq, d)), rand_bits(rng, (B, H, Nk, d)), rand_bits(rng, (B, H, Nk, d))
    vl = np.array([600, 1, 128, 385, 0], dtype=np.int32)    # full, single key, tile edge, ragged, none
    # finite garbage in masked rows must not matter
    Kf, Vf = inputs.bf16_bits_to_f32(Kb).reshape(Kb.shape).copy(), inputs.bf16_bits_to_f32(Vb).reshape(Vb.shape).copy()
    for b in range(B):
        Kf[b, :, vl[b]:] = 1000.0
        Vf[b, :, vl[b]:] = -3000.0
    Kb, Vb = inputs.f32_to_bf16_bits(Kf).reshape(Kb.shape), inputs.f32_to_bf16_bits(Vf).reshape(Vb.shape)
    scale = 1 / math.sqrt(d)
    ref = oracle.attention(Qb, Kb, Vb, scale, valid_len=vl)["O"]
    got = run_fused_bf16(api, Qb, Kb, Vb, scale, vl=vl, variant=variant)
    check_bf16(got, ref, "masked d=%d v%d" % (d, variant))
    assert np.all(got[4] == 0.0)                            # no valid key: O = 0


@pytest.mark.parametrize("variant", [1, 2, 3, 4, 5], ids=["simt", "tc", "tc2", "tc2single", "tc3"])
def test_fused_bf16_planted_keys(api, variant):
    """Peaked softmax on a planted key with position-coded V: a dropped, duplicated, shifted or
    mis-masked key tile moves O by O(1)."""
    w = inputs.Workload("planted", 2, 2, 384, 1000, 64, masked=True)
    Qb, Kb, Vb, planted = inputs.make_planted_qkv_bf16(w, seed=5)
    vl = inputs.make_valid_len(w, seed=5)
    ref = oracle.attention(Qb, Kb, Vb, w.scale, valid_len=vl, want_weights=True)
    # the construction does what it says: the planted key dominates
    A = ref["A"]
    for b in range(w.B):
        top = A[b, 0].argmax(-1)
        assert np.mean(top == planted[b]) > 0.95
    got = run_fused_bf16(api, Qb, Kb, Vb, w.scale, vl=vl, variant=variant)
    check_bf16(got, ref["O"], "planted v%d" % variant)


@pytest.mark.parametrize("variant", [0, 5], ids=["auto", "tc3"])
def test_many_items_per_cta(api, variant):
    """More (head, row-slab) work items than SMs, so the persistent CTAs of the d = 64 kernel take several
    items each, one behind the other: ragged query slabs, per-batch key counts that differ between
    neighbouring items (including 0 and 1), and rows whose maximum keeps rising (peaked logits), so that
    the redo path also runs right before and after an item boundary."""
    B, H, Nq, Nk, d = 40, 16, 300, 333, 64                  # 640 heads x 2 slabs = 1280 items: over 8 per SM, the persistent grid
    rng = np.random.default_rng(1234)
    # (V of standard deviation 1/4: with logits this peaked O is close to single V rows, and the absolute
    # tolerance is meant for |O| of order 1, where the bf16 rounding of O and of the weights stays well below it)
    Qb, Kb, Vb = rand_bits(rng, (B, H, Nq, d), 1.5), rand_bits(rng, (B, H, Nk, d), 1.5), rand_bits(rng, (B, H, Nk, d), 0.25)
    vl = rng.integers(1, Nk + 1, size=B).astype(np.int32)
    vl[[0, 5, 11]] = [0, 1, Nk]
    vl[7], vl[8], vl[9] = 128, 129, 256                      # tile edges
    scale = 0.6                                              # logits of a few tens: the lazy maximum is overtaken often
    ref = oracle.attention(Qb, Kb, Vb, scale, valid_len=vl)["O"]
    got = run_fused_bf16(api, Qb, Kb, Vb, scale, vl=vl, variant=variant)
    check_bf16(got, ref, "many items v%d" % variant)
    assert np.all(got[0] == 0.0)


@pytest.mark.parametrize("variant", [0, 5], ids=["auto", "tc3"])
def test_reference_maximum_carried_from_item_to_item(api, variant):
    """The persistent CTAs of the d = 64 kernel start an item on the reference maximum of the item before.
    Heads whose logits differ by orders of magnitude follow each other here, in both directions: a reference
    far too high (the first step's sums vanish), far too low (they overflow), and moderately off (kept: the
    weights are then tiny or large but the quotient is the same)."""
    B, H, Nq, Nk, d = 40, 16, 512, 384, 64                  # 640 heads x 2 slabs: the persistent grid
    rng = np.random.default_rng(77)
    q = rng.standard_normal((B, H, Nq, d)).astype(np.float32)
    factor = np.array([1.0, 30.0, 0.02, 6.0, 100.0, 0.3, 12.0, 0.001], dtype=np.float32)
    q *= factor[rng.integers(0, len(factor), size=(B, H))][:, :, None, None]
    from paper_2107_06419_b200 import inputs
    Qb = inputs.f32_to_bf16_bits(q).reshape(q.shape)
    Kb, Vb = rand_bits(rng, (B, H, Nk, d)), rand_bits(rng, (B, H, Nk, d), 0.25)
    scale = 0.5
    ref = oracle.attention(Qb, Kb, Vb, scale)["O"]
    got = run_fused_bf16(api, Qb, Kb, Vb, scale, variant=variant)
    check_bf16(got, ref, "carried reference v%d" % variant)


@pytest.mark.parametrize("shape", [(40, 16, 700, 700), (40, 16, 520, 900), (80, 16, 256, 256)],
                         ids=["three_slabs", "three_slabs_more_keys", "one_slab"])
def test_causal_many_items_per_cta(api, shape):
    """The causal mask on the persistent grid of the d = 64 kernel: the slabs of a head are dealt in
    complementary pairs; with an odd number of slabs the middle one has no partner (an empty slot that must
    neither compute nor store), and with one slab per head every second slot is empty.  O is preset to NaN,
    so a row that no item wrote, or that an empty slot overwrote with zeros, fails the comparison."""
    B, H, Nq, Nk = shape
    d = 64
    rng = np.random.default_rng(B * Nq + Nk)
    Qb, Kb, Vb = rand_bits(rng, (B, H, Nq, d)), rand_bits(rng, (B, H, Nk, d)), rand_bits(rng, (B, H, Nk, d))
    vl = rng.integers(Nk // 2, Nk + 1, size=B).astype(np.int32)
    scale = d ** -0.5
    ref = oracle.attention(Qb, Kb, Vb, scale, valid_len=vl, causal=True)["O"]
    for variant in (0, 5):
        got = run_fused_bf16(api, Qb, Kb, Vb, scale, vl=vl, variant=variant, causal=True)
        check_bf16(got, ref, "causal many items v%d" % variant)


CAUSAL_SHAPES = [
    # B, H, Nq, Nk, d, masked
    (1, 2, 256, 256, 64, False),        # square: row i sees keys 0..i
    (2, 2, 300, 300, 64, True),         # ragged tiles, key-padding on top
    (1, 2, 130, 517, 64, False),        # Nk > Nq: the last query sees every key
    (1, 1, 200, 70, 64, False),         # Nk < Nq: the first 130 queries see no key (O = 0)
    (2, 1, 384, 640, 128, True),
    (1, 2, 100, 100, 32, False),
    (3, 2, 1000, 1000, 64, False),      # several slabs and key steps per head
    (2, 2, 640, 1664, 64, True),
]


@pytest.mark.parametrize("shape", CAUSAL_SHAPES)
@pytest.mark.parametrize("variant", [0, 1, 3, 4, 5], ids=["auto", "simt", "tc2", "tc2single", "tc3"])
def test_fused_bf16_causal(api, shape, variant):
    """Causal mask (query i sees keys j <= i + Nk - Nq), alone and on top of a key-padding mask."""
    B, H, Nq, Nk, d, masked = shape
    if variant in (4, 5) and d != 64:
        pytest.skip("d = 64 only")
    if variant in (3, 4, 5) and d not in (64, 128):
        pytest.skip("tensor-core kernels: d in {64, 128}")
    rng = np.random.default_rng(abs(hash(shape)) % (2 ** 31))
    Qb, Kb, Vb = rand_bits(rng, (B, H, Nq, d)), rand_bits(rng, (B, H, Nk, d)), rand_bits(rng, (B, H, Nk, d))
    vl = None
    if masked:
        vl = rng.integers(1, Nk + 1, size=B).astype(np.int32)
        vl[0] = Nk // 2 + 1
    scale = 1 / math.sqrt(d)
    ref = oracle.attention(Qb, Kb, Vb, scale, valid_len=vl, causal=True)["O"]
    got = run_fused_bf16(api, Qb, Kb, Vb, scale, vl=vl, variant=variant, causal=True)
    check_bf16(got, ref, "causal %s v%d" % (shape, variant))
    if Nk < Nq:
        assert np.all(got[:, :, :Nq - Nk] == 0.0)


def test_causal_f32_and_naive(api):
    B, H, Nq, Nk, d = 1, 2, 150, 333, 64
    rng = np.random.default_rng(99)
    Qf = rng.standard_normal((B, H, Nq, d)).astype(np.float32)
    Kf = rng.standard_normal((B, H, Nk, d)).astype(np.float32)
    Vf = rng.standard_normal((B, H, Nk, d)).astype(np.float32)
    ref = oracle.attention(Qf, Kf, Vf, 0.125, causal=True)["O"]
    Q, K, V = (torch.from_numpy(x).cuda() for x in (Qf, Kf, Vf))
    O = torch.full(Q.shape, float("nan"), dtype=torch.float32, device="cuda")
    api.flat_attn_fwd_ex(Q, K, V, O, 0.125, causal=True)
    check_f32(O.double().cpu().numpy(), ref, "causal f32")
    # the unfused baseline with the same mask (bf16: tensor-core logits, masked softmax, attend)
    Qb, Kb, Vb = (inputs.f32_to_bf16_bits(x).reshape(x.shape) for x in (Qf, Kf, Vf))
    refb = oracle.attention(Qb, Kb, Vb, 0.125, causal=True)
    Qt, Kt, Vt = bf16_tensor(Qb), bf16_tensor(Kb), bf16_tensor(Vb)
    Ot = torch.full(Qt.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    L = torch.empty((B, H, Nq, Nk), dtype=torch.float32, device="cuda")
    A = torch.empty((B, H, Nq, Nk), dtype=torch.bfloat16, device="cuda")
    api.flat_attn_naive_fwd_ex(Qt, Kt, Vt, Ot, L, A, 0.125, causal=True)
    torch.cuda.synchronize()
    check_bf16(bf16_to_f64(Ot), refb["O"], "causal naive")
    iu = np.triu_indices(Nq, k=Nk - Nq + 1, m=Nk)
    assert np.all(A.float().cpu().numpy()[0, 0][iu] == 0.0)


@pytest.mark.parametrize("seed", [20240607, 7, 424242])
def test_randomised_shapes_against_the_ffma_kernel(api, seed):
    """Forty random problems (shape, key-padding, causal, scale, logit spread) through the dispatcher and
    through every tensor-core variant that applies, each compared element by element with the FFMA kernel
    (an independent implementation: different tiling, exact running maximum, no polynomial) under the
    bf16 tolerance, and the smaller ones with the oracle as well.  Some have more than eight work
    items per SM (the persistent grid of the d = 64 kernel), some a single key step."""
    rng = np.random.default_rng(seed)
    for case in range(40):
        d = int(rng.choice([64, 64, 64, 128]))
        big = case % 5 == 0
        if big:
            B, H = int(rng.integers(20, 40)), 16
            Nq, Nk = int(rng.integers(260, 520)), int(rng.integers(1, 400))
        else:
            B, H = int(rng.integers(1, 4)), int(rng.integers(1, 5))
            Nq, Nk = int(rng.integers(1, 900)), int(rng.integers(1, 1400))
        causal = bool(rng.integers(0, 2))
        sigma = float(rng.choice([0.5, 1.0, 2.0]))
        scale = float(rng.choice([1 / math.sqrt(d), 0.3, -0.2]))
        Qb, Kb = rand_bits(rng, (B, H, Nq, d), sigma), rand_bits(rng, (B, H, Nk, d), sigma)
        Vb = rand_bits(rng, (B, H, Nk, d), 0.25)
        vl = None
        if rng.integers(0, 2):
            vl = rng.integers(0, Nk + 1, size=B).astype(np.int32)
        what = "case %d: B%d H%d Nq%d Nk%d d%d causal=%s scale=%.3g sigma=%g vl=%s" % (
            case, B, H, Nq, Nk, d, causal, scale, sigma, None if vl is None else vl.tolist()[:6])
        ref = run_fused_bf16(api, Qb, Kb, Vb, scale, vl=vl, variant=1, causal=causal)
        if B * H * Nq * Nk < 3e6:
            check_bf16(ref, oracle.attention(Qb, Kb, Vb, scale, valid_len=vl, causal=causal)["O"], what + " (ffma vs oracle)")
        variants = [0, 3] + ([4, 5] if d == 64 else [])
        for variant in variants:
            got = run_fused_bf16(api, Qb, Kb, Vb, scale, vl=vl, variant=variant, causal=causal)
            # two bf16 results, each within half the tolerance of the exact one
            check_bf16(got, ref, what + " v%d" % variant)


@pytest.mark.parametrize("scale", [1.0, 0.05, -0.125, 3.0, 0.0])
def test_fused_bf16_scales_tc(api, scale):
    B, H, Nq, Nk, d = 1, 2, 256, 512, 64
    rng = np.random.default_rng(5)
    Qb, Kb, Vb = rand_bits(rng, (B, H, Nq, d)), rand_bits(rng, (B, H, Nk, d)), rand_bits(rng, (B, H, Nk, d))
    ref = oracle.attention(Qb, Kb, Vb, scale)["O"]
    for variant in (2, 3, 4, 5):
        got = run_fused_bf16(api, Qb, Kb, Vb, scale, variant=variant)
        check_bf16(got, ref, "scale %g v%d" % (scale, variant))


def test_rising_maximum_forces_rescale(api):
    """Keys ordered so that the row maximum keeps rising tile after tile (logits grow with j)."""
    B, H, Nq, Nk, d = 1, 1, 128, 1024, 64
    rng = np.random.default_rng(9)
    Qf = np.abs(rng.standard_normal((B, H, Nq, d))).astype(np.float32)
    ramp = (np.arange(Nk, dtype=np.float32) / Nk * 6.0)[None, None, :, None]
    Kf = (np.abs(rng.standard_normal((B, H, Nk, d))) * 0.2 + ramp * 0.25).astype(np.float32)
    Vf = rng.standard_normal((B, H, Nk, d)).astype(np.float32)
    Qb, Kb, Vb = (inputs.f32_to_bf16_bits(x).reshape(x.shape) for x in (Qf, Kf, Vf))
    ref = oracle.attention(Qb, Kb, Vb, 1.0, want_logits=True)
    L = ref["L"].reshape(Nq, Nk)
    assert np.all(L[:, -128:].max(1) - L[:, :128].max(1) > 20)      # > 8 log2 units per several tiles
    for variant in (1, 2, 3, 4, 5):
        got = run_fused_bf16(api, Qb, Kb, Vb, 1.0, variant=variant)
        check_bf16(got, ref["O"], "rising max v%d" % variant)


@pytest.mark.parametrize("shape", [(1, 2, 200, 333, 64), (2, 1, 128, 257, 128), (1, 1, 70, 130, 32), (1, 2, 65, 64, 16)])
def test_fused_f32(api, shape):
    B, H, Nq, Nk, d = shape
    rng = np.random.default_rng(31 + d)
    Q = rng.standard_normal((B, H, Nq, d)).astype(np.float32)
    K = rng.standard_normal((B, H, Nk, d)).astype(np.float32)
    V = rng.standard_normal((B, H, Nk, d)).astype(np.float32)
    vl = np.array([Nk, max(1, Nk // 3)], dtype=np.int32)[:B]
    scale = 1 / math.sqrt(d)
    ref = oracle.attention(Q, K, V, scale, valid_len=vl)["O"]
    Qt, Kt, Vt = (torch.from_numpy(x).cuda() for x in (Q, K, V))
    O = torch.full(Qt.shape, float("nan"), device="cuda")
    api.flat_attn_fwd_ex(Qt, Kt, Vt, O, scale, k_valid_len=torch.from_numpy(vl).cuda())
    torch.cuda.synchronize()
    check_f32(O.cpu().numpy().astype(np.float64), ref, "fused f32 %s" % (shape,))


@pytest.mark.parametrize("Nk", [333, 336, 1024], ids=["ffma", "tc-ragged", "tc"])
@pytest.mark.parametrize("d", [64, 128])
def test_naive_bf16(api, d, Nk):
    """Nk % 8 == 0 takes the tensor-core contractions, otherwise the FFMA kernels."""
    B, H, Nq = 2, 2, 200
    rng = np.random.default_rng(13 + d)
    Qb, Kb, Vb = rand_bits(rng, (B, H, Nq, d)), rand_bits(rng, (B, H, Nk, d)), rand_bits(rng, (B, H, Nk, d))
    vl = np.array([Nk, 130], dtype=np.int32)
    scale = 1 / math.sqrt(d)
    ref = oracle.attention(Qb, Kb, Vb, scale, valid_len=vl, want_logits=True, want_weights=True)
    Q, K, V = bf16_tensor(Qb), bf16_tensor(Kb), bf16_tensor(Vb)
    O = torch.full(Q.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    L = torch.full((B, H, Nq, Nk), float("nan"), dtype=torch.float32, device="cuda")
    A = torch.full((B, H, Nq, Nk), float("nan"), dtype=torch.bfloat16, device="cuda")
    api.flat_attn_naive_fwd_ex(Q, K, V, O, L, A, scale, k_valid_len=torch.from_numpy(vl).cuda())
    torch.cuda.synchronize()
    check_bf16(bf16_to_f64(O), ref["O"], "naive O d=%d" % d)
    Lg, Ag = L.cpu().numpy().astype(np.float64), bf16_to_f64(A)
    for b in range(B):
        n = vl[b]
        assert np.max(np.abs(Lg[b, :, :, :n] - ref["L"][b, :, :, :n])) < 1e-4
        assert np.all(Ag[b, :, :, n:] == 0.0)
    assert np.max(np.abs(Ag - ref["A"])) < 4e-3          # bf16 rounding of weights <= 1
    # unmasked entry point agrees with the fused kernel's result on the same data
    api.flat_attn_naive_fwd(Q, K, V, O, L, A, scale)
    torch.cuda.synchronize()
    check_bf16(bf16_to_f64(O), oracle.attention(Qb, Kb, Vb, scale)["O"], "naive unmasked d=%d" % d)


def test_naive_f32(api):
    B, H, Nq, Nk, d = 1, 2, 130, 200, 64
    rng = np.random.default_rng(17)
    Q = rng.standard_normal((B, H, Nq, d)).astype(np.float32)
    K = rng.standard_normal((B, H, Nk, d)).astype(np.float32)
    V = rng.standard_normal((B, H, Nk, d)).astype(np.float32)
    ref = oracle.attention(Q, K, V, 0.125, want_weights=True)
    Qt, Kt, Vt = (torch.from_numpy(x).cuda() for x in (Q, K, V))
    O = torch.empty_like(Qt)
    L = torch.empty((B, H, Nq, Nk), device="cuda")
    A = torch.empty((B, H, Nq, Nk), device="cuda")
    api.flat_attn_naive_fwd_ex(Qt, Kt, Vt, O, L, A, 0.125)
    torch.cuda.synchronize()
    check_f32(O.cpu().numpy().astype(np.float64), ref["O"], "naive f32")
    assert np.max(np.abs(A.cpu().numpy().astype(np.float64) - ref["A"])) < 1e-6


def test_host_entry_point(api):
    B, H, Nq, Nk, d = 2, 2, 256, 300, 64
    rng = np.random.default_rng(23)
    Qb, Kb, Vb = rand_bits(rng, (B, H, Nq, d)), rand_bits(rng, (B, H, Nk, d)), rand_bits(rng, (B, H, Nk, d))
    vl = np.array([300, 77], dtype=np.int32)
    Q, K, V = (bf16_tensor(x, device=None).pin_memory() for x in (Qb, Kb, Vb))
    O = torch.empty(Q.shape, dtype=torch.bfloat16).pin_memory()
    ws = torch.empty(api.flat_attn_host_workspace_bytes(B, H, Nq, Nk, d), dtype=torch.uint8, device="cuda")
    api.flat_attn_fwd_host(Q, K, V, O, 0.125, ws, k_valid_len=torch.from_numpy(vl).pin_memory())
    torch.cuda.synchronize()
    ref = oracle.attention(Qb, Kb, Vb, 0.125, valid_len=vl)["O"]
    check_bf16(bf16_to_f64(O), ref, "host entry")
    with pytest.raises(api.FlatAttnError) as e:
        api.flat_attn_fwd_host(Q, K, V, O, 0.125, ws[:1024])
    assert e.value.code == 5


def test_cuda_graph_capture_and_replay(api):
    """The entry points only enqueue work on the caller's stream (no allocation, no synchronisation), so a
    launch can be captured in a CUDA graph and replayed; the replays must reproduce the direct launch bit
    for bit.  Both default kernels: d = 64 (persistent two-threads-per-row kernel) and d = 128."""
    for (B, H, N, d) in [(8, 16, 2304, 64), (1, 8, 4736, 128)]:
        rng = np.random.default_rng(N)
        Q, K, V = (bf16_tensor(rand_bits(rng, (B, H, N, d))) for _ in range(3))
        O_direct = torch.empty_like(Q)
        api.flat_attn_fwd(Q, K, V, O_direct, d ** -0.5)           # also warms the per-device launch set-up
        torch.cuda.synchronize()
        O = torch.zeros_like(Q)
        g = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                api.flat_attn_fwd(Q, K, V, O, d ** -0.5, stream=side)
        torch.cuda.current_stream().wait_stream(side)
        for _ in range(3):
            O.zero_()
            g.replay()
            torch.cuda.synchronize()
            assert torch.equal(O.view(torch.int16), O_direct.view(torch.int16)), (B, H, N, d)


def test_output_padding_untouched(api):
    """Canary rows around O: the kernels write exactly B*H*Nq*d elements."""
    B, H, Nq, Nk, d = 1, 3, 130, 140, 64
    rng = np.random.default_rng(29)
    Qb, Kb, Vb = rand_bits(rng, (B, H, Nq, d)), rand_bits(rng, (B, H, Nk, d)), rand_bits(rng, (B, H, Nk, d))
    Q, K, V = bf16_tensor(Qb), bf16_tensor(Kb), bf16_tensor(Vb)
    n = B * H * Nq * d
    for variant in (1, 2, 3, 5):
        buf = torch.full((n + 2048,), 7.0, dtype=torch.bfloat16, device="cuda")
        O = buf[1024:1024 + n].view(B, H, Nq, d)
        api.flat_attn_fwd_ex(Q, K, V, O, 0.125, variant=variant)
        torch.cuda.synchronize()
        assert torch.all(buf[:1024] == 7.0) and torch.all(buf[1024 + n:] == 7.0)
        check_bf16(bf16_to_f64(O), oracle.attention(Qb, Kb, Vb, 0.125)["O"], "canary v%d" % variant)


def test_bounded_wait_gives_up_cleanly(api):
    """A wait that nothing satisfies runs out, reports its code and leaves the GPU usable."""
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.flat_attn_selftest_wait_timeout(status)
    torch.cuda.synchronize()
    assert int(status.item()) == api.FLAT_SELFTEST_TIMEOUT_CODE
    # the context is still healthy: a normal call right after gives the right answer
    rng = np.random.default_rng(99)
    Qb, Kb, Vb = rand_bits(rng, (1, 1, 128, 64)), rand_bits(rng, (1, 1, 256, 64)), rand_bits(rng, (1, 1, 256, 64))
    got = run_fused_bf16(api, Qb, Kb, Vb, 0.125, variant=3)
    check_bf16(got, oracle.attention(Qb, Kb, Vb, 0.125)["O"], "after timeout self-test")


def test_give_up_without_a_status_word_leaves_a_trace(api):
    """Callers that pass no status word (flat_attn_fwd) can still learn of a device-side give-up: the
    code goes to the library's sticky word.  The wait that runs out is the self-test's (a barrier that
    nothing completes); nothing faults."""
    api.flat_attn_clear_device_error()
    rng = np.random.default_rng(98)
    Qb, Kb, Vb = rand_bits(rng, (2, 8, 2048, 64)), rand_bits(rng, (2, 8, 2048, 64)), rand_bits(rng, (2, 8, 2048, 64))
    Q, K, V = bf16_tensor(Qb), bf16_tensor(Kb), bf16_tensor(Vb)
    O = torch.empty_like(Q)
    api.flat_attn_fwd(Q, K, V, O, 0.125)
    torch.cuda.synchronize()
    assert api.flat_attn_last_device_error() == 0          # a healthy call leaves the word alone
    assert api.flat_attn_last_variant() == api.FLAT_VARIANT_TC3
    api.flat_attn_selftest_wait_timeout(None)
    torch.cuda.synchronize()
    assert api.flat_attn_last_device_error() == api.FLAT_SELFTEST_TIMEOUT_CODE
    O2 = torch.empty_like(Q)
    api.flat_attn_fwd(Q, K, V, O2, 0.125)
    torch.cuda.synchronize()
    assert api.flat_attn_last_device_error() == api.FLAT_SELFTEST_TIMEOUT_CODE   # sticky until cleared
    assert torch.equal(O.view(torch.int16), O2.view(torch.int16))
    api.flat_attn_clear_device_error()
    assert api.flat_attn_last_device_error() == 0


@pytest.mark.parametrize("sigma,scale", [(3.0, 1.0), (1.0, 20.0), (6.0, 0.5)])
def test_wide_dynamic_range(api, sigma, scale):
    """Logits with a standard deviation of dozens to hundreds: row maxima jump by far more than the
    exponent range between tiles, so the stale-reference check, the rescale of O and the clamps of
    the polynomial exponential all fire; softmax rows are nearly one-hot."""
    B, H, Nq, Nk, d = 1, 2, 256, 1536, 64
    rng = np.random.default_rng(int(sigma * 10 + scale))
    Qb, Kb = rand_bits(rng, (B, H, Nq, d), sigma), rand_bits(rng, (B, H, Nk, d), sigma)
    Vb = rand_bits(rng, (B, H, Nk, d))
    ref = oracle.attention(Qb, Kb, Vb, scale, want_logits=True)
    spread = ref["L"].max(-1) - np.median(ref["L"], -1)
    assert np.median(spread) > 100                                  # far beyond 2^126 in base-2 terms
    for variant in (1, 2, 3, 4, 5):
        got = run_fused_bf16(api, Qb, Kb, Vb, scale, variant=variant)
        check_bf16(got, ref["O"], "wide range sigma=%g scale=%g v%d" % (sigma, scale, variant))


@pytest.mark.parametrize("spike_col", [3, 67, 127], ids=["col3", "col67", "col127"])
def test_spike_on_polynomial_lane(api, spike_col):
    """One key far above all others (hundreds of log2 units), sitting in a later tile on a column
    that the kernel evaluates with the polynomial exponential and not with the ex2 unit: the clamp
    must turn it into an overflow that forces the careful pass, not into garbage."""
    B, H, Nq, Nk, d = 1, 1, 256, 1280, 64
    rng = np.random.default_rng(4242)
    u = np.ones(d, dtype=np.float32)
    Qf = (u[None, :] * (1.0 + rng.random((Nq, 1), dtype=np.float32)) + 0.1 * rng.standard_normal((Nq, d))).astype(np.float32)
    Kf = (0.01 * rng.standard_normal((Nk, d))).astype(np.float32)
    # (column 3 and 67: polynomial lanes of the first / second half of a 128-key step, which the
    # kernel that splits a row over two threads handles in different warps; 127: last ex2 lane)
    Kf[131] = 2.0 * u           # tile 1, column 3
    big = 1024 + spike_col
    Kf[big] = 6.0 * u           # tile 8: 4 * 64 * (1..2) = 256..512 above the first spike
    Vf = rng.standard_normal((Nk, d)).astype(np.float32)
    Qb, Kb, Vb = (inputs.f32_to_bf16_bits(x).reshape(1, 1, *x.shape) for x in (Qf, Kf, Vf))
    ref = oracle.attention(Qb, Kb, Vb, 1.0, want_weights=True)
    assert np.all(ref["A"][0, 0].argmax(-1) == big)
    for variant in (2, 3, 4, 5):
        got = run_fused_bf16(api, Qb, Kb, Vb, 1.0, variant=variant)
        check_bf16(got, ref["O"], "spike v%d" % variant)


def test_polynomial_exp2_accuracy_and_clamps(api):
    x = np.concatenate([np.linspace(-126.0, 126.0, 200001), np.linspace(-1.0, 1.0, 50001),
                        np.arange(-126, 127, dtype=np.float64) + 0.5, np.arange(-126, 127, dtype=np.float64),
                        [-1e30, -500.0, -127.0, -126.5, 126.5, 127.0, 500.0, 1e30]]).astype(np.float32)
    xt = torch.from_numpy(x).cuda()
    y = api.flat_attn_selftest_exp2_poly(xt, torch.empty_like(xt)).cpu().numpy().astype(np.float64)
    ref = np.exp2(np.clip(x.astype(np.float64), -126.0, 126.0))
    assert np.all(np.isfinite(y)) and np.all(y > 0)
    normal = ref >= 2.0 ** -125
    assert np.max(np.abs(y[normal] / ref[normal] - 1.0)) < 1e-4
    assert np.all(y[~normal] < 2.0 ** -124)                # the bottom of the range may come out denormal
    assert y[-1] >= 2.0 ** 125 and y[-2] >= 2.0 ** 125     # far above the range: a huge finite value
