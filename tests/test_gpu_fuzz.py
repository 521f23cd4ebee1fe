"""Seeded random small problems through every fused kernel variant against the oracle: random batch, head and
sequence sizes (ragged against every tile size), key-padding masks that include empty and full batches, the causal
mask with Nq != Nk, both head sizes, both storage types, the row log-sum-exp.  The cases are drawn from a fixed
seed, so the test is the same on every run; a variant that does not take a case must refuse it, nothing else."""
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


def cases(seed, count):
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(count):
        B, H = int(rng.integers(1, 4)), int(rng.integers(1, 4))
        Nq = int(rng.choice([1, 63, 64, 65, 127, 128, 129, 200, 255, 256, 257, 300, 384, 513, 700]))
        Nk = int(rng.choice([1, 17, 63, 64, 65, 127, 128, 129, 191, 192, 256, 257, 320, 511, 512, 513, 640, 900, 1100]))
        d = int(rng.choice([64, 64, 128]))
        causal = bool(rng.integers(0, 2))
        mask = int(rng.integers(0, 3))                   # 0: none, 1: random lengths, 2: lengths incl. 0 and Nk
        out.append((B, H, Nq, Nk, d, causal, mask, int(rng.integers(0, 2 ** 31))))
    return out


BF16_VARIANTS = [0, 1, 2, 3, 4, 5, 8, 9, 10, 11, 12, 13, 14, 15, 16]


@pytest.mark.parametrize("case", cases(20210706, 96), ids=lambda c: "B%dH%dq%dk%dd%d%s%s" % (c[0], c[1], c[2], c[3], c[4], "c" if c[5] else "", "m%d" % c[6]))
def test_bf16_variants(api, case):
    B, H, Nq, Nk, d, causal, mask, seed = case
    rng = np.random.default_rng(seed)
    Qb, Kb, Vb = rand_bits(rng, (B, H, Nq, d)), rand_bits(rng, (B, H, Nk, d)), rand_bits(rng, (B, H, Nk, d))
    vl = None
    if mask == 1:
        vl = rng.integers(1, Nk + 1, size=B).astype(np.int32)
    elif mask == 2:
        vl = np.array([0, Nk, Nk // 2][:B], dtype=np.int32)
    scale = float(rng.choice([d ** -0.5, 0.3, -0.2]))
    ref = oracle.attention(Qb, Kb, Vb, scale, valid_len=vl, causal=causal, want_lse=True)
    Q, K, V = bf16_tensor(Qb), bf16_tensor(Kb), bf16_tensor(Vb)
    ran = 0
    for variant in BF16_VARIANTS:
        O = torch.full(Q.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
        lse = torch.full(Q.shape[:3], float("nan"), dtype=torch.float32, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        want_lse = variant != 2                          # (the single-tile predecessor kernel does not write it)
        try:
            api.flat_attn_fwd_ex(Q, K, V, O, scale, k_valid_len=None if vl is None else torch.from_numpy(vl).cuda(),
                                 status=status, variant=variant, causal=causal, lse=lse if want_lse else None)
        except api.FlatAttnError as e:
            assert e.code == 3, (variant, e.code)        # FLAT_ERR_UNSUPPORTED is the only refusal allowed here
            continue
        torch.cuda.synchronize()
        assert int(status.item()) == 0, (variant, hex(int(status.item())))
        check_bf16(bf16_to_f64(O), ref["O"], "fuzz %s variant %d" % (case[:7], variant))
        if want_lse:
            got = lse.double().cpu().numpy()
            dead = np.isneginf(ref["LSE"])
            assert np.array_equal(np.isneginf(got), dead), (case[:7], variant)
            if (~dead).any():
                assert np.max(np.abs(got[~dead] - ref["LSE"][~dead])) < 2e-3, (case[:7], variant)
        ran += 1
    assert ran >= 2                                      # AUTO and the FFMA kernel take everything


@pytest.mark.parametrize("case", cases(2107, 40), ids=lambda c: "B%dH%dq%dk%dd%d%s%s" % (c[0], c[1], c[2], c[3], c[4], "c" if c[5] else "", "m%d" % c[6]))
def test_f32_variants(api, case):
    B, H, Nq, Nk, d, causal, mask, seed = case
    rng = np.random.default_rng(seed)
    Q, K, V = (rng.standard_normal(s).astype(np.float32) for s in ((B, H, Nq, d), (B, H, Nk, d), (B, H, Nk, d)))
    vl = None
    if mask == 1:
        vl = rng.integers(1, Nk + 1, size=B).astype(np.int32)
    elif mask == 2:
        vl = np.array([0, Nk, Nk // 2][:B], dtype=np.int32)
    scale = float(rng.choice([d ** -0.5, 0.3, -0.2]))
    ref = oracle.attention(Q, K, V, scale, valid_len=vl, causal=causal, want_lse=True)
    Qt, Kt, Vt = (torch.from_numpy(x).cuda() for x in (Q, K, V))
    for variant in (0, 1, 7):
        O = torch.full(Qt.shape, float("nan"), dtype=torch.float32, device="cuda")
        lse = torch.full(Qt.shape[:3], float("nan"), dtype=torch.float32, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        try:
            api.flat_attn_fwd_ex(Qt, Kt, Vt, O, scale, k_valid_len=None if vl is None else torch.from_numpy(vl).cuda(),
                                 status=status, variant=variant, causal=causal, lse=lse)
        except api.FlatAttnError as e:
            assert e.code == 3 and variant == 7 and d != 64, (variant, e.code)
            continue
        torch.cuda.synchronize()
        assert int(status.item()) == 0, (variant, hex(int(status.item())))
        check_f32(O.double().cpu().numpy(), ref["O"], "fuzz f32 %s variant %d" % (case[:7], variant))
        got = lse.double().cpu().numpy()
        dead = np.isneginf(ref["LSE"])
        assert np.array_equal(np.isneginf(got), dead), (case[:7], variant)
        if (~dead).any():
            assert np.max(np.abs(got[~dead] - ref["LSE"][~dead])) < 1e-4, (case[:7], variant)


@pytest.mark.parametrize("case", cases(6419, 24), ids=lambda c: "B%dH%dq%dk%dd%d%s%s" % (c[0], c[1], c[2], c[3], c[4], "c" if c[5] else "", "m%d" % c[6]))
def test_backward(api, case):
    """dQ, dK, dV of the same random problems: forward with the row log-sum-exp, then the two backward kernels."""
    B, H, Nq, Nk, d, causal, mask, seed = case
    rng = np.random.default_rng(seed)
    Qb, Kb, Vb, dOb = (rand_bits(rng, s) for s in ((B, H, Nq, d), (B, H, Nk, d), (B, H, Nk, d), (B, H, Nq, d)))
    vl = None
    if mask == 1:
        vl = rng.integers(1, Nk + 1, size=B).astype(np.int32)
    elif mask == 2:
        vl = np.array([0, Nk, Nk // 2][:B], dtype=np.int32)
    scale = float(rng.choice([d ** -0.5, 0.3]))
    ref = oracle.attention_bwd(Qb, Kb, Vb, dOb, scale, valid_len=vl, causal=causal)
    Q, K, V, dO = bf16_tensor(Qb), bf16_tensor(Kb), bf16_tensor(Vb), bf16_tensor(dOb)
    O = torch.empty_like(Q)
    lse = torch.empty(Q.shape[:3], dtype=torch.float32, device="cuda")
    delta = torch.empty_like(lse)
    dQ = torch.full(Q.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    dK = torch.full(K.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    dV = torch.full(K.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    vlt = None if vl is None else torch.from_numpy(vl).cuda()
    api.flat_attn_fwd_ex(Q, K, V, O, scale, k_valid_len=vlt, status=status, causal=causal, lse=lse)
    api.flat_attn_bwd_ex(Q, K, V, O, dO, lse, dQ, dK, dV, delta, scale, k_valid_len=vlt, status=status, causal=causal)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for name, got in (("dQ", dQ), ("dK", dK), ("dV", dV)):
        g = bf16_to_f64(got)
        assert np.isfinite(g).all(), name
        r = ref[name]
        top = max(float(np.abs(r).max()), 1e-30)
        # (a gradient that is exactly zero -- a single visible key -- comes out as rounding noise of the bf16 O inside delta:
        # the absolute floors stand for 'zero at the scale of the other gradients', which are of order 1 here)
        assert float(np.abs(g - r).max()) <= 2e-2 * top + 1e-4, (case[:7], name)
        assert float(np.abs(g - r).mean()) <= 1e-2 * float(np.abs(r).mean()) + 1e-5, (case[:7], name)


@pytest.mark.parametrize("case", cases(777, 24), ids=lambda c: "B%dH%dq%dk%dd%d%s%s" % (c[0], c[1], c[2], c[3], c[4], "c" if c[5] else "", "m%d" % c[6]))
def test_bias_and_pruning_map(api, case):
    """The same random problems with an additive bias (bf16 or fp32, a random broadcast form, a few -inf entries;
    row lengths that are multiples of 8 take the tiles staged in shared memory at d = 64, the others the per-thread
    loads) and, separately, with a random pruning map over 128 x 128 blocks."""
    B, H, Nq, Nk, d, causal, mask, seed = case
    rng = np.random.default_rng(seed)
    if rng.integers(0, 2):
        Nk = (Nk + 7) // 8 * 8                           # 16-byte aligned bias rows
    Qb, Kb, Vb = rand_bits(rng, (B, H, Nq, d)), rand_bits(rng, (B, H, Nk, d)), rand_bits(rng, (B, H, Nk, d))
    vl = None
    if mask == 1:
        vl = rng.integers(1, Nk + 1, size=B).astype(np.int32)
    elif mask == 2:
        vl = np.array([0, Nk, Nk // 2][:B], dtype=np.int32)
    vlt = None if vl is None else torch.from_numpy(vl).cuda()
    Q, K, V = bf16_tensor(Qb), bf16_tensor(Kb), bf16_tensor(Vb)
    lead = [(B, H), (1, H), (B, 1), (1, 1)][int(rng.integers(0, 4))]
    bf = (rng.standard_normal(lead + (Nq, Nk)) * 1.5).astype(np.float32)
    bf[..., rng.integers(0, Nq), :] = -np.inf            # a whole row switched off
    bf[..., :, rng.integers(0, Nk)] = -np.inf            # and a whole key
    if rng.integers(0, 2):
        bias = inputs.f32_to_bf16_bits(bf).reshape(bf.shape)
        bt = bf16_tensor(bias)
    else:
        bias = bf
        bt = torch.from_numpy(bf).cuda()
    ref = oracle.attention(Qb, Kb, Vb, 0.2, valid_len=vl, causal=causal, bias=bias, want_lse=True)
    for variant in (0, 1):
        O = torch.full(Q.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
        lse = torch.full(Q.shape[:3], float("nan"), dtype=torch.float32, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        api.flat_attn_fwd_ex(Q, K, V, O, 0.2, k_valid_len=vlt, status=status, variant=variant, causal=causal, bias=bt, lse=lse)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        check_bf16(bf16_to_f64(O), ref["O"], "fuzz bias %s variant %d" % (case[:7], variant))
        dead = np.isneginf(ref["LSE"])
        got = lse.double().cpu().numpy()
        assert np.array_equal(np.isneginf(got), dead), (case[:7], variant)
        if (~dead).any():
            assert np.max(np.abs(got[~dead] - ref["LSE"][~dead])) < 2e-3
    # pruning map
    tq, tk = -(-Nq // 128), -(-Nk // 128)
    mlead = [(B, H), (1, H), (B, 1), (1, 1)][int(rng.integers(0, 4))]
    bm = (rng.random(mlead + (tq, tk)) < 0.6).astype(np.uint8)
    refm = oracle.attention(Qb, Kb, Vb, 0.2, valid_len=vl, causal=causal, block_mask=bm, want_lse=True)
    O = torch.full(Q.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full(Q.shape[:3], float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.flat_attn_fwd_ex(Q, K, V, O, 0.2, k_valid_len=vlt, status=status, causal=causal, block_mask=torch.from_numpy(bm).cuda(), lse=lse)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    check_bf16(bf16_to_f64(O), refm["O"], "fuzz pruning map %s" % (case[:7],))
    dead = np.isneginf(refm["LSE"])
    assert np.array_equal(np.isneginf(lse.double().cpu().numpy()), dead)


def test_auto_against_the_two_tile_kernel_at_medium_sizes(api):
    """The dispatcher's choices that only medium-sized problems reach (two warpgroups per tile, key splits over
    clusters, the even deal, one CTA per item, persistent CTAs): 90 seeded random problems, each run three times
    with FLAT_VARIANT_AUTO (same bits every time, no device code) and once with the two-tile kernel, whose output
    the dispatcher's kernel must match within the sum of the two kernels' parity bars."""
    rng = np.random.default_rng(20210706)
    seen = set()
    for it in range(90):
        d = 64 if rng.random() < 0.6 else 128
        B, H = int(rng.integers(1, 9)), int(rng.integers(1, 17))
        Nq = int(rng.integers(1, 13)) * 128 + int(rng.integers(0, 2)) * int(rng.integers(1, 128))
        Nk = int(rng.integers(2, 64)) * 128 + int(rng.integers(0, 2)) * int(rng.integers(1, 128))
        causal = bool(rng.random() < 0.25)
        vl = rng.integers(0, Nk + 1, B).astype(np.int32) if rng.random() < 0.5 else None
        g = torch.Generator(device="cuda").manual_seed(it)
        Q = torch.randn(B, H, Nq, d, device="cuda", dtype=torch.bfloat16, generator=g)
        K = torch.randn(B, H, Nk, d, device="cuda", dtype=torch.bfloat16, generator=g)
        V = torch.randn(B, H, Nk, d, device="cuda", dtype=torch.bfloat16, generator=g)
        vlt = None if vl is None else torch.from_numpy(vl).cuda()
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        outs = []
        for _ in range(3):
            O = torch.full_like(Q, float("nan"))
            api.flat_attn_fwd_ex(Q, K, V, O, d ** -0.5, k_valid_len=vlt, status=status, causal=causal)
            outs.append(O)
        v = api.flat_attn_last_variant()
        seen.add((d, v, api.flat_attn_last_schedule() if v == api.FLAT_VARIANT_TC3 else 0))
        O2 = torch.full_like(Q, float("nan"))
        api.flat_attn_fwd_ex(Q, K, V, O2, d ** -0.5, k_valid_len=vlt, status=status, causal=causal, variant=api.FLAT_VARIANT_TC2)
        torch.cuda.synchronize()
        what = "case %d %s d=%d causal=%d variant %d" % (it, (B, H, Nq, Nk), d, causal, v)
        assert int(status.item()) == 0, what
        assert bool(torch.isfinite(outs[0].float()).all()), what
        assert torch.equal(outs[0], outs[1]) and torch.equal(outs[0], outs[2]), what
        assert float((outs[0].float() - O2.float()).abs().max()) <= 2 * 2e-2, what
    assert len(seen) >= 6, seen                          # (the cases do reach the different kernels and deals)
