"""Key split over a thread-block cluster (launches that would leave most SMs empty): every query tile's keys go
to 2, 4 or 8 CTAs, whose partial softmaxes are merged through distributed shared memory.  Against the oracle:
shapes where some ranks get no key tile at all, ragged tails, both masks, the row log-sum-exp, planted keys (a
partial that is lost or merged twice moves the output by O(1)), and what AUTO picks."""
import numpy as np
import pytest
import torch

import oracle
from paper_2107_06419_b200 import inputs
from helpers import bf16_tensor, bf16_to_f64, check_bf16, rand_bits

pytestmark = pytest.mark.gpu

# FLAT_VARIANT_TC2_SPLIT2 / 4 / 8, then FLAT_VARIANT_TC2_HALVES and HALVES_SPLIT2 / 4 / 8 (the tile's two warpgroups
# on alternate key tiles, merged through shared memory, with the keys over a cluster on top)
SPLITS = [8, 9, 10, 11, 12, 13, 14, 16]           # (16: the two-warpgroup form over clusters of sixteen)


@pytest.fixture(scope="module")
def api():
    from paper_2107_06419_b200 import api as _api
    return _api


def run(api, Qb, Kb, Vb, scale, variant, vl=None, causal=False):
    O = torch.full(Qb.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    lse = torch.full(Qb.shape[:3], float("nan"), dtype=torch.float32, device="cuda")
    api.flat_attn_fwd_ex(bf16_tensor(Qb), bf16_tensor(Kb), bf16_tensor(Vb), O, scale,
                         k_valid_len=None if vl is None else torch.from_numpy(vl).cuda(), status=status, variant=variant,
                         causal=causal, lse=lse)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return bf16_to_f64(O), lse.double().cpu().numpy()


# (B, H, Nq, Nk): one key tile (all ranks but the first idle), fewer tiles than ranks, ragged, many tiles
SHAPES = [(1, 2, 128, 128), (2, 2, 200, 333), (1, 12, 512, 512), (1, 1, 100, 2048), (1, 3, 77, 1000), (2, 1, 384, 4200)]


@pytest.mark.parametrize("variant", SPLITS)
@pytest.mark.parametrize("shape", SHAPES)
def test_dense(api, shape, variant):
    B, H, Nq, Nk = shape
    rng = np.random.default_rng(Nq + Nk + variant)
    Qb, Kb, Vb = rand_bits(rng, (B, H, Nq, 64)), rand_bits(rng, (B, H, Nk, 64)), rand_bits(rng, (B, H, Nk, 64))
    ref = oracle.attention(Qb, Kb, Vb, 0.125, want_lse=True)
    O, lse = run(api, Qb, Kb, Vb, 0.125, variant)
    assert api.flat_attn_last_variant() == variant
    check_bf16(O, ref["O"], "split v%d %s" % (variant, shape))
    assert np.max(np.abs(lse - ref["LSE"])) < 1e-3


@pytest.mark.parametrize("variant", SPLITS)
@pytest.mark.parametrize("causal", [False, True])
def test_masks(api, variant, causal):
    B, H, Nq, Nk = 2, 2, 300, 1100
    rng = np.random.default_rng(41 + variant + causal)
    Qb, Kb, Vb = rand_bits(rng, (B, H, Nq, 64)), rand_bits(rng, (B, H, Nk, 64)), rand_bits(rng, (B, H, Nk, 64))
    vl = np.array([700, 0], dtype=np.int32)              # (the second batch sees no key: every rank's share is empty)
    ref = oracle.attention(Qb, Kb, Vb, 0.2, valid_len=vl, causal=causal, want_lse=True)
    O, lse = run(api, Qb, Kb, Vb, 0.2, variant, vl=vl, causal=causal)
    check_bf16(O, ref["O"], "split masks v%d causal=%d" % (variant, causal))
    assert np.all(O[1] == 0.0)
    assert np.array_equal(np.isneginf(lse), np.isneginf(ref["LSE"]))
    fin = np.isfinite(ref["LSE"])
    assert np.max(np.abs(lse[fin] - ref["LSE"][fin])) < 1e-3


@pytest.mark.parametrize("variant", SPLITS)
def test_planted_keys_and_rising_maximum(api, variant):
    """One planted key per row carries the weight, at a position of its own in every row (so the rank that holds it
    changes from row to row), and the keys' scores rise along the sequence (every later share has the larger
    maximum): the merge has to rescale the earlier partials."""
    w = inputs.WORKLOADS["c1_bert_base_512"]
    Qb, Kb, Vb, planted = inputs.make_planted_qkv_bf16(w)
    ref = oracle.attention(Qb, Kb, Vb, w.scale)["O"]
    O, _ = run(api, Qb, Kb, Vb, w.scale, variant)
    check_bf16(O, ref, "split planted v%d" % variant)
    rng = np.random.default_rng(5)
    Nq, Nk = 256, 2048
    Qf = np.abs(rng.standard_normal((1, 2, Nq, 64))).astype(np.float32)
    ramp = (np.arange(Nk, dtype=np.float32) / Nk * 6.0)[None, None, :, None]
    Kf = (np.abs(rng.standard_normal((1, 2, Nk, 64))) * 0.2 + ramp * 0.25).astype(np.float32)
    Vf = rng.standard_normal((1, 2, Nk, 64)).astype(np.float32)
    Qb2, Kb2, Vb2 = (inputs.f32_to_bf16_bits(x).reshape(x.shape) for x in (Qf, Kf, Vf))
    ref2 = oracle.attention(Qb2, Kb2, Vb2, 0.5)["O"]
    O2, _ = run(api, Qb2, Kb2, Vb2, 0.5, variant)
    check_bf16(O2, ref2, "split rising maximum v%d" % variant)


def test_auto_takes_the_split_for_underfilled_launches(api):
    rng = np.random.default_rng(9)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    if sms != 148:
        pytest.skip("the expected choices are those of a 148-SM GPU")
    # (more tiles than seven SMs in eight: two-per-SM CTAs, unsplit; one key tile: nothing to split)
    for (B, H, Nq, Nk, expect) in [(1, 1, 128, 8192, api.FLAT_VARIANT_TC2_HALVES_SPLIT16), (1, 4, 128, 4096, api.FLAT_VARIANT_TC2_HALVES_SPLIT8), (1, 12, 512, 512, api.FLAT_VARIANT_TC2_HALVES_SPLIT2),
                                   (1, 12, 512, 2048, api.FLAT_VARIANT_TC2_HALVES_SPLIT2), (1, 8, 256, 2048, api.FLAT_VARIANT_TC2_HALVES_SPLIT4),
                                   (1, 24, 512, 1024, api.FLAT_VARIANT_TC2_HALVES), (1, 34, 512, 512, api.FLAT_VARIANT_TC2_SINGLE),
                                   (1, 2, 128, 128, api.FLAT_VARIANT_TC2_SINGLE)]:
        Qb, Kb, Vb = rand_bits(rng, (B, H, Nq, 64)), rand_bits(rng, (B, H, Nk, 64)), rand_bits(rng, (B, H, Nk, 64))
        ref = oracle.attention(Qb, Kb, Vb, 0.125)["O"]
        O, _ = run(api, Qb, Kb, Vb, 0.125, api.FLAT_VARIANT_AUTO)
        assert api.flat_attn_last_variant() == expect, (B, H, Nq, Nk)
        check_bf16(O, ref, "auto split %s" % ((B, H, Nq, Nk),))


@pytest.mark.parametrize("variant", [8, 9, 10, 15])      # (the two-warpgroup form is built for d = 64; 15: clusters of sixteen)
@pytest.mark.parametrize("shape", [(1, 2, 128, 128), (2, 2, 200, 333), (1, 3, 300, 2100), (1, 1, 77, 4096)])
def test_head_size_128(api, shape, variant):
    B, H, Nq, Nk = shape
    rng = np.random.default_rng(Nq + Nk + variant + 128)
    Qb, Kb, Vb = rand_bits(rng, (B, H, Nq, 128)), rand_bits(rng, (B, H, Nk, 128)), rand_bits(rng, (B, H, Nk, 128))
    vl = np.array([Nk, Nk // 2], dtype=np.int32)[:B]
    for causal in (False, True):
        ref = oracle.attention(Qb, Kb, Vb, 128 ** -0.5, valid_len=vl, causal=causal, want_lse=True)
        O, lse = run(api, Qb, Kb, Vb, 128 ** -0.5, variant, vl=vl, causal=causal)
        assert api.flat_attn_last_variant() == variant
        check_bf16(O, ref["O"], "split d128 v%d %s causal=%d" % (variant, shape, causal))
        fin = np.isfinite(ref["LSE"])
        assert np.array_equal(np.isneginf(lse), np.isneginf(ref["LSE"])) and np.max(np.abs(lse[fin] - ref["LSE"][fin])) < 1e-3


def test_auto_takes_the_split_at_head_size_128(api):
    rng = np.random.default_rng(19)
    for (B, H, Nq, Nk, expect) in [(1, 8, 128, 16384, api.FLAT_VARIANT_TC2_SPLIT8), (1, 8, 512, 4096, api.FLAT_VARIANT_TC2_SPLIT4),
                                   (1, 2, 128, 8192, api.FLAT_VARIANT_TC2_SPLIT16), (4, 16, 2048, 2048, api.FLAT_VARIANT_TC2)]:
        Qb, Kb, Vb = rand_bits(rng, (B, H, Nq, 128)), rand_bits(rng, (B, H, Nk, 128)), rand_bits(rng, (B, H, Nk, 128))
        rows = inputs.sample_rows(inputs.Workload("x", B, H, Nq, Nk, 128), 4)
        ref = oracle.attention(Qb, Kb, Vb, 0.1, rows=rows)["O"]
        O, _ = run(api, Qb, Kb, Vb, 0.1, api.FLAT_VARIANT_AUTO)
        assert api.flat_attn_last_variant() == expect, (B, H, Nq, Nk)
        check_bf16(O.reshape(-1, 128)[rows], ref, "auto split d128 %s" % ((B, H, Nq, Nk),))


def test_refusals(api):
    Q = torch.zeros(1, 1, 128, 32, device="cuda", dtype=torch.bfloat16)
    with pytest.raises(api.FlatAttnError):               # d = 32
        api.flat_attn_fwd_ex(Q, Q, Q, torch.empty_like(Q), 1.0, variant=api.FLAT_VARIANT_TC2_SPLIT2)
    Q64 = torch.zeros(1, 1, 128, 64, device="cuda", dtype=torch.bfloat16)
    bias = torch.zeros(1, 1, 128, 128, device="cuda", dtype=torch.bfloat16)
    with pytest.raises(api.FlatAttnError):               # no bias operand in the split kernel
        api.flat_attn_fwd_ex(Q64, Q64, Q64, torch.empty_like(Q64), 1.0, variant=api.FLAT_VARIANT_TC2_SPLIT4, bias=bias)
    with pytest.raises(api.FlatAttnError):
        api.flat_attn_fwd_ex(Q64, Q64, Q64, torch.empty_like(Q64), 1.0, variant=api.FLAT_VARIANT_TC2_HALVES, bias=bias)
    Q128 = torch.zeros(1, 1, 128, 128, device="cuda", dtype=torch.bfloat16)
    with pytest.raises(api.FlatAttnError):               # the two-warpgroup form: d = 64 only
        api.flat_attn_fwd_ex(Q128, Q128, Q128, torch.empty_like(Q128), 1.0, variant=api.FLAT_VARIANT_TC2_HALVES_SPLIT2)


def test_cluster_launch_in_a_cuda_graph(api):
    rng = np.random.default_rng(13)
    Qb, Kb, Vb = rand_bits(rng, (1, 4, 256, 64)), rand_bits(rng, (1, 4, 1536, 64)), rand_bits(rng, (1, 4, 1536, 64))
    ref = oracle.attention(Qb, Kb, Vb, 0.125)["O"]
    Q, K, V = bf16_tensor(Qb), bf16_tensor(Kb), bf16_tensor(Vb)
    O = torch.zeros(Q.shape, dtype=torch.bfloat16, device="cuda")
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        api.flat_attn_fwd_ex(Q, K, V, O, 0.125, variant=api.FLAT_VARIANT_TC2_SPLIT4, stream=s.cuda_stream)   # warm-up
        s.synchronize()
        O.zero_()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            api.flat_attn_fwd_ex(Q, K, V, O, 0.125, variant=api.FLAT_VARIANT_TC2_SPLIT4, stream=s.cuda_stream)
        assert float(O.float().abs().max()) == 0.0       # capture ran nothing
        g.replay()
        s.synchronize()
    check_bf16(bf16_to_f64(O), ref, "split in a graph")


@pytest.mark.parametrize("variant", [4, 8, 9, 11, 12])
def test_back_to_back_launches_that_depend_on_each_other(api, variant):
    """The one-tile kernels let the next kernel of the stream start its set-up early (programmatic dependent launch)
    and wait for their predecessor before the first access to device memory.  A chain in which every call reads
    the previous call's output -- and the third call overwrites the first call's input -- must give the bits of the
    same chain run with a device synchronisation after every call."""
    rng = np.random.default_rng(77)
    B, H, Nq, Nk = 1, 6, 512, 512
    Qb, Kb, Vb = rand_bits(rng, (B, H, Nq, 64)), rand_bits(rng, (B, H, Nk, 64)), rand_bits(rng, (B, H, Nk, 64))
    K, V = bf16_tensor(Kb), bf16_tensor(Vb)

    def chain(sync):
        X = bf16_tensor(Qb).clone()
        Y = torch.zeros_like(X)
        Z = torch.zeros_like(X)
        for _ in range(4):
            api.flat_attn_fwd_ex(X, K, V, Y, 0.125, variant=variant)      # Y = f(X)
            if sync: torch.cuda.synchronize()
            api.flat_attn_fwd_ex(Y, K, V, Z, 0.125, variant=variant)      # Z = f(Y)
            if sync: torch.cuda.synchronize()
            api.flat_attn_fwd_ex(Z, K, V, X, 0.125, variant=variant)      # X = f(Z): overwrites the first call's input
            if sync: torch.cuda.synchronize()
        torch.cuda.synchronize()
        return X.view(torch.int16).clone(), Y.view(torch.int16).clone(), Z.view(torch.int16).clone()

    ref = chain(True)
    for _ in range(3):
        got = chain(False)
        for a, b in zip(ref, got):
            assert torch.equal(a, b)
    # and the first link against the oracle
    O = torch.zeros(B, H, Nq, 64, dtype=torch.bfloat16, device="cuda")
    api.flat_attn_fwd_ex(bf16_tensor(Qb), K, V, O, 0.125, variant=variant)
    torch.cuda.synchronize()
    check_bf16(bf16_to_f64(O), oracle.attention(Qb, Kb, Vb, 0.125)["O"], "chain link v%d" % variant)


@pytest.mark.parametrize("variant", [11, 12, 14])
def test_two_warpgroup_form_repeated_launches_on_a_masked_batch(api, variant):
    """Every key tile of the two-warpgroup form has one consumer, and the stage a tile lands in must always belong to
    that consumer: with a ring whose depth is odd a warpgroup that ran ahead could mistake its previous tile's
    completion for the next one's (seen as a wrong row in about one launch in fifty on this shape, then a stuck ring).
    Many launches of a batch with unequal valid lengths must all give the same bits, and those bits must be right."""
    B, H, Nq, Nk = 8, 7, 128, 6955
    rng = np.random.default_rng(53)
    Qb, Kb, Vb = rand_bits(rng, (B, H, Nq, 64)), rand_bits(rng, (B, H, Nk, 64)), rand_bits(rng, (B, H, Nk, 64))
    vl = np.array([3712, 6753, 3835, 5265, 6669, 4554, 6216, 4632], dtype=np.int32)
    rows = inputs.sample_rows(inputs.Workload("x", B, H, Nq, Nk, 64), 8)
    ref = oracle.attention(Qb, Kb, Vb, 0.125, valid_len=vl, rows=rows)["O"]
    Q, K, V, vlt = bf16_tensor(Qb), bf16_tensor(Kb), bf16_tensor(Vb), torch.from_numpy(vl).cuda()
    n = 160
    status = torch.zeros(n, dtype=torch.int32, device="cuda")
    outs = [torch.empty(Q.shape, dtype=torch.bfloat16, device="cuda") for _ in range(4)]
    first = None
    for it in range(n):
        api.flat_attn_fwd_ex(Q, K, V, outs[it % 4], 0.125, k_valid_len=vlt, status=status[it:it + 1], variant=variant)
        if it % 4 == 3:
            torch.cuda.synchronize()
            if first is None:
                first = outs[0].clone()
                check_bf16(bf16_to_f64(first).reshape(-1, 64)[rows], ref, "two warpgroups, variant %d" % variant)
            for o in outs:
                assert torch.equal(o, first), "launch %d differs" % it
    assert int(status.abs().max().item()) == 0
