"""Pruned (block-sparse) Logit-Attend: the one-tile tensor-core kernel walking its query tile's list of kept
key tiles, against the oracle, element by element."""
import numpy as np
import pytest
import torch

import oracle
from paper_2107_06419_b200 import inputs
from helpers import bf16_tensor, bf16_to_f64, check_bf16, rand_bits

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def api():
    from paper_2107_06419_b200 import api as _api
    return _api


def run(api, Qb, Kb, Vb, scale, mask, vl=None, causal=False, want_lse=False):
    Q, K, V = bf16_tensor(Qb), bf16_tensor(Kb), bf16_tensor(Vb)
    O = torch.full(Q.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    lse = torch.full(Q.shape[:3], float("nan"), dtype=torch.float32, device="cuda") if want_lse else None
    api.flat_attn_fwd_ex(Q, K, V, O, scale, k_valid_len=None if vl is None else torch.from_numpy(vl).cuda(),
                         status=status, causal=causal, block_mask=torch.from_numpy(mask).cuda(), lse=lse)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert api.flat_attn_last_variant() == api.FLAT_VARIANT_TC2_SINGLE
    return bf16_to_f64(O), (None if lse is None else lse.cpu().numpy())


def random_mask(rng, lead, tq, tk, density=0.5):
    m = (rng.random(lead + (tq, tk)) < density).astype(np.uint8)
    return m


@pytest.mark.parametrize("shape", [(2, 3, 300, 900, 64), (1, 2, 1024, 1024, 64), (2, 2, 200, 700, 128), (1, 2, 640, 2048, 128)])
@pytest.mark.parametrize("lead", ["full", "per_head", "per_batch", "one"])
def test_random_half_pruned(api, shape, lead):
    B, H, Nq, Nk, d = shape
    rng = np.random.default_rng(sum(shape) + len(lead))
    Qb, Kb, Vb = (rand_bits(rng, s) for s in ((B, H, Nq, d), (B, H, Nk, d), (B, H, Nk, d)))
    ls = {"full": (B, H), "per_head": (1, H), "per_batch": (B, 1), "one": (1, 1)}[lead]
    m = random_mask(rng, ls, -(-Nq // 128), -(-Nk // 128))
    m[..., -1, :] = 0                                    # the last query tile keeps nothing: O = 0 there
    got, lse = run(api, Qb, Kb, Vb, d ** -0.5, m, want_lse=True)
    ref = oracle.attention(Qb, Kb, Vb, d ** -0.5, block_mask=m, want_lse=True)
    check_bf16(got, ref["O"], "sparse %s %s" % (shape, lead))
    dead = np.isneginf(ref["LSE"])
    assert np.array_equal(np.isneginf(lse), dead) and np.abs(lse[~dead] - ref["LSE"][~dead]).max() <= 1e-3
    assert np.all(got[:, :, (Nq - 1) // 128 * 128:] == 0)
    assert np.abs(ref["O"] - oracle.attention(Qb, Kb, Vb, d ** -0.5)["O"]).max() > 0.05      # pruning matters


@pytest.mark.parametrize("d", [64, 128])
def test_pruning_with_the_other_masks_and_dense_map(api, d):
    B, H, Nq, Nk = 2, 2, 520, 520
    rng = np.random.default_rng(d)
    Qb, Kb, Vb = (rand_bits(rng, s) for s in ((B, H, Nq, d), (B, H, Nk, d), (B, H, Nk, d)))
    m = random_mask(rng, (1, H), 5, 5, density=0.6)
    m[..., np.arange(5), np.arange(5)] = 1               # keep the diagonal so that every causal row has a key
    vl = np.array([520, 300], dtype=np.int32)
    for causal in (False, True):
        got, _ = run(api, Qb, Kb, Vb, 0.125, m, vl=vl, causal=causal)
        check_bf16(got, oracle.attention(Qb, Kb, Vb, 0.125, block_mask=m, valid_len=vl, causal=causal)["O"],
                   "sparse + masks d=%d causal=%d" % (d, causal))
    ones = np.ones((1, 1, 5, 5), dtype=np.uint8)
    got, _ = run(api, Qb, Kb, Vb, 0.125, ones)
    check_bf16(got, oracle.attention(Qb, Kb, Vb, 0.125)["O"], "all blocks kept")


def test_sparse_refusals(api):
    q = torch.zeros(1, 1, 128, 64, dtype=torch.bfloat16, device="cuda")
    m = torch.ones(1, 1, 1, 1, dtype=torch.uint8, device="cuda")
    for variant in (1, 2, 3, 5, 6):
        with pytest.raises(api.FlatAttnError) as e:
            api.flat_attn_fwd_ex(q, q, q, torch.empty_like(q), 1.0, variant=variant, block_mask=m)
        assert e.value.code == 3
    with pytest.raises(api.FlatAttnError) as e:
        api.flat_attn_fwd_ex(q, q, q, torch.empty_like(q), 1.0, block_mask=m, bias=torch.zeros(1, 1, 128, 128, dtype=torch.bfloat16, device="cuda"))
    assert e.value.code == 3
    qf = q.float()
    with pytest.raises(api.FlatAttnError) as e:
        api.flat_attn_fwd_ex(qf, qf, qf, torch.empty_like(qf), 1.0, block_mask=m)
    assert e.value.code == 3


def test_c2_half_pruned_sampled_rows_and_time(api):
    """c2 with a seeded random half of the 128 x 128 blocks pruned (the setting of the paper's Section 8.2
    at block granularity): sampled rows against the oracle, and the time against the dense call."""
    w = inputs.WORKLOADS["c2_bert_large_4k"]
    Qb, Kb, Vb = inputs.make_qkv_bf16(w)
    rng = np.random.default_rng(2107)
    m = random_mask(rng, (1, w.H), 32, 32)
    m[..., 0] = 1                                        # every row keeps at least its first block
    rows = inputs.sample_rows(w, 8)
    ref = oracle.attention(Qb, Kb, Vb, w.scale, block_mask=m, rows=rows)["O"]
    Q, K, V = bf16_tensor(Qb), bf16_tensor(Kb), bf16_tensor(Vb)
    O = torch.empty_like(Q)
    mt = torch.from_numpy(m).cuda()
    f = lambda **kw: api.flat_attn_fwd_ex(Q, K, V, O, w.scale, **kw)
    def ms(**kw):
        for _ in range(3):
            f(**kw)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize(); e0.record()
        for _ in range(10):
            f(**kw)
        e1.record(); torch.cuda.synchronize()
        return e0.elapsed_time(e1) / 10
    t_sparse = ms(block_mask=mt)
    got = O.view(-1, w.d)[torch.from_numpy(rows).cuda()].float().cpu().numpy().astype(np.float64)
    check_bf16(got, ref, "c2 half pruned")
    t_dense1 = ms(variant=api.FLAT_VARIANT_TC2_SINGLE)
    t_dense = ms()
    print("c2: density %.3f: pruned %.3f ms; dense on the same kernel %.3f ms; dense, dispatcher's kernel %.3f ms"
          % (float(m.mean()), t_sparse, t_dense1, t_dense))
    assert t_sparse < 0.75 * t_dense1                    # the pruned tiles are skipped, not computed and masked
