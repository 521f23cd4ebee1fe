"""Packed variable-length batches: pins of the oracle (CPU) and parity of the kernel (GPU)."""
import numpy as np
import pytest

import oracle
from paper_2107_06419_b200 import inputs


def rand_bits(rng, shape, sigma=1.0):
    return inputs.f32_to_bf16_bits((rng.standard_normal(shape) * sigma).astype(np.float32)).reshape(shape)


def cu(lengths):
    return np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)


def test_packing_equal_lengths_is_the_batched_definition():
    rng = np.random.default_rng(1)
    B, H, N, d = 3, 2, 7, 4
    Q, K, V = rand_bits(rng, (B, H, N, d)), rand_bits(rng, (B, H, N, d)), rand_bits(rng, (B, H, N, d))
    ref = oracle.attention(Q, K, V, 0.3)["O"]                              # [B, H, N, d]
    pack = lambda t: np.ascontiguousarray(t.transpose(0, 2, 1, 3)).reshape(B * N, H, d)
    got = oracle.attention_varlen(pack(Q), pack(K), pack(V), cu([N] * B), cu([N] * B), 0.3)
    assert np.array_equal(got.reshape(B, N, H, d).transpose(0, 2, 1, 3), ref)


def test_sequences_do_not_see_each_other_and_trivial_sequences():
    rng = np.random.default_rng(2)
    H, d = 2, 4
    lq, lk = [3, 1, 0, 5], [4, 1, 2, 0]                                     # a one-token sequence, one without queries, one without keys
    Q, K, V = rand_bits(rng, (sum(lq), H, d)), rand_bits(rng, (sum(lk), H, d)), rand_bits(rng, (sum(lk), H, d))
    cq, ck = cu(lq), cu(lk)
    O = oracle.attention_varlen(Q, K, V, cq, ck, 1.0)
    # one key: the output is that key's value row, whatever the logit
    v = inputs.bf16_bits_to_f32(V).reshape(V.shape).astype(np.float64)
    assert np.allclose(O[3], v[4], rtol=0, atol=1e-15)
    # no keys: O = 0
    assert np.all(O[4:9] == 0.0)
    # changing the keys of sequence 0 leaves sequence 1 alone
    K2 = K.copy(); K2[0:4] = rand_bits(rng, (4, H, d))
    O2 = oracle.attention_varlen(Q, K2, V, cq, ck, 1.0)
    assert np.array_equal(O2[3], O[3]) and not np.array_equal(O2[0:3], O[0:3])


def test_causal_offset_is_per_sequence():
    rng = np.random.default_rng(3)
    H, d = 1, 2
    lq, lk = [2, 3], [4, 3]
    Q, K, V = rand_bits(rng, (5, H, d)), rand_bits(rng, (7, H, d)), rand_bits(rng, (7, H, d))
    O = oracle.attention_varlen(Q, K, V, cu(lq), cu(lk), 1.0, causal=True)
    # sequence 0: 2 queries, 4 keys: query 0 sees keys 0..2, query 1 all four
    q = np.ascontiguousarray(Q[0:1].transpose(1, 0, 2))[None]
    k = np.ascontiguousarray(K[0:3].transpose(1, 0, 2))[None]; v = np.ascontiguousarray(V[0:3].transpose(1, 0, 2))[None]
    assert np.allclose(O[0], oracle.attention(q, k, v, 1.0)["O"][0, :, 0], rtol=0, atol=1e-15)
    # sequence 1 (square): its first query sees only its first key
    vv = inputs.bf16_bits_to_f32(V).reshape(V.shape).astype(np.float64)
    assert np.allclose(O[2], vv[4], rtol=0, atol=1e-15)


# ---------------------------------------------------------------------------------------------- GPU
VARLEN_CASES = [
    # (query lengths, key lengths or None for the same, H, causal)
    ([300, 1, 128, 129, 517, 256, 77], None, 2, False),
    ([300, 1, 128, 129, 517, 256, 77], None, 2, True),
    ([64, 200, 5], [700, 200, 1], 3, False),                               # cross lengths
    ([64, 200, 5], [700, 260, 9], 3, True),                                # causal with more keys than queries
    ([100, 0, 50], [100, 30, 0], 1, False),                                # a sequence without queries, one without keys
    ([40] * 700, None, 2, False),                                          # many short sequences: the persistent grid
    ([1000, 30, 513] * 40, None, 4, True),                                 # uneven slabs, empty slots, persistent, causal
    ([300, 1, 128, 129, 517, 256, 77], None, 2, False, 128),               # head size 128: the two-tile kernel
    ([300, 1, 128, 129, 517, 256, 77], [300, 5, 700, 129, 517, 300, 77], 2, True, 128),
    ([100, 0, 50, 1000], [100, 30, 0, 900], 3, True, 128),
]


@pytest.mark.gpu
@pytest.mark.parametrize("case", VARLEN_CASES, ids=[str(i) for i in range(len(VARLEN_CASES))])
def test_varlen_against_oracle(case):
    import torch
    from helpers import bf16_tensor, bf16_to_f64, check_bf16
    from paper_2107_06419_b200 import api
    lq, lk, H, causal = case[:4]
    lk = lq if lk is None else lk
    d = case[4] if len(case) > 4 else 64
    rng = np.random.default_rng(sum(lq) + 7 * sum(lk) + H)
    Qb, Kb, Vb = rand_bits(rng, (sum(lq), H, d)), rand_bits(rng, (sum(lk), H, d)), rand_bits(rng, (sum(lk), H, d))
    cq, ck = cu(lq), cu(lk)
    Q, K, V = bf16_tensor(Qb), bf16_tensor(Kb), bf16_tensor(Vb)
    O = torch.full(Q.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    scale = d ** -0.5
    api.flat_attn_varlen_fwd(Q, K, V, O, torch.from_numpy(cq).cuda(), torch.from_numpy(ck).cuda(), max(lq), scale,
                             causal=causal, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = oracle.attention_varlen(Qb, Kb, Vb, cq, ck, scale, causal=causal)
    check_bf16(bf16_to_f64(O), ref, "varlen")


def test_varlen_argument_errors():
    from paper_2107_06419_b200 import api
    f = api._lib.flat_attn_varlen_fwd
    ok = dict(Q=0x10000, K=0x20000, V=0x30000, O=0x40000, cq=0x50000, ck=0x60000, S=3, H=2, d=64, tq=100, tk=120, mq=50,
              scale=0.125, causal=0)
    def call(**kw):
        a = dict(ok, **kw)
        return f(a["Q"], a["K"], a["V"], a["O"], a["cq"], a["ck"], a["S"], a["H"], a["d"], a["tq"], a["tk"], a["mq"],
                 a["scale"], a["causal"], None, None)
    assert call(Q=None) == 1 and call(ck=None) == 1
    assert call(S=0) == 2 and call(tq=0) == 2 and call(mq=101) == 2 and call(scale=float("inf")) == 2
    assert call(d=32) == 3 and call(causal=3) == 3
    assert call(V=0x30008) == 4 and call(cq=0x50002) == 4
