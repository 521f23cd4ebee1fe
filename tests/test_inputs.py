"""The seeded input generator: determinism, slice independence, bf16 rounding, ranges."""
import numpy as np

from paper_2107_06419_b200 import inputs


def test_slices_are_position_independent():
    a = inputs.normal_f32(7, inputs.TENSOR_K, 0, 5000)
    b = inputs.normal_f32(7, inputs.TENSOR_K, 1234, 100)
    assert np.array_equal(a[1234:1334], b)
    assert not np.array_equal(a[:100], inputs.normal_f32(7, inputs.TENSOR_V, 0, 100))
    assert not np.array_equal(a[:100], inputs.normal_f32(8, inputs.TENSOR_K, 0, 100))


def test_normal_moments():
    x = inputs.normal_f32(inputs.DEFAULT_SEED, inputs.TENSOR_Q, 0, 1 << 20).astype(np.float64)
    assert abs(x.mean()) < 5e-3 and abs(x.std() - 1.0) < 5e-3
    assert abs((x ** 3).mean()) < 2e-2 and abs((x ** 4).mean() - 3.0) < 5e-2
    assert np.all(np.isfinite(x)) and np.abs(x).max() < 6.0


def test_bf16_round_to_nearest_even():
    x = np.array([1.0, 1.00390625, 1.01171875, -2.5, 0.0, 3.3895313892515355e38], dtype=np.float32)
    # 1 + 2^-8 is a tie between 1.0 and 1 + 2^-7 -> even mantissa (1.0); 1 + 3*2^-8 ties up to 1 + 2^-6
    b = inputs.f32_to_bf16_bits(x)
    back = inputs.bf16_bits_to_f32(b)
    assert back[0] == 1.0 and back[1] == 1.0 and back[2] == 1.015625 and back[3] == -2.5 and back[4] == 0.0
    r = np.random.default_rng(0).standard_normal(10000).astype(np.float32)
    rb = inputs.bf16_bits_to_f32(inputs.f32_to_bf16_bits(r))
    assert np.all(np.abs(rb - r) <= np.abs(r) * 2.0 ** -8)


def test_valid_len_range_and_sample_rows():
    w = inputs.WORKLOADS["c5_cross_masked"]
    vl = inputs.make_valid_len(w)
    assert vl.dtype == np.int32 and vl.shape == (w.B,)
    assert np.all(vl >= w.Nk // 2) and np.all(vl <= w.Nk)
    assert np.array_equal(vl, inputs.make_valid_len(w))
    small = inputs.Workload("s", 2, 2, 300, 64, 8)
    rows = inputs.sample_rows(small, 16)
    assert rows.shape == (2 * 2 * 16,) and len(np.unique(rows)) == rows.size
    per_head = rows.reshape(4, 16) - (np.arange(4) * 300)[:, None]
    assert np.all(per_head >= 0) and np.all(per_head < 300)
    assert np.all(per_head[:, 0] == 0) and np.all(per_head.max(axis=1) == 299)


def test_workload_table_matches_configurations():
    w = inputs.WORKLOADS
    assert (w["c1_bert_base_512"].B, w["c1_bert_base_512"].H, w["c1_bert_base_512"].Nq, w["c1_bert_base_512"].d) == (1, 12, 512, 64)
    assert w["c2_bert_large_4k"].flops == 4 * 16 * 16 * 4096 * 4096 * 64
    assert w["c4_64k_d128"].qkvo_bytes() == 4 * 8 * 65536 * 128 * 2
    assert abs(w["c4_64k_d128"].scale - 128 ** -0.5) < 1e-8


def test_planted_inputs_shapes():
    w = inputs.Workload("p", 2, 2, 64, 300, 16, masked=True)
    q, k, v, planted = inputs.make_planted_qkv_bf16(w, seed=3)
    vl = inputs.make_valid_len(w, seed=3)
    assert q.shape == (2, 2, 64, 16) and k.shape == v.shape == (2, 2, 300, 16)
    assert planted.shape == (2, 64)
    for b in range(2):
        assert np.all(planted[b] >= 0) and np.all(planted[b] < vl[b])
