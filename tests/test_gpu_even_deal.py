"""The even deal of fused_tc3_kernel: few work items of unequal length (key-padding masks), or a last round that
would stay mostly empty, are dealt by key steps -- every CTA takes an equal share, items are cut where a share ends
and the parts of an item are merged through the library's device workspace.  Against the oracle: batches without
a valid key, with one, with all; shapes whose slabs form teams and shapes that are dealt item by item; planted keys
(a part that is lost or merged twice moves the output by O(1)); rising maxima along the keys (every later part has
the larger reference); and the cases in which the library must fall back to the plain deal."""
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


def run(api, Qb, Kb, Vb, scale, vl=None, stream=None, variant=None):
    O = torch.full(Qb.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    kw = {} if stream is None else {"stream": stream}
    api.flat_attn_fwd_ex(bf16_tensor(Qb), bf16_tensor(Kb), bf16_tensor(Vb), O, scale,
                         k_valid_len=None if vl is None else torch.from_numpy(vl).cuda(), status=status,
                         variant=api.FLAT_VARIANT_TC3 if variant is None else variant, **kw)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return bf16_to_f64(O)


def sampled_rows(B, H, Nq, per_head, seed):
    """Rows of the flattened [B*H*Nq] output to check: every head's first and last row and a few in between."""
    rng = np.random.default_rng(seed)
    rows = []
    for bh in range(B * H):
        r = np.unique(np.concatenate([[0, Nq - 1], rng.integers(0, Nq, per_head)]))
        rows.append(bh * Nq + r)
    return np.concatenate(rows).astype(np.int64)


# (B, H, Nq, Nk, valid_len): teams of 4 / 3 / 5 CTAs per head, single items (one slab), 64 batches
MASKED = [
    (4, 12, 1024, 4096, [4096, 1, 0, 2000]),
    (3, 7, 700, 6000, [6000, 129, 5999]),
    (2, 9, 1200, 5000, [5000, 2500]),
    (2, 60, 256, 4096, [100, 4096]),
    (64, 1, 512, 4096, [(i * 131) % 4097 for i in range(64)]),
]


@pytest.mark.parametrize("case", MASKED, ids=lambda c: "B%d_H%d_%dx%d" % c[:4])
def test_masked_batches(api, case):
    B, H, Nq, Nk, vl = case
    rng = np.random.default_rng(Nq + Nk + B)
    Qb, Kb, Vb = rand_bits(rng, (B, H, Nq, 64)), rand_bits(rng, (B, H, Nk, 64)), rand_bits(rng, (B, H, Nk, 64))
    vl = np.array(vl, dtype=np.int32)
    rows = sampled_rows(B, H, Nq, 24, 3)
    ref = oracle.attention(Qb, Kb, Vb, 0.125, valid_len=vl, rows=rows)["O"]
    O = run(api, Qb, Kb, Vb, 0.125, vl=vl)
    assert api.flat_attn_last_schedule() == api.FLAT_SCHEDULE_EVEN_DEAL, case[:4]
    check_bf16(O.reshape(-1, 64)[rows], ref, "even deal %s" % (case[:4],))
    for b in range(B):
        if vl[b] == 0:
            assert np.all(O[b] == 0.0)


def test_unmasked_last_round_mostly_empty(api):
    """200 equal items on a GPU with fewer SMs than that and more than half of it: the second round would be
    a third full."""
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    H = (sms + sms // 3) // 4                            # 4 slabs per head
    B, Nq, Nk = 1, 1024, 3000
    rng = np.random.default_rng(17)
    Qb, Kb, Vb = rand_bits(rng, (B, H, Nq, 64)), rand_bits(rng, (B, H, Nk, 64)), rand_bits(rng, (B, H, Nk, 64))
    rows = sampled_rows(B, H, Nq, 16, 5)
    ref = oracle.attention(Qb, Kb, Vb, 0.125, rows=rows)["O"]
    O = run(api, Qb, Kb, Vb, 0.125)
    assert api.flat_attn_last_schedule() == api.FLAT_SCHEDULE_EVEN_DEAL
    check_bf16(O.reshape(-1, 64)[rows], ref, "even deal, unmasked")


def test_planted_keys_and_rising_maximum(api):
    """Every row's weight sits on one planted key whose position differs from row to row, so the part of the item
    that holds it changes from row to row; then scores that rise along the keys, so that every later part ends on a
    larger reference than the one before it and the merge must rescale."""
    w = inputs.Workload("planted", 2, 12, 1024, 4096, 64, masked=True)
    Qb, Kb, Vb, planted = inputs.make_planted_qkv_bf16(w)
    vl = inputs.make_valid_len(w)                        # (the planted keys lie among each batch's valid keys)
    rows = sampled_rows(w.B, w.H, w.Nq, 24, 7)
    ref = oracle.attention(Qb, Kb, Vb, w.scale, valid_len=vl, rows=rows)["O"]
    O = run(api, Qb, Kb, Vb, w.scale, vl=vl)
    assert api.flat_attn_last_schedule() == api.FLAT_SCHEDULE_EVEN_DEAL
    check_bf16(O.reshape(-1, 64)[rows], ref, "even deal, planted keys")
    rng = np.random.default_rng(5)
    B, H, Nq, Nk = 2, 12, 1024, 4096
    Qf = np.abs(rng.standard_normal((B, H, Nq, 64))).astype(np.float32)
    ramp = (np.arange(Nk, dtype=np.float32) / Nk * 6.0)[None, None, :, None]
    Kf = (np.abs(rng.standard_normal((B, H, Nk, 64))) * 0.2 + ramp * 0.25).astype(np.float32)
    Vf = rng.standard_normal((B, H, Nk, 64)).astype(np.float32)
    Qb2, Kb2, Vb2 = (inputs.f32_to_bf16_bits(x).reshape(x.shape) for x in (Qf, Kf, Vf))
    ref2 = oracle.attention(Qb2, Kb2, Vb2, 0.5, valid_len=vl, rows=rows)["O"]
    O2 = run(api, Qb2, Kb2, Vb2, 0.5, vl=vl)
    assert api.flat_attn_last_schedule() == api.FLAT_SCHEDULE_EVEN_DEAL
    check_bf16(O2.reshape(-1, 64)[rows], ref2, "even deal, rising maximum")


def test_same_bits_as_the_plain_deal_where_no_item_is_cut(api):
    """A CTA that holds a whole item runs the ordinary epilogue; the rows of items that were not cut must match a
    launch of the other d = 64 kernel to bf16 rounding, and all rows must agree within the parity bar."""
    B, H, Nq, Nk = 4, 12, 1024, 4096
    rng = np.random.default_rng(23)
    Qb, Kb, Vb = rand_bits(rng, (B, H, Nq, 64)), rand_bits(rng, (B, H, Nk, 64)), rand_bits(rng, (B, H, Nk, 64))
    vl = np.array([4096, 3000, 2000, 1000], dtype=np.int32)
    O = run(api, Qb, Kb, Vb, 0.125, vl=vl)
    assert api.flat_attn_last_schedule() == api.FLAT_SCHEDULE_EVEN_DEAL
    O2 = run(api, Qb, Kb, Vb, 0.125, vl=vl, variant=api.FLAT_VARIANT_TC2)
    assert np.max(np.abs(O - O2)) <= 2e-2
    assert np.mean(np.abs(O - O2)) <= 2e-4


def test_falls_back_to_the_plain_deal(api):
    rng = np.random.default_rng(29)
    B, H, Nq, Nk = 4, 12, 1024, 4096
    Qb, Kb, Vb = rand_bits(rng, (B, H, Nq, 64)), rand_bits(rng, (B, H, Nk, 64)), rand_bits(rng, (B, H, Nk, 64))
    vl = np.array([4096, 3000, 2000, 1000], dtype=np.int32)
    rows = sampled_rows(B, H, Nq, 8, 11)
    ref = oracle.attention(Qb, Kb, Vb, 0.125, valid_len=vl, rows=rows)["O"]
    Q, K, V, vlt = bf16_tensor(Qb), bf16_tensor(Kb), bf16_tensor(Vb), torch.from_numpy(vl).cuda()
    # during stream capture: a captured launch could be replayed beside anything, so it never uses the workspace
    O = torch.zeros(Q.shape, dtype=torch.bfloat16, device="cuda")
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        api.flat_attn_fwd_ex(Q, K, V, O, 0.125, k_valid_len=vlt, variant=api.FLAT_VARIANT_TC3, stream=s.cuda_stream)
        s.synchronize()
        assert api.flat_attn_last_schedule() == api.FLAT_SCHEDULE_EVEN_DEAL
        O.zero_()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            api.flat_attn_fwd_ex(Q, K, V, O, 0.125, k_valid_len=vlt, variant=api.FLAT_VARIANT_TC3, stream=s.cuda_stream)
        assert api.flat_attn_last_schedule() == api.FLAT_SCHEDULE_ITEMS
        g.replay()
        s.synchronize()
    check_bf16(bf16_to_f64(O).reshape(-1, 64)[rows], ref, "captured launch")
    # a second stream while the first stream's launch may still be running: the plain deal, and both are right
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    O1, O2 = torch.zeros_like(O), torch.zeros_like(O)
    torch.cuda.synchronize()
    api.flat_attn_fwd_ex(Q, K, V, O1, 0.125, k_valid_len=vlt, variant=api.FLAT_VARIANT_TC3, stream=s1.cuda_stream)
    first = api.flat_attn_last_schedule()
    api.flat_attn_fwd_ex(Q, K, V, O2, 0.125, k_valid_len=vlt, variant=api.FLAT_VARIANT_TC3, stream=s2.cuda_stream)
    second = api.flat_attn_last_schedule()
    torch.cuda.synchronize()
    assert first == api.FLAT_SCHEDULE_EVEN_DEAL
    assert second in (api.FLAT_SCHEDULE_ITEMS, api.FLAT_SCHEDULE_EVEN_DEAL)   # (even deal only if the first had finished)
    check_bf16(bf16_to_f64(O1).reshape(-1, 64)[rows], ref, "first stream")
    check_bf16(bf16_to_f64(O2).reshape(-1, 64)[rows], ref, "second stream")
    # the causal mask, the lse output and more than 64 batches keep the plain deal
    api.flat_attn_fwd_ex(Q, K, V, O, 0.125, k_valid_len=vlt, variant=api.FLAT_VARIANT_TC3, causal=True)
    assert api.flat_attn_last_schedule() == api.FLAT_SCHEDULE_ITEMS
    lse = torch.empty(Q.shape[:3], dtype=torch.float32, device="cuda")
    api.flat_attn_fwd_ex(Q, K, V, O, 0.125, k_valid_len=vlt, variant=api.FLAT_VARIANT_TC3, lse=lse)
    assert api.flat_attn_last_schedule() == api.FLAT_SCHEDULE_ITEMS
    torch.cuda.synchronize()
    B2 = 65
    Qb2, Kb2, Vb2 = rand_bits(rng, (B2, 1, 512, 64)), rand_bits(rng, (B2, 1, 4096, 64)), rand_bits(rng, (B2, 1, 4096, 64))
    vl2 = np.full(B2, 4096, dtype=np.int32)
    O3 = run(api, Qb2, Kb2, Vb2, 0.125, vl=vl2)
    assert api.flat_attn_last_schedule() == api.FLAT_SCHEDULE_ITEMS
    rows2 = sampled_rows(B2, 1, 512, 4, 13)
    check_bf16(O3.reshape(-1, 64)[rows2], oracle.attention(Qb2, Kb2, Vb2, 0.125, valid_len=vl2, rows=rows2)["O"], "65 batches")


def test_many_launches_in_a_row(api):
    """The flags of the workspace carry the epoch of the launch that wrote them and are never reset: a chain of
    launches of different shapes on one stream must not see one another's parts."""
    rng = np.random.default_rng(31)
    shapes = [(4, 12, 1024, 4096), (2, 9, 1200, 5000), (4, 12, 1024, 4096), (3, 7, 700, 6000)]
    outs = []
    for (B, H, Nq, Nk) in shapes * 3:
        Qb, Kb, Vb = rand_bits(rng, (B, H, Nq, 64)), rand_bits(rng, (B, H, Nk, 64)), rand_bits(rng, (B, H, Nk, 64))
        vl = rng.integers(Nk // 2, Nk + 1, B).astype(np.int32)
        O = torch.full(Qb.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        api.flat_attn_fwd_ex(bf16_tensor(Qb), bf16_tensor(Kb), bf16_tensor(Vb), O, 0.125,
                             k_valid_len=torch.from_numpy(vl).cuda(), status=status, variant=api.FLAT_VARIANT_TC3)
        assert api.flat_attn_last_schedule() == api.FLAT_SCHEDULE_EVEN_DEAL
        outs.append((Qb, Kb, Vb, vl, O, status))         # (no synchronisation between the launches)
    torch.cuda.synchronize()
    for i, (Qb, Kb, Vb, vl, O, status) in enumerate(outs):
        assert int(status.item()) == 0
        B, H, Nq, _ = Qb.shape
        rows = sampled_rows(B, H, Nq, 6, i)
        ref = oracle.attention(Qb, Kb, Vb, 0.125, valid_len=vl, rows=rows)["O"]
        check_bf16(bf16_to_f64(O).reshape(-1, 64)[rows], ref, "launch %d of the chain" % i)


def test_two_host_threads_on_two_streams(api):
    """The workspace is one per device: launches from two host threads on two streams must never share it while
    one of them may still be running (the second falls back to the plain deal), and every result must be right."""
    import threading
    rng = np.random.default_rng(37)
    jobs = []
    for (B, H, Nq, Nk) in [(4, 12, 1024, 4096), (2, 9, 1200, 5000)]:
        Qb, Kb, Vb = rand_bits(rng, (B, H, Nq, 64)), rand_bits(rng, (B, H, Nk, 64)), rand_bits(rng, (B, H, Nk, 64))
        vl = rng.integers(Nk // 2, Nk + 1, B).astype(np.int32)
        rows = sampled_rows(B, H, Nq, 6, 41)
        ref = oracle.attention(Qb, Kb, Vb, 0.125, valid_len=vl, rows=rows)["O"]
        jobs.append((bf16_tensor(Qb), bf16_tensor(Kb), bf16_tensor(Vb), torch.from_numpy(vl).cuda(), rows, ref))
    torch.cuda.synchronize()
    results, errors, schedules = [[], []], [], [[], []]

    def worker(k):
        try:
            Q, K, V, vlt, rows, ref = jobs[k]
            s = torch.cuda.Stream()
            for _ in range(12):
                O = torch.full(Q.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
                status = torch.zeros(1, dtype=torch.int32, device="cuda")
                s.wait_stream(torch.cuda.current_stream())
                api.flat_attn_fwd_ex(Q, K, V, O, 0.125, k_valid_len=vlt, status=status, variant=api.FLAT_VARIANT_TC3,
                                     stream=s.cuda_stream)
                schedules[k].append(api.flat_attn_last_schedule())
                results[k].append((O, status))
            s.synchronize()
        except Exception as e:                           # (surfaces in the main thread)
            errors.append(e)

    threads = [threading.Thread(target=worker, args=(k,)) for k in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    torch.cuda.synchronize()
    assert not errors, errors
    for k in range(2):
        rows, ref = jobs[k][4], jobs[k][5]
        assert all(x in (api.FLAT_SCHEDULE_ITEMS, api.FLAT_SCHEDULE_EVEN_DEAL) for x in schedules[k])
        for O, status in results[k]:
            assert int(status.item()) == 0
            check_bf16(bf16_to_f64(O).reshape(-1, 64)[rows], ref, "thread %d" % k)


def test_while_another_stream_holds_sms(api):
    """The launch is not a cooperative one: when another stream's kernels hold SMs, some CTAs start late and a CTA
    that waits for another's part may spin for a while.  Every launch must still finish without a device code and
    with the bits of an undisturbed launch."""
    w = inputs.WORKLOADS["c5_cross_masked"]
    g = torch.Generator(device="cuda").manual_seed(43)
    Q = torch.randn(w.B, w.H, w.Nq, 64, device="cuda", dtype=torch.bfloat16, generator=g)
    K = torch.randn(w.B, w.H, w.Nk, 64, device="cuda", dtype=torch.bfloat16, generator=g)
    V = torch.randn(w.B, w.H, w.Nk, 64, device="cuda", dtype=torch.bfloat16, generator=g)
    vlt = torch.from_numpy(inputs.make_valid_len(w)).cuda()
    ref = torch.empty_like(Q)
    status0 = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.flat_attn_fwd_ex(Q, K, V, ref, w.scale, k_valid_len=vlt, status=status0, variant=api.FLAT_VARIANT_TC3)
    torch.cuda.synchronize()
    assert api.flat_attn_last_schedule() == api.FLAT_SCHEDULE_EVEN_DEAL and int(status0.item()) == 0
    A = torch.randn(8192, 8192, device="cuda", dtype=torch.bfloat16, generator=g)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    n = 40
    status = torch.zeros(n, dtype=torch.int32, device="cuda")
    outs = []
    for it in range(n):
        with torch.cuda.stream(s1):
            _ = A @ A                                    # (a library GEMM as the disturbance: all SMs for about 0.7 ms)
            _ = A @ A
        O = torch.empty_like(Q)
        api.flat_attn_fwd_ex(Q, K, V, O, w.scale, k_valid_len=vlt, status=status[it:it + 1], variant=api.FLAT_VARIANT_TC3,
                             stream=s2.cuda_stream)
        outs.append(O)
    torch.cuda.synchronize()
    assert int(status.abs().max().item()) == 0, [hex(c) for c in status.cpu().numpy().tolist() if c]
    assert all(torch.equal(o, ref) for o in outs)
