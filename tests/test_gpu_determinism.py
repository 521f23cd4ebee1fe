"""Repeated launches: every kernel of the library walks its tiles in a fixed order and merges partial results in
a fixed order, so the same call must give the same bits every time, and no launch may leave a device code behind.
A race between the roles of a CTA (a barrier phase taken for another, a ring stage reused too early) shows up
here as a launch whose output differs, long before it shows up as a parity failure."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

C5_VALID = [11861, 11425, 10456, 12051, 9350, 16376, 12309, 13716]

# (B, H, Nq, Nk, d, variant, valid_len, causal, dtype, launches)
FORWARD = [
    (8, 12, 1024, 16384, 64, 0, C5_VALID, False, torch.bfloat16, 40),            # even deal (teams of four CTAs)
    (4, 12, 1024, 4096, 64, 0, [4096, 1, 0, 2000], False, torch.bfloat16, 80),
    (3, 7, 700, 6000, 64, 0, [6000, 129, 5999], False, torch.bfloat16, 80),      # two warpgroups per tile
    (8, 7, 128, 6955, 64, 12, [3712, 6753, 3835, 5265, 6669, 4554, 6216, 4632], False, torch.bfloat16, 120),
    (1, 1, 128, 16384, 64, 0, None, False, torch.bfloat16, 80),                  # ... over a cluster of sixteen
    (1, 37, 1024, 3000, 64, 5, None, False, torch.bfloat16, 80),                 # one CTA per item
    (4, 16, 4096, 4096, 64, 0, None, False, torch.bfloat16, 24),                 # persistent CTAs
    (4, 16, 4096, 4096, 64, 0, None, True, torch.bfloat16, 24),                  # ... paired under the causal mask
    (2, 8, 2048, 2048, 128, 0, None, False, torch.bfloat16, 60),                 # d = 128, tiles taking turns
    (4, 8, 1024, 4096, 128, 0, [4096, 1000, 3000, 77], True, torch.bfloat16, 60),
    (1, 8, 128, 16384, 128, 0, None, False, torch.bfloat16, 60),                 # keys over clusters of eight
    (1, 1, 128, 32768, 128, 0, None, False, torch.bfloat16, 60),                 # ... of sixteen
    (4, 16, 2048, 2048, 64, 0, None, False, torch.float32, 16),                  # split tf32
    (2, 4, 1000, 3000, 64, 0, [3000, 1234], False, torch.float32, 16),
]


@pytest.fixture(scope="module")
def api():
    from paper_2107_06419_b200 import api as _api
    return _api


@pytest.mark.parametrize("case", FORWARD, ids=lambda c: "B%dH%dq%dk%dd%d_v%d%s%s_%s" % (
    c[0], c[1], c[2], c[3], c[4], c[5], "m" if c[6] else "", "c" if c[7] else "", str(c[8])[6:]))
def test_forward_launches_repeat_bit_for_bit(api, case):
    B, H, Nq, Nk, d, variant, vl, causal, dtype, n = case
    g = torch.Generator(device="cuda").manual_seed(B * 1000 + Nk)
    Q = torch.randn(B, H, Nq, d, device="cuda", dtype=dtype, generator=g)
    K = torch.randn(B, H, Nk, d, device="cuda", dtype=dtype, generator=g)
    V = torch.randn(B, H, Nk, d, device="cuda", dtype=dtype, generator=g)
    vlt = None if vl is None else torch.tensor(vl, dtype=torch.int32, device="cuda")
    status = torch.zeros(n, dtype=torch.int32, device="cuda")
    outs = [torch.empty_like(Q) for _ in range(4)]       # four launches in flight between synchronisations
    first = None
    for it in range(n):
        api.flat_attn_fwd_ex(Q, K, V, outs[it % 4], d ** -0.5, k_valid_len=vlt, status=status[it:it + 1], variant=variant,
                             causal=causal)
        if it % 4 == 3:
            torch.cuda.synchronize()
            if first is None:
                first = outs[0].clone()
                assert bool(torch.isfinite(first.float()).all())
            for k, o in enumerate(outs):
                assert torch.equal(o, first), "launch %d differs from the first" % (it - 3 + k)
    assert int(status.abs().max().item()) == 0, [hex(c) for c in status.cpu().numpy().tolist() if c]


@pytest.mark.parametrize("case", [(4, 16, 2048, 64, None, False), (2, 8, 2048, 64, [2048, 1000], False),
                                  (2, 8, 2048, 64, None, True), (2, 4, 2048, 128, None, False)],
                         ids=lambda c: "B%dH%dN%dd%d%s%s" % (c[0], c[1], c[2], c[3], "m" if c[4] else "", "c" if c[5] else ""))
def test_backward_launches_repeat_bit_for_bit(api, case):
    B, H, N, d, vl, causal = case
    g = torch.Generator(device="cuda").manual_seed(N + d)
    mk = lambda: torch.randn(B, H, N, d, device="cuda", dtype=torch.bfloat16, generator=g)
    Q, K, V, dO = mk(), mk(), mk(), mk()
    O = torch.empty_like(Q)
    lse = torch.empty(B, H, N, dtype=torch.float32, device="cuda")
    delta = torch.empty_like(lse)
    vlt = None if vl is None else torch.tensor(vl, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.flat_attn_fwd_ex(Q, K, V, O, d ** -0.5, k_valid_len=vlt, status=status, lse=lse, causal=causal)
    first = None
    for it in range(24):
        dQ, dK, dV = torch.empty_like(Q), torch.empty_like(Q), torch.empty_like(Q)
        api.flat_attn_bwd_ex(Q, K, V, O, dO, lse, dQ, dK, dV, delta, d ** -0.5, k_valid_len=vlt, status=status, causal=causal)
        torch.cuda.synchronize()
        if first is None:
            first = (dQ, dK, dV)
        else:
            assert all(torch.equal(a, b) for a, b in zip(first, (dQ, dK, dV))), "launch %d differs" % it
    assert int(status.item()) == 0


def _repeat(fn, n):
    first = None
    for it in range(n):
        out = fn()
        torch.cuda.synchronize()
        if first is None:
            first = [o.clone() for o in out]
        else:
            assert all(torch.equal(a, b) for a, b in zip(first, out)), "launch %d differs" % it


@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("causal", [False, True])
def test_packed_batches_repeat_bit_for_bit(api, d, causal):
    H, lens = 8, [3900, 777, 5000, 128, 2049, 1]
    cu = torch.tensor(np.concatenate([[0], np.cumsum(lens)]), dtype=torch.int32, device="cuda")
    g = torch.Generator(device="cuda").manual_seed(d)
    mk = lambda: torch.randn(sum(lens), H, d, device="cuda", dtype=torch.bfloat16, generator=g)
    Q, K, V = mk(), mk(), mk()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")

    def call():
        O = torch.empty_like(Q)
        api.flat_attn_varlen_fwd(Q, K, V, O, cu, cu, max(lens), d ** -0.5, causal=causal, status=status)
        return [O]
    _repeat(call, 30)
    assert int(status.item()) == 0


def test_bias_pruned_and_layer_calls_repeat_bit_for_bit(api):
    B, H, Nq, Nk = 2, 8, 1024, 2048
    g = torch.Generator(device="cuda").manual_seed(7)
    Q = torch.randn(B, H, Nq, 64, device="cuda", dtype=torch.bfloat16, generator=g)
    K = torch.randn(B, H, Nk, 64, device="cuda", dtype=torch.bfloat16, generator=g)
    V = torch.randn(B, H, Nk, 64, device="cuda", dtype=torch.bfloat16, generator=g)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for shape, dt in (((1, H, Nq, Nk), torch.bfloat16), ((B, H, Nq, Nk), torch.bfloat16), ((1, 1, Nq, Nk), torch.float32)):
        bias = torch.randn(*shape, device="cuda", dtype=dt, generator=g)

        def call():
            O = torch.empty_like(Q)
            api.flat_attn_fwd_ex(Q, K, V, O, 0.125, status=status, bias=bias)
            return [O]
        _repeat(call, 20)
    keep = (torch.rand(1, H, Nq // 128, Nk // 128, device="cuda", generator=g) < 0.5).to(torch.uint8)
    keep[..., 0] = 1

    def pruned():
        O = torch.empty_like(Q)
        api.flat_attn_fwd_ex(Q, K, V, O, 0.125, status=status, block_mask=keep)
        return [O]
    _repeat(pruned, 20)
    Bn, N, Hh, dd, Dm = 2, 1024, 8, 64, 512
    X = torch.randn(Bn, N, Dm, device="cuda", dtype=torch.bfloat16, generator=g) * 0.5
    Wqkv = torch.randn(3 * Hh * dd, Dm, device="cuda", dtype=torch.bfloat16, generator=g) * 0.05
    Wo = torch.randn(Dm, Hh * dd, device="cuda", dtype=torch.bfloat16, generator=g) * 0.05

    def layer():
        Y = torch.empty_like(X)
        bufs = [torch.empty(Bn, Hh, N, dd, device="cuda", dtype=torch.bfloat16) for _ in range(4)]
        api.flat_attn_layer_fwd(X, Wqkv, Wo, Y, *bufs, 0.125, status=status)
        return [Y]
    _repeat(layer, 12)
    assert int(status.item()) == 0
