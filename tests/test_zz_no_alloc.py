"""flat_attn_naive_fwd_static: the baseline for callers that cannot allocate device memory
(fixed-budget plugins, loops that must stay out of the driver's allocator).  Its logit and
weight tensors sit in an array inside the library, so the only thing to verify is that it
computes what flat_attn_naive_fwd computes with caller-provided buffers -- on two calls in a
row, because every call reuses the same array and finds the previous call's data in it.

This file is named to be collected last, so a run that stops at the first failure has
already exercised everything else."""
import ctypes

import numpy as np
import pytest
import torch

from helpers import bf16_tensor, rand_bits


@pytest.fixture(scope="module")
def api():
    from paper_2107_06419_b200 import api as _api
    return _api


def test_static_rejects_oversize_without_touching_the_device(api):
    # 16*16*128*128 = 4 Mi elements fits exactly; one more key row per query does not.
    big = (ctypes.c_void_p(0x10000), ctypes.c_void_p(0x20000), ctypes.c_void_p(0x30000), ctypes.c_void_p(0x40000))
    assert api._lib.flat_attn_naive_fwd_static(*big, 16, 16, 128, 129, 64, 1.0, None) == 5
    assert api._lib.flat_attn_naive_fwd_static(*big, 60000, 60000, 2 ** 31 - 1, 2 ** 31 - 1, 64, 1.0, None) == 5
    assert api._lib.flat_attn_naive_fwd_static(*big, 1, 1, 0, 8, 64, 1.0, None) == 2
    # the other argument rules are applied before the device is looked at, too
    assert api._lib.flat_attn_naive_fwd_static(None, big[1], big[2], big[3], 1, 1, 8, 8, 64, 1.0, None) == 1
    assert api._lib.flat_attn_naive_fwd_static(*big, 1, 1, 8, 8, 48, 1.0, None) == 3
    assert api._lib.flat_attn_naive_fwd_static(ctypes.c_void_p(0x10008), big[1], big[2], big[3], 1, 1, 8, 8, 64, 1.0, None) == 4
    assert "workspace" in api.flat_attn_status_string(5)


@pytest.mark.gpu
def test_static_matches_caller_buffer_baseline_twice(api):
    rng = np.random.default_rng(41)
    # second problem is smaller and shaped differently, so it runs over the first one's leftovers
    for (B, H, Nq, Nk, d) in [(2, 4, 333, 700, 64), (1, 3, 130, 257, 128)]:
        Qb, Kb, Vb = rand_bits(rng, (B, H, Nq, d)), rand_bits(rng, (B, H, Nk, d)), rand_bits(rng, (B, H, Nk, d))
        Q, K, V = bf16_tensor(Qb), bf16_tensor(Kb), bf16_tensor(Vb)
        scale = d ** -0.5
        O_ref = torch.full(Q.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
        L = torch.empty((B, H, Nq, Nk), dtype=torch.float32, device="cuda")
        A = torch.empty((B, H, Nq, Nk), dtype=torch.bfloat16, device="cuda")
        api.flat_attn_naive_fwd(Q, K, V, O_ref, L, A, scale)
        O = torch.full(Q.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
        api.flat_attn_naive_fwd_static(Q, K, V, O, scale)
        torch.cuda.synchronize()
        # the same three kernels on the same inputs: anything but identical bits would mean that
        # leftovers of the previous call in the shared array reached the result
        assert bool(torch.isfinite(O.float()).all())
        assert torch.equal(O.view(torch.int16), O_ref.view(torch.int16))
    with pytest.raises(api.FlatAttnError) as e:
        big = torch.zeros((1, 1, 4096, 2048), dtype=torch.bfloat16, device="cuda")[..., :64].contiguous()
        kv = torch.zeros((1, 1, 2048, 64), dtype=torch.bfloat16, device="cuda")
        api.flat_attn_naive_fwd_static(big, kv, kv, torch.empty_like(big), 1.0)
    assert e.value.code == 5
