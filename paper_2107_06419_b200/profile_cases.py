"""One named case of the library, a few launches, for profiler captures (ncu) and quick timings.

    python -m paper_2107_06419_b200.profile_cases CASE [--workload NAME] [--launches N]

CASE: fused | fused_lse | naive | backward | fp32 | bias | layernorm | layer.  The workload is one of
`inputs.WORKLOADS` (default p_4k_small, a quarter of c2: inputs larger than L2, a few hundred MB on the
device); inputs are the seeded generator's.  Prints the mean launch time from CUDA events.  `fp32` runs the
split-tf32 tensor-core kernel at d = 64 (`--variant 1`: the FFMA kernel).
"""
from __future__ import annotations

import argparse

import numpy as np
import torch

from . import api, inputs


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("case", choices=["fused", "fused_lse", "naive", "backward", "fp32", "bias", "layernorm", "layer"])
    ap.add_argument("--workload", default="p_4k_small")
    ap.add_argument("--launches", type=int, default=4)
    ap.add_argument("--variant", type=int, default=0)
    args = ap.parse_args()
    w = inputs.WORKLOADS[args.workload]
    dev = torch.device("cuda")
    Qb, Kb, Vb = inputs.make_qkv_bf16(w)
    t = lambda bits: torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(dev)
    Q, K, V = t(Qb), t(Kb), t(Vb)
    O = torch.empty_like(Q)
    vl = torch.from_numpy(inputs.make_valid_len(w)).to(dev) if w.masked else None
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    flops = float(w.flops)
    if args.case == "fused":
        step = lambda: api.flat_attn_fwd_ex(Q, K, V, O, w.scale, k_valid_len=vl, status=status, variant=args.variant)
    elif args.case == "fused_lse":
        lse = torch.empty((w.B, w.H, w.Nq), dtype=torch.float32, device=dev)
        step = lambda: api.flat_attn_fwd_ex(Q, K, V, O, w.scale, k_valid_len=vl, status=status, variant=args.variant, lse=lse)
    elif args.case == "naive":
        L = torch.empty((w.B, w.H, w.Nq, w.Nk), dtype=torch.float32, device=dev)
        A = torch.empty((w.B, w.H, w.Nq, w.Nk), dtype=torch.bfloat16, device=dev)
        step = lambda: api.flat_attn_naive_fwd_ex(Q, K, V, O, L, A, w.scale, k_valid_len=vl)
    elif args.case == "backward":
        dO = t(inputs.f32_to_bf16_bits(inputs.normal_f32(inputs.DEFAULT_SEED, 5, 0, Qb.size)).reshape(Qb.shape))
        lse = torch.empty((w.B, w.H, w.Nq), dtype=torch.float32, device=dev)
        delta = torch.empty_like(lse)
        dQ, dK, dV = torch.empty_like(Q), torch.empty_like(K), torch.empty_like(K)
        api.flat_attn_fwd_ex(Q, K, V, O, w.scale, k_valid_len=vl, status=status, lse=lse)
        step = lambda: api.flat_attn_bwd_ex(Q, K, V, O, dO, lse, dQ, dK, dV, delta, w.scale, k_valid_len=vl, status=status)
        flops *= 2.5
    elif args.case == "fp32":
        Qf, Kf, Vf = Q.float(), K.float(), V.float()
        Of = torch.empty_like(Qf)
        step = lambda: api.flat_attn_fwd_ex(Qf, Kf, Vf, Of, w.scale, k_valid_len=vl, status=status, variant=args.variant)
    elif args.case == "bias":
        bias = t(inputs.f32_to_bf16_bits(inputs.normal_f32(inputs.DEFAULT_SEED, 6, 0, w.H * w.Nq * w.Nk)).reshape(1, w.H, w.Nq, w.Nk))
        step = lambda: api.flat_attn_fwd_ex(Q, K, V, O, w.scale, k_valid_len=vl, status=status, bias=bias)
    elif args.case == "layernorm":
        # the token-major activations of the workload's layer: [B * Nq, H * d]
        X = Q.view(w.B * w.Nq, w.H * w.d)
        R = torch.empty_like(X).copy_(K.view(-1)[:X.numel()].view_as(X)) if K.numel() >= X.numel() else torch.zeros_like(X)
        Y = torch.empty_like(X)
        g = t(inputs.f32_to_bf16_bits(inputs.normal_f32(inputs.DEFAULT_SEED, 7, 0, w.H * w.d)))
        b = t(inputs.f32_to_bf16_bits(inputs.normal_f32(inputs.DEFAULT_SEED, 8, 0, w.H * w.d)))
        step = lambda: api.flat_layernorm_fwd(X, g, b, Y, residual=R)
        flops = 0.0
    else:  # layer
        Dm = w.H * w.d
        X = t(inputs.f32_to_bf16_bits(inputs.normal_f32(inputs.DEFAULT_SEED, 9, 0, w.B * w.Nq * Dm)).reshape(w.B, w.Nq, Dm))
        Wqkv = t(inputs.f32_to_bf16_bits(inputs.normal_f32(inputs.DEFAULT_SEED, 10, 0, 3 * Dm * Dm) * np.float32(Dm ** -0.5)).reshape(3 * Dm, Dm))
        Wo = t(inputs.f32_to_bf16_bits(inputs.normal_f32(inputs.DEFAULT_SEED, 11, 0, Dm * Dm) * np.float32(Dm ** -0.5)).reshape(Dm, Dm))
        Y = torch.empty_like(X)
        Kl, Vl, Ol = torch.empty_like(Q), torch.empty_like(Q), torch.empty_like(Q)
        step = lambda: api.flat_attn_layer_fwd(X, Wqkv, Wo, Y, Q, Kl, Vl, Ol, w.scale, status=status)
        flops += 2.0 * w.B * w.Nq * Dm * 4 * Dm
    step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.launches):
        step()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.launches
    code = int(status.item())
    print("%s on %s: %.4f ms per call%s, device status %d" % (
        args.case, w.name, ms, (", %.1f TFLOP/s" % (flops / ms / 1e9)) if flops else "", code))
    assert code == 0


if __name__ == "__main__":
    main()
