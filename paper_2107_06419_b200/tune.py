"""Granularity sweep: times every fused kernel variant on a set of shapes (CUDA events).

The paper explores, per workload, how many query rows a fused tile should hold (its R-granularity
trade-off, Section 5.3: fewer rows mean more K/V re-fetches and a worse-filled compute array) and
picks the best mapping by search (Section 6.1).  On B200 the candidates are the compiled kernel
variants: 64-row FFMA tiles, 128-row tensor-core CTAs (one or two per SM; with the keys of a tile split
over a cluster of 2, 4 or 8 CTAs for launches that leave SMs empty) and 256-row CTAs (with one or two
softmax threads per row).

    python -m paper_2107_06419_b200.tune [--workloads c1_bert_base_512,c2_bert_large_4k,...] [--steps 10]
    python -m paper_2107_06419_b200.tune --layer      (the attention layer around the fused path, step by step)
    python -m paper_2107_06419_b200.tune --causal     (the variants under the causal mask)
    python -m paper_2107_06419_b200.tune --varlen     (packed variable-length batches; with --causal too)

Prints one JSON line per (workload, variant) and the winner per workload; the batched sweeps run on
the seeded generator's inputs (the bytes bench.py times), the layer and packed sweeps on random bf16
(timing only -- parity is the tests' business).
"""
from __future__ import annotations

import argparse
import json
import time

import numpy as np
import torch

from . import api, inputs

VARIANTS = {
    api.FLAT_VARIANT_SIMT: "simt: 64-row FFMA tiles",
    api.FLAT_VARIANT_TC: "tc: 128-row CTA, exact running maximum",
    api.FLAT_VARIANT_TC2_SINGLE: "tc2_single: 128-row CTA, two per SM (d = 64)",
    api.FLAT_VARIANT_TC2: "tc2: 256-row CTA (two tiles ping-pong)",
    api.FLAT_VARIANT_TC3: "tc3: 256-row CTA, half-row softmax threads, logits three tile-steps ahead (d = 64)",
    api.FLAT_VARIANT_RGRAN: "rgran: whole logit rows on chip, two-pass softmax (d = 64, Nk <= 512)",
    api.FLAT_VARIANT_TC2_SPLIT2: "tc2_split2: 128-row CTA, keys split over a cluster of 2 CTAs",
    api.FLAT_VARIANT_TC2_SPLIT4: "tc2_split4: ... over a cluster of 4 CTAs",
    api.FLAT_VARIANT_TC2_SPLIT8: "tc2_split8: ... over a cluster of 8 CTAs",
    api.FLAT_VARIANT_TC2_HALVES: "tc2_halves: 128-row CTA, two warpgroups on alternate key tiles (d = 64)",
    api.FLAT_VARIANT_TC2_HALVES_SPLIT2: "tc2_halves_split2: ... and the keys over a cluster of 2 CTAs",
    api.FLAT_VARIANT_TC2_HALVES_SPLIT4: "tc2_halves_split4: ... of 4 CTAs",
    api.FLAT_VARIANT_TC2_HALVES_SPLIT8: "tc2_halves_split8: ... of 8 CTAs",
    api.FLAT_VARIANT_TC2_SPLIT16: "tc2_split16: keys over a cluster of 16 CTAs (d = 128)",
    api.FLAT_VARIANT_TC2_HALVES_SPLIT16: "tc2_halves_split16: two warpgroups per tile, keys over a cluster of 16 CTAs (d = 64)",
    api.FLAT_VARIANT_AUTO: "auto (the dispatcher's choice)",
}


_QKV_CACHE = {}


def _seeded_qkv(w, dev):
    """The workload's inputs from the seeded generator (the bytes that bench.py and the tests use),
    generated once per workload."""
    if w.name not in _QKV_CACHE:
        _QKV_CACHE.clear()
        as_t = lambda bits: torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(dev)
        _QKV_CACHE[w.name] = tuple(as_t(x) for x in inputs.make_qkv_bf16(w))
    return _QKV_CACHE[w.name]


def time_variant(w, variant, steps, warmup=2, causal=False):
    dev = torch.device("cuda")
    Q, K, V = _seeded_qkv(w, dev)
    O = torch.empty_like(Q)
    vl = None
    if w.masked:
        vl = torch.from_numpy(inputs.make_valid_len(w)).to(dev)
    try:
        for _ in range(warmup):
            api.flat_attn_fwd_ex(Q, K, V, O, w.scale, k_valid_len=vl, variant=variant, causal=causal)
    except api.FlatAttnError as e:
        return None, str(e), None
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    # let the power state of the previous variant decay (the long ones reach the power cap), then
    # bring the clocks back up with two launches before timing
    time.sleep(1.0)
    for _ in range(2):
        api.flat_attn_fwd_ex(Q, K, V, O, w.scale, k_valid_len=vl, variant=variant, causal=causal)
    e0.record()
    for _ in range(steps):
        api.flat_attn_fwd_ex(Q, K, V, O, w.scale, k_valid_len=vl, variant=variant, causal=causal)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    if ms > 0.1:
        return ms, None, None
    # short launches: the host cannot issue them as fast as the GPU runs them; replaying a CUDA graph
    # of twenty launches gives the time the GPU itself needs
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        api.flat_attn_fwd_ex(Q, K, V, O, w.scale, k_valid_len=vl, variant=variant, causal=causal)
        s.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=s):
            for _ in range(20):
                api.flat_attn_fwd_ex(Q, K, V, O, w.scale, k_valid_len=vl, variant=variant, causal=causal)
        graph.replay()
        s.synchronize()
        e0.record(s)
        for _ in range(steps):
            graph.replay()
        e1.record(s)
        s.synchronize()
    return ms, None, e0.elapsed_time(e1) / (20 * steps)


def time_layer(w, steps):
    """The whole attention layer (Section 2 steps 1-5) of a self-attention workload with model width
    H * d: times the Q/K/V projection, the fused attention, the Output projection and the layer call."""
    dev = torch.device("cuda")
    B, H, N, d = w.B, w.H, w.Nq, w.d
    Dm = H * d
    X = torch.randn(B, N, Dm, device=dev, dtype=torch.bfloat16)
    Wqkv = (torch.randn(3 * H * d, Dm, device=dev) * Dm ** -0.5).to(torch.bfloat16)
    Wo = (torch.randn(Dm, H * d, device=dev) * Dm ** -0.5).to(torch.bfloat16)
    Q = torch.empty(B, H, N, d, device=dev, dtype=torch.bfloat16)
    K, V, O = torch.empty_like(Q), torch.empty_like(Q), torch.empty_like(Q)
    Y = torch.empty(B, N, Dm, device=dev, dtype=torch.bfloat16)
    proj = 2.0 * B * N * Dm * H * d
    # the two fully connected operators that follow the attention layer in a block, with the usual
    # four-fold expansion of the model width
    W1 = (torch.randn(4 * Dm, Dm, device=dev) * Dm ** -0.5).to(torch.bfloat16)
    W2 = (torch.randn(Dm, 4 * Dm, device=dev) * (4 * Dm) ** -0.5).to(torch.bfloat16)
    F1 = torch.empty(B, N, 4 * Dm, device=dev, dtype=torch.bfloat16)
    Y2 = torch.empty_like(Y)

    def block():
        api.flat_attn_layer_fwd(X, Wqkv, Wo, Y, Q, K, V, O, w.scale)
        api.flat_fc_fwd(Y, W1, F1)
        api.flat_fc_fwd(F1, W2, Y2)

    parts = [("qkv_projection", lambda: api.flat_qkv_proj_fwd(X, Wqkv, Q, K, V), 3 * proj),
             ("fused_attention", lambda: api.flat_attn_fwd(Q, K, V, O, w.scale), float(w.flops)),
             ("out_projection", lambda: api.flat_out_proj_fwd(O, Wo, Y), proj),
             ("layer", lambda: api.flat_attn_layer_fwd(X, Wqkv, Wo, Y, Q, K, V, O, w.scale), 4 * proj + w.flops),
             ("fc1", lambda: api.flat_fc_fwd(Y, W1, F1), 2.0 * B * N * Dm * 4 * Dm),
             ("fc2", lambda: api.flat_fc_fwd(F1, W2, Y2), 2.0 * B * N * Dm * 4 * Dm),
             ("block_gemm_operators", block, 4 * proj + w.flops + 4.0 * B * N * Dm * 4 * Dm)]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for name, fn, flops in parts:
        try:
            for _ in range(2):
                fn()
        except api.FlatAttnError as e:
            print(json.dumps({"workload": w.name, "step": name, "unsupported": str(e)}), flush=True)
            return
        torch.cuda.synchronize()
        time.sleep(1.0)
        for _ in range(2):
            fn()
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / steps
        print(json.dumps({"workload": w.name, "model_width": Dm, "step": name, "ms": round(ms, 4),
                          "tflops": round(flops / ms / 1e9, 1)}), flush=True)


def time_varlen(w, steps, causal):
    """The packed variable-length entry point on the tokens of a self-attention workload: once with
    B equal sequences (the workload itself, packed) and once with a seeded mix of lengths that adds
    up to the same number of tokens (lengths between 1/8 and 15/8 of the workload's)."""
    import numpy as np
    dev = torch.device("cuda")
    B, H, N, d = w.B, w.H, w.Nq, w.d
    total = B * N
    rng = np.random.default_rng(2107)
    S = max(2 * B, 8)                                    # the mix has more, shorter and longer sequences
    mean = total // S
    mix = rng.integers(mean // 8, mean * 15 // 8 + 1, size=S)
    mix = np.maximum(1, (mix * (total / mix.sum())).astype(np.int64))
    mix[-1] += total - mix.sum()
    Q = torch.randn(total, H, d, device=dev, dtype=torch.bfloat16)
    K, V, O = torch.randn_like(Q), torch.randn_like(Q), torch.empty_like(Q)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for label, lens in (("equal", np.full(B, N, dtype=np.int64)), ("mixed", mix)):
        cu = torch.from_numpy(np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)).to(dev)
        flops = 4.0 * H * d * float((lens.astype(np.float64) ** 2).sum())
        fn = lambda: api.flat_attn_varlen_fwd(Q, K, V, O, cu, cu, int(lens.max()), w.scale, causal=causal)
        try:
            for _ in range(2):
                fn()
        except api.FlatAttnError as e:
            print(json.dumps({"workload": w.name, "varlen": label, "unsupported": str(e)}), flush=True)
            return
        torch.cuda.synchronize()
        time.sleep(1.0)
        for _ in range(2):
            fn()
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / steps
        print(json.dumps({"workload": w.name, "varlen": label, "sequences": int(len(lens)), "longest": int(lens.max()),
                          "shortest": int(lens.min()), "causal": causal, "ms": round(ms, 4),
                          "tflops_nominal": round(flops / ms / 1e9, 1)}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workloads", default="c1_bert_base_512,c2_bert_large_4k,c3_16k,c4_64k_d128,c5_cross_masked")
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--skip-simt-above", type=float, default=2e12,
                    help="skip the FFMA variant for workloads above this many FLOP (it takes long)")
    ap.add_argument("--causal", action="store_true",
                    help="time the variants under the causal mask (TFLOP/s then count the nominal, unmasked FLOP)")
    ap.add_argument("--varlen", action="store_true",
                    help="time the packed variable-length entry point (equal lengths and a seeded mix)")
    ap.add_argument("--layer", action="store_true",
                    help="time the whole attention layer (projections + fused attention) instead of the variants")
    ap.add_argument("--shapes", default="",
                    help="extra shapes B:H:N:d or B:H:Nq:Nk:d, comma separated (e.g. 16:16:512:64,1:1:128:16384:64), timed after the workloads")
    args = ap.parse_args()
    todo = [inputs.WORKLOADS[name] for name in args.workloads.split(",") if name]
    for spec in args.shapes.split(","):
        if spec:
            f = [int(x) for x in spec.split(":")]
            B, H, Nq, Nk, d = f if len(f) == 5 else (f[0], f[1], f[2], f[2], f[3])
            todo.append(inputs.Workload("B%d_H%d_Nq%d_Nk%d_d%d" % (B, H, Nq, Nk, d), B, H, Nq, Nk, d))
    for w in todo:
        name = w.name
        if args.varlen:
            if w.Nq == w.Nk and not w.masked:
                time_varlen(w, args.steps, args.causal)
            continue
        if args.layer:
            if w.Nq == w.Nk and not w.masked:
                time_layer(w, args.steps)
            continue
        best = None
        for variant, label in VARIANTS.items():
            if variant == api.FLAT_VARIANT_SIMT and w.flops > args.skip_simt_above:
                continue
            ms, err, ms_graph = time_variant(w, variant, args.steps if variant != api.FLAT_VARIANT_SIMT else 2, causal=args.causal)
            row = {"workload": name, "variant": variant, "kernel": label}
            if args.causal:
                row["causal"] = True
            if ms is None:
                row["unsupported"] = err
            else:
                row.update(ms=round(ms, 4), tflops=round(w.flops / ms / 1e9, 1))
                if ms_graph is not None:
                    row.update(ms_graph_replay=round(ms_graph, 4), tflops_graph_replay=round(w.flops / ms_graph / 1e9, 1))
                if variant != api.FLAT_VARIANT_AUTO and (best is None or ms < best[0]):
                    best = (ms, variant)
            print(json.dumps(row), flush=True)
        if best:
            print(json.dumps({"workload": name, "best_variant": best[1], "ms": round(best[0], 4)}), flush=True)


if __name__ == "__main__":
    main()
