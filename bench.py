#!/usr/bin/env python
"""Benchmark of the fused attention hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

A step is one pass of the whole hot path (TMA loads of Q/K/V tiles, both tcgen05 contractions,
the streaming softmax, the store of O) over one batch of synthetic input -- one kernel launch.
Prints ONE JSON line: the metric is fused-attention TFLOP/s, 4*B*H*Nq*Nk*d FLOP per call.
With N > 1 ranks (torchrun), every rank runs the same workload on its own batch: the (batch, head)
pairs are independent units, so there is no data-path collective (weak scaling).
`--impl reference` times the CPU oracle, as it stands, on a bounded row sample (rank 0 only).
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "fused attention TFLOP/s"
UNIT = "TFLOP/s"
DEFAULT_WORKLOAD = "c2_bert_large_4k"
L2_FLUSH_BELOW = 256 << 20          # workloads smaller than this get an L2 flush before every timed launch
KERNEL_NAMES = {1: "fused_simt_kernel", 2: "fused_tc_kernel", 3: "fused_tc2_kernel", 4: "fused_tc2_kernel",
                5: "fused_tc3_kernel"}


def kernel_name(variant, w):
    """The kernel a launch of this workload runs (variant 0: the dispatcher's choice for problems that fill the GPU)."""
    if variant in KERNEL_NAMES:
        return KERNEL_NAMES[variant]
    ctas = ((w.Nq + 255) // 256) * w.B * w.H            # 256-row CTAs; the dispatcher's rule with 148 SMs
    if w.d == 64:
        slabs_fill = 3 * 256 * ((w.Nq + 255) // 256) <= 4 * w.Nq
        tc3 = (2 * ctas >= 148 and w.Nk > 1024) or (ctas >= 2 * 148 and not w.masked and slabs_fill)
        return "fused_tc3_kernel" if tc3 else "fused_tc2_kernel"
    return "fused_tc2_kernel" if (ctas >= 148 or w.Nk > 256) else "fused_tc_kernel"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"bf16_tflops": float(p["bf16_tflops"]), "bf16_tflops_sustained": float(p["bf16_tflops_sustained"]),
                "hbm_gbs": float(p["hbm_gbs"]), "source": "measured"}
    return {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the dominant kernel, copied from
# the ncu captures summarised in profiles/fused_tc3_kernel_dram_and_pipes.md and
# profiles/fused_tc2_kernel_dram_and_pipes.md (None where nothing was captured).
MEASURED_DRAM_TRAFFIC = {
    ("fused_tc3_kernel", "c2_bert_large_4k"): 514_200_000,
    ("fused_tc3_kernel", "p_4k_small"): 116_900_000,
    ("fused_tc2_kernel", "c2_bert_large_4k"): 516_000_000,
    ("fused_tc2_kernel", "p_4k_small"): 117_600_000,
    ("fused_tc2_kernel", "p_16k_d128_small"): 51_900_000,
}


def load_traffic(workload, kernel="fused_tc2_kernel"):
    return MEASURED_DRAM_TRAFFIC.get((kernel, workload))


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + q,
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for ln in self.proc.stdout:
            self.lines.append(ln.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 6:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for nm, v in zip(names, f[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def cpu_baseline(w, Qb, Kb, Vb, vl, target_seconds=15.0):
    """The oracle, as it stands, on a bounded seeded row sample of the same workload."""
    import oracle
    from paper_2107_06419_b200 import inputs
    threads = oracle.hardware_threads()
    rows = inputs.sample_rows(w, 1)[:threads]                       # calibration: one row per thread
    t0 = time.perf_counter()
    oracle.attention(Qb, Kb, Vb, w.scale, valid_len=vl, rows=rows)
    per_row = (time.perf_counter() - t0) / max(1, len(rows)) * threads    # thread-seconds per row
    total_rows = w.B * w.H * w.Nq
    nrows = int(min(total_rows, max(threads, target_seconds * threads / max(per_row, 1e-9))))
    per_head = max(1, nrows // (w.B * w.H))
    rows = inputs.sample_rows(w, per_head)
    t0 = time.perf_counter()
    r = oracle.attention(Qb, Kb, Vb, w.scale, valid_len=vl, rows=rows)
    dt = time.perf_counter() - t0
    flops = 4.0 * len(rows) * w.Nk * w.d
    return {"value": flops / dt / 1e12, "unit": UNIT, "cores": int(r["threads"]), "kind": "oracle",
            "sample": "%d seeded query rows (%d per (b,h)) of %s, all %d keys, %.1f s wall"
                      % (len(rows), per_head, w.name, w.Nk, dt)}, rows, r["O"]


def run_reference(args, w):
    """--impl reference: the CPU oracle on the host cores (bounded sample per step)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2107_06419_b200 import inputs
    import oracle
    Qb, Kb, Vb = inputs.make_qkv_bf16(w)
    vl = inputs.make_valid_len(w) if w.masked else None
    threads = oracle.hardware_threads()
    rows = inputs.sample_rows(w, 1)[:threads]
    t0 = time.perf_counter()
    oracle.attention(Qb, Kb, Vb, w.scale, valid_len=vl, rows=rows)
    per_row = (time.perf_counter() - t0) / max(1, len(rows)) * threads
    steps = args.steps + args.warmup
    budget = min(20.0, 150.0 / max(1, steps))                        # seconds per step
    nrows = int(max(threads, min(w.B * w.H * w.Nq, budget * threads / max(per_row, 1e-9))))
    per_head = max(1, nrows // (w.B * w.H))
    rows = inputs.sample_rows(w, per_head)
    for _ in range(args.warmup):
        oracle.attention(Qb, Kb, Vb, w.scale, valid_len=vl, rows=rows)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        r = oracle.attention(Qb, Kb, Vb, w.scale, valid_len=vl, rows=rows)
    dt = (time.perf_counter() - t0) / args.steps
    val = 4.0 * len(rows) * w.Nk * w.d / dt / 1e12
    sample = "%d seeded query rows (%d per (b,h)) of %s per step, all %d keys" % (len(rows), per_head, w.name, w.Nk)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w, extra={"sample": sample}),
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": int(r["threads"]), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def workload_config(w, extra=None):
    c = {"workload": w.name, "B": w.B, "H": w.H, "Nq": w.Nq, "Nk": w.Nk, "d": w.d, "scale": "1/sqrt(d)",
         "mask": "per-batch key padding, valid length uniform in [Nk/2, Nk]" if w.masked else "none",
         "inputs": "bf16 iid N(0,1), seeded counter-based generator",
         "l2": ("inputs (%d MiB) larger than the 126 MB L2; no flush between steps" % (w.qkvo_bytes() >> 20))
               if w.qkvo_bytes() > L2_FLUSH_BELOW else
               ("inputs (%.1f MiB) fit in L2: a 256 MiB buffer is rewritten before every timed launch and the "
                "step time is the sum of the per-launch event times" % (w.qkvo_bytes() / 2 ** 20))}
    if extra:
        c.update(extra)
    return c


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--variant", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--with-naive", action="store_true",
                    help="also time the unfused baseline (L and A materialised in device memory)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    from paper_2107_06419_b200 import inputs
    w = inputs.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch
    import torch.distributed as dist
    from paper_2107_06419_b200 import api          # raises if the CUDA library is missing
    from paper_2107_06419_b200 import shard

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    # Each rank owns one full batch of the workload (its own seed): units are independent.
    seed = shard.rank_seed(inputs.DEFAULT_SEED, rank)
    Qb, Kb, Vb = inputs.make_qkv_bf16(w, seed)
    vl = inputs.make_valid_len(w, seed) if w.masked else None
    as_t = lambda bits: torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16)
    Qh, Kh, Vh = (as_t(x).pin_memory() for x in (Qb, Kb, Vb))
    Oh = torch.empty(Qh.shape, dtype=torch.bfloat16).pin_memory()
    vlh = None if vl is None else torch.from_numpy(vl).pin_memory()
    Q, K, V = Qh.to(dev), Kh.to(dev), Vh.to(dev)
    O = torch.empty_like(Q)
    vld = None if vl is None else vlh.to(dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    ws = torch.empty(api.flat_attn_host_workspace_bytes(w.B, w.H, w.Nq, w.Nk, w.d), dtype=torch.uint8, device=dev)

    def step():
        api.flat_attn_fwd_ex(Q, K, V, O, w.scale, k_valid_len=vld, status=status, variant=args.variant)

    def step_e2e():
        api.flat_attn_fwd_host(Qh, Kh, Vh, Oh, w.scale, ws, k_valid_len=vlh, status=status, variant=args.variant)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    flush = None
    if w.qkvo_bytes() <= L2_FLUSH_BELOW:
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def timed(fn, steps):
        """K launches bracketed by barrier + synchronize; returns (total ms, per-launch ms list).
        With an L2 flush between launches the total is the sum of the per-launch times."""
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        t_begin.record()
        for a, b in evs:
            if flush is not None:
                flush.fill_(1)
            a.record(); fn(); b.record()
        t_end.record()
        barrier()
        per = [a.elapsed_time(b) for a, b in evs]
        return (sum(per) if flush is not None else t_begin.elapsed_time(t_end)), per

    for _ in range(args.warmup):
        step()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    total_ms, per_launch = timed(step, args.steps)
    launches = api.flat_attn_last_launch_count() * args.steps
    clocks = sampler.stop() if rank == 0 else None
    assert int(status.item()) == 0, "device status 0x%x" % int(status.item())

    for _ in range(2):
        step_e2e()
    e2e_ms, _ = timed(step_e2e, max(3, min(args.steps, 5)))
    e2e_ms /= max(3, min(args.steps, 5))

    total_ms, e2e_ms = shard.max_over_ranks([total_ms, e2e_ms], dev)
    ms_per_step = total_ms / args.steps
    value = shard.whole_job_rate(float(w.flops), world, ms_per_step) / 1e12
    e2e_value = shard.whole_job_rate(float(w.flops), world, e2e_ms) / 1e12

    if rank == 0:
        peaks = load_peaks()
        kernel_ms = float(np.mean(per_launch))
        achieved = float(w.flops) / (kernel_ms * 1e-3) / 1e12
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": workload_config(w, {"parallelism": "dp%d over independent batches, no collective" % world}),
            "e2e": {"value": e2e_value, "unit": UNIT, "ms_per_step": e2e_ms,
                    "h2d_bytes_per_step": int(2 * (Qh.numel() + Kh.numel() + Vh.numel()) + (0 if vl is None else 4 * w.B)),
                    "d2h_bytes_per_step": int(2 * Oh.numel())},
            "gpu_launches": launches,
            "clocks": clocks,
            "roofline": {"bound": "tensor", "kernel": kernel_name(args.variant, w),
                         "achieved": achieved,
                         "peak": peaks["bf16_tflops"], "unit": UNIT, "frac": achieved / peaks["bf16_tflops"],
                         "peak_kind": "burst bf16 matmul, of " + peaks["source"],
                         "frac_of_sustained": achieved / peaks["bf16_tflops_sustained"],
                         "kernel_ms": kernel_ms, "kernel_ms_min": float(np.min(per_launch)),
                         "kernel_ms_median": float(np.median(per_launch)), "flops_per_launch": w.flops,
                         "traffic": load_traffic(w.name, kernel_name(args.variant, w)),
                         "algorithmic_bytes": w.qkvo_bytes()},
        }
        if vl is not None:
            # Masked workload: `value` counts the masked keys too (the stated metric, 4 B H Nq Nk d);
            # this is the same rate counted over the valid keys only.
            useful = 4.0 * w.H * w.Nq * w.d * float(np.sum(vl))
            out["useful_work"] = {"value": value * useful / float(w.flops), "unit": UNIT,
                                  "valid_key_fraction": useful / float(w.flops)}
        if args.with_naive and world == 1:
            # The paper's unfused baseline on the same inputs: L (fp32) and A (bf16) go through HBM.
            elems = w.B * w.H * w.Nq * w.Nk
            L = torch.empty((w.B, w.H, w.Nq, w.Nk), dtype=torch.float32, device=dev)
            A = torch.empty((w.B, w.H, w.Nq, w.Nk), dtype=torch.bfloat16, device=dev)
            O2 = torch.empty_like(Q)
            naive = lambda: api.flat_attn_naive_fwd_ex(Q, K, V, O2, L, A, w.scale, k_valid_len=vld)
            naive()
            n_ms, _ = timed(naive, 3)
            n_ms /= 3
            out["naive"] = {"ms_per_step": n_ms, "value": float(w.flops) / (n_ms * 1e-3) / 1e12, "unit": UNIT,
                            "kernels_per_step": 3, "materialised_bytes": 6 * elems,
                            "algorithmic_bytes": 12 * elems + w.qkvo_bytes(),
                            "max_abs_diff_vs_fused": float((O2.float() - O.float()).abs().max())}
            del L, A, O2
        if not args.no_cpu_baseline and world == 1:
            cb, rows, Oref = cpu_baseline(w, Qb, Kb, Vb, vl)
            got = O.view(-1, w.d)[torch.from_numpy(rows).to(dev)].float().cpu().numpy().astype(np.float64)
            err = np.abs(got - Oref)
            cb["parity_on_sample"] = {"max_abs": float(err.max()), "mean_abs": float(err.mean())}
            out["cpu_baseline"] = cb
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
