#!/usr/bin/env python
"""Benchmark of the fused attention hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

A step is one pass of the whole hot path (TMA loads of Q/K/V tiles, both tcgen05 contractions,
the streaming softmax, the store of O) over one batch of synthetic input -- one kernel launch.
Prints ONE JSON line: the metric is fused-attention TFLOP/s, 4*B*H*Nq*Nk*d FLOP per call, on the
headline workload; the line's `workloads` list carries the other benchmark configurations (fewer
steps each, with a parity check on a seeded row sample) and `naive` the unfused baseline.
With N > 1 ranks every rank runs the same workload on its own batch: the (batch, head) pairs are
independent units, so there is no data-path collective (weak scaling).  Ranks come from the
launcher's environment (torchrun); without one, `--gpus N` starts N ranks itself.
`--impl reference` times the CPU oracle, as it stands, on a bounded row sample (rank 0 only).
"""
import argparse
import json
import os
import socket
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
OTHER_WORKLOADS = ["c1_bert_base_512", "c3_16k", "c4_64k_d128", "c5_cross_masked"]
# launches that leave most SMs empty (few query tiles, long key sequences): what the key split over a cluster is for
UNDERFILLED = [("u1_128q_16k_d64", 1, 1, 128, 16384, 64), ("u2_128q_16k_h8_d128", 1, 8, 128, 16384, 128)]
FP32_WORKLOAD = "c3_16k"             # the configuration the fp32 path is timed on (widened to fp32 tensors)
L2_FLUSH_BELOW = 256 << 20          # workloads smaller than this get an L2 flush before every timed launch
# FLAT_VARIANT_* (as reported by the library after a call) -> the kernel that variant launches
KERNEL_OF_VARIANT = {1: "fused_simt_kernel", 2: "fused_tc_kernel", 3: "fused_tc2_kernel<2 tiles>",
                     4: "fused_tc2_kernel<1 tile>", 5: "fused_tc3_kernel", 6: "fused_rgran_kernel", 7: "fused_tf32_kernel",
                     8: "fused_tc2_kernel<1 tile, keys over a 2-CTA cluster>", 9: "fused_tc2_kernel<1 tile, keys over a 4-CTA cluster>",
                     10: "fused_tc2_kernel<1 tile, keys over an 8-CTA cluster>",
                     11: "fused_tc2_kernel<1 tile, two warpgroups on alternate key tiles>",
                     12: "fused_tc2_kernel<1 tile, two warpgroups, keys over a 2-CTA cluster>",
                     13: "fused_tc2_kernel<1 tile, two warpgroups, keys over a 4-CTA cluster>",
                     14: "fused_tc2_kernel<1 tile, two warpgroups, keys over an 8-CTA cluster>",
                     15: "fused_tc2_kernel<1 tile, keys over a 16-CTA cluster>",
                     16: "fused_tc2_kernel<1 tile, two warpgroups, keys over a 16-CTA cluster>"}
TF32_OVER_BF16 = 1.1 / 2.25          # nominal dense tensor peaks: the tf32 roofline is the measured bf16 peak times this

# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the dominant kernel from ncu
# captures, with the capture they come from; a (kernel, workload) pair without a capture reports null.
MEASURED_DRAM_TRAFFIC = {
    ("fused_tc3_kernel", "c2_bert_large_4k"): (515_300_000, "profiles/fused_tc3_kernel_dram_and_pipes.md"),
    ("fused_tc3_kernel", "p_4k_small"): (116_900_000, "profiles/fused_tc3_kernel_dram_and_pipes.md"),
    ("fused_tc3_kernel", "c5_cross_masked"): (349_600_000, "profiles/fused_tc3_kernel_even_deal_cuda_events.md"),
    ("fused_tc3_kernel", "c3_16k"): (520_600_000, "profiles/fused_tc3_kernel_dram_and_pipes.md"),
    ("fused_tc2_kernel<2 tiles>", "c4_64k_d128"): (597_400_000, "profiles/fused_tc2_kernel_dram_and_pipes.md"),
    ("fused_tc2_kernel<2 tiles>", "c2_bert_large_4k"): (516_000_000, "profiles/fused_tc2_kernel_dram_and_pipes.md"),
    ("fused_tc2_kernel<2 tiles>", "p_4k_small"): (117_600_000, "profiles/fused_tc2_kernel_dram_and_pipes.md"),
    ("fused_tc2_kernel<2 tiles>", "p_16k_d128_small"): (51_900_000, "profiles/fused_tc2_kernel_dram_and_pipes.md"),
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"bf16_tflops": float(p["bf16_tflops"]), "bf16_tflops_sustained": float(p["bf16_tflops_sustained"]),
                "hbm_gbs": float(p["hbm_gbs"]), "source": "measured"}
    return {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


def traffic_fields(kernel, workload):
    hit = MEASURED_DRAM_TRAFFIC.get((kernel, workload))
    if hit:
        return {"traffic": hit[0], "traffic_source": "ncu dram__bytes_read.sum + dram__bytes_write.sum, " + hit[1]}
    return {"traffic": None, "traffic_note": "no ncu capture of %s on %s" % (kernel, workload)}


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []
        self.first = 0

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
        return self

    def _read(self):
        for ln in self.proc.stdout:
            self.lines.append(ln.strip())

    def mark(self):
        """Only samples taken from now on count (the sampler is started ahead of the warm-up launches, so that the
        start-up of nvidia-smi does not fall into the timed region)."""
        self.first = len(self.lines)
        return self

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
        for ln in self.lines[self.first:]:
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


def oracle_on_sample(w, Qb, Kb, Vb, vl, per_head=None, target_seconds=15.0):
    """The oracle, as it stands, on a seeded row sample of the workload: (timing dict, rows, O rows).
    per_head = None sizes the sample for about `target_seconds` of wall time."""
    import oracle
    from paper_2107_06419_b200 import inputs
    threads = oracle.hardware_threads()
    if per_head is None:
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


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_ranks(n):
    """No launcher gave this process a rank: start `n` ranks of this script (one per GPU) under
    torch.distributed.run on this node and pass their exit code on."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n),
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def dry_run(args, w):
    """The rank plumbing without a GPU (CPU tests): every rank draws its seed, 'times' a fake step and
    joins the max-reduction over the chosen backend; rank 0 prints the line."""
    import torch
    import torch.distributed as dist
    from paper_2107_06419_b200 import inputs, shard
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group(args.backend)
    seed = shard.rank_seed(inputs.DEFAULT_SEED, rank)
    ms = 1.0 + rank                                                   # the slowest rank decides
    (ms_max,) = shard.max_over_ranks([ms], torch.device("cpu"))
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": shard.whole_job_rate(float(w.flops), world, ms_max) / 1e12,
                          "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
                          "ms_per_step": ms_max, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                          "dtype": "bf16", "data": "synthetic", "dry_run": True, "seed_rank0": seed,
                          "config": workload_config(w, {"parallelism": "dp%d over independent batches, no collective" % world})}))
    if world > 1:
        dist.destroy_process_group()


class Bench:
    """One GPU's view of the benchmark: device buffers of a workload, timed launches."""

    def __init__(self, torch, api, dev, world, variant):
        self.torch, self.api, self.dev, self.world, self.variant = torch, api, dev, world, variant
        # written before a timed launch whose inputs fit in L2, and once in front of every timed region; allocated
        # here, not between warm-up and timing, where the allocation would leave the GPU idle for milliseconds
        self.flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
        self.schedule = None

    def barrier(self):
        if self.world > 1:
            import torch.distributed as dist
            dist.barrier()
        self.torch.cuda.synchronize()

    def timed(self, fn, steps, flush):
        """K launches bracketed by barrier + synchronize; returns (total ms, per-launch ms list).
        With an L2 flush between launches the total is the sum of the per-launch times."""
        torch = self.torch
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        self.barrier()
        if not flush:
            # The stream is empty after the barrier: without device work in front of it, the first event pair
            # would also time the host marshalling the first call's arguments (25-50 us seen on a 1.1 ms kernel).
            # One fill of the flush buffer (~80 us, outside t_begin .. t_end) lets the host run ahead.
            self.flush.fill_(1)
        t_begin.record()
        for a, b in evs:
            if flush:
                self.flush.fill_(1)
            a.record(); fn(); b.record()
        t_end.record()
        self.barrier()
        per = [a.elapsed_time(b) for a, b in evs]
        return (sum(per) if flush else t_begin.elapsed_time(t_end)), per

    def load(self, w, seed):
        """Generates the workload on the host (pinned) and uploads it."""
        from paper_2107_06419_b200 import inputs
        torch = self.torch
        Qb, Kb, Vb = inputs.make_qkv_bf16(w, seed)
        vl = inputs.make_valid_len(w, seed) if w.masked else None
        as_t = lambda bits: torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16)
        host = {"Q": as_t(Qb).pin_memory(), "K": as_t(Kb).pin_memory(), "V": as_t(Vb).pin_memory(),
                "vl": None if vl is None else torch.from_numpy(vl).pin_memory()}
        devt = {k: (None if v is None else v.to(self.dev)) for k, v in host.items()}
        devt["O"] = torch.empty_like(devt["Q"])
        devt["status"] = torch.zeros(1, dtype=torch.int32, device=self.dev)
        return (Qb, Kb, Vb, vl), host, devt

    def measure(self, w, d, steps, warmup, sample_clocks):
        """Warm-up, then `steps` timed launches of the fused call on resident inputs."""
        api = self.api
        step = lambda: api.flat_attn_fwd_ex(d["Q"], d["K"], d["V"], d["O"], w.scale, k_valid_len=d["vl"],
                                            status=d["status"], variant=self.variant)
        sampler = ClockSampler(self.dev.index).start() if sample_clocks else None
        if sampler:
            time.sleep(0.3)                              # nvidia-smi attaches to the GPU: not during the launches
        for _ in range(warmup):
            step()
        kernel = KERNEL_OF_VARIANT.get(api.flat_attn_last_variant(), "?")
        # how fused_tc3_kernel handed the items to the SMs (as reported by the library for the last launch)
        self.schedule = None
        if api.flat_attn_last_variant() == api.FLAT_VARIANT_TC3:
            self.schedule = {api.FLAT_SCHEDULE_ITEMS: "one CTA per item", api.FLAT_SCHEDULE_PERSISTENT: "persistent CTAs",
                             api.FLAT_SCHEDULE_EVEN_DEAL: "key steps dealt evenly"}.get(api.flat_attn_last_schedule())
        if sampler:
            sampler.mark()
        total_ms, per = self.timed(step, steps, flush=w.qkvo_bytes() <= L2_FLUSH_BELOW)
        clocks = sampler.stop() if sampler else None
        # a run that saw a hardware or thermal slowdown is not a measurement: taken once more after a pause
        # (a power cap is normal on a 1 kW part and is kept and noted); every rank takes the same decision
        # because the region is bracketed by barriers, and with one rank sampling it is that rank's alone
        throttled = {"hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown"}
        if clocks and self.world == 1 and throttled & set(clocks.get("reasons", [])):
            time.sleep(5.0)
            first = clocks
            sampler = ClockSampler(self.dev.index).start()
            time.sleep(0.3)
            for _ in range(warmup):
                step()
            sampler.mark()
            total_ms, per = self.timed(step, steps, flush=w.qkvo_bytes() <= L2_FLUSH_BELOW)
            clocks = sampler.stop()
            clocks["remeasured_after"] = first.get("reasons", [])
        code = int(d["status"].item())
        assert code == 0, "device status 0x%x" % code
        return total_ms, per, kernel, clocks


def roofline_entry(w, per_launch, kernel, peaks):
    kernel_ms = float(np.mean(per_launch))
    achieved = float(w.flops) / (kernel_ms * 1e-3) / 1e12
    r = {"bound": "tensor", "kernel": kernel, "achieved": achieved, "peak": peaks["bf16_tflops"], "unit": UNIT,
         "frac": achieved / peaks["bf16_tflops"], "peak_kind": "burst bf16 matmul, of " + peaks["source"],
         "frac_of_sustained": achieved / peaks["bf16_tflops_sustained"], "kernel_ms": kernel_ms,
         "kernel_ms_min": float(np.min(per_launch)), "kernel_ms_median": float(np.median(per_launch)),
         "flops_per_launch": w.flops, "algorithmic_bytes": w.qkvo_bytes()}
    r.update(traffic_fields(kernel, w.name))
    return r


def parity_on_sample(torch, w, data, O, dev, per_head):
    Qb, Kb, Vb, vl = data
    cb, rows, Oref = oracle_on_sample(w, Qb, Kb, Vb, vl, per_head=per_head)
    got = O.view(-1, w.d)[torch.from_numpy(rows).to(dev)].float().cpu().numpy().astype(np.float64)
    err = np.abs(got - Oref)
    return cb, {"rows": int(len(rows)), "max_abs": float(err.max()), "mean_abs": float(err.mean())}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--variant", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--headline-only", action="store_true",
                    help="skip the other workloads and the unfused baseline (they run at N = 1 only anyway)")
    ap.add_argument("--backend", default="nccl", choices=["nccl", "gloo"])
    ap.add_argument("--dry-run", action="store_true", help="rank plumbing only, no CUDA call (CPU tests)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    from paper_2107_06419_b200 import inputs
    w = inputs.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, w)
        return
    if "WORLD_SIZE" not in os.environ and args.gpus > 1:
        sys.exit(spawn_ranks(args.gpus))
    if args.dry_run:
        dry_run(args, w)
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
        dist.init_process_group(args.backend, device_id=dev)
    bench = Bench(torch, api, dev, world, args.variant)

    # Each rank owns one full batch of the workload (its own seed): units are independent.
    seed = shard.rank_seed(inputs.DEFAULT_SEED, rank)
    data, host, d = bench.load(w, seed)
    total_ms, per_launch, kernel, clocks = bench.measure(w, d, args.steps, args.warmup, sample_clocks=rank == 0)
    headline_schedule = bench.schedule
    launches = api.flat_attn_last_launch_count() * args.steps

    Oh = torch.empty(host["Q"].shape, dtype=torch.bfloat16).pin_memory()
    ws = torch.empty(api.flat_attn_host_workspace_bytes(w.B, w.H, w.Nq, w.Nk, w.d), dtype=torch.uint8, device=dev)
    step_e2e = lambda: api.flat_attn_fwd_host(host["Q"], host["K"], host["V"], Oh, w.scale, ws, k_valid_len=host["vl"],
                                              status=d["status"], variant=args.variant)
    for _ in range(2):
        step_e2e()
    e2e_steps = max(3, min(args.steps, 5))
    e2e_ms, _ = bench.timed(step_e2e, e2e_steps, flush=False)
    e2e_ms /= e2e_steps

    total_ms, e2e_ms = shard.max_over_ranks([total_ms, e2e_ms], dev)
    ms_per_step = total_ms / args.steps
    value = shard.whole_job_rate(float(w.flops), world, ms_per_step) / 1e12
    e2e_value = shard.whole_job_rate(float(w.flops), world, e2e_ms) / 1e12

    if rank == 0:
        peaks = load_peaks()
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": workload_config(w, {"parallelism": "dp%d over independent batches, no collective" % world}),
            "e2e": {"value": e2e_value, "unit": UNIT, "ms_per_step": e2e_ms,
                    "h2d_bytes_per_step": int(2 * (host["Q"].numel() + host["K"].numel() + host["V"].numel())
                                              + (0 if data[3] is None else 4 * w.B)),
                    "d2h_bytes_per_step": int(2 * Oh.numel())},
            "gpu_launches": launches,
            "clocks": clocks,
            "roofline": roofline_entry(w, per_launch, kernel, peaks),
        }
        if headline_schedule:
            out["roofline"]["schedule"] = headline_schedule
        if data[3] is not None:
            # Masked workload: `value` counts the masked keys too (the stated metric, 4 B H Nq Nk d);
            # this is the same rate counted over the valid keys only.
            useful = 4.0 * w.H * w.Nq * w.d * float(np.sum(data[3]))
            out["useful_work"] = {"value": value * useful / float(w.flops), "unit": UNIT,
                                  "valid_key_fraction": useful / float(w.flops)}
        if not args.no_cpu_baseline and world == 1:
            cb, par = parity_on_sample(torch, w, data, d["O"], dev, per_head=None)
            cb["parity_on_sample"] = par
            out["cpu_baseline"] = cb
        if not args.headline_only and world == 1:
            del ws, Oh
            out["naive"] = run_naive(bench, torch, api, w, d) if w.name == DEFAULT_WORKLOAD else None
            out["backward"] = run_backward(bench, torch, api, w, d, data, seed, args, peaks)
            host = d = data = None
            torch.cuda.empty_cache()
            out["workloads"] = [run_other(bench, torch, api, inputs.WORKLOADS[n], seed, args, peaks, dev)
                                for n in OTHER_WORKLOADS if n != w.name]
            out["fp32"] = run_fp32(bench, torch, api, inputs.WORKLOADS[FP32_WORKLOAD], seed, args, peaks, dev)
            out["underfilled"] = [run_underfilled(torch, api, inputs.Workload(*spec), seed, args, dev) for spec in UNDERFILLED]
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def run_naive(bench, torch, api, w, d):
    """The paper's unfused baseline on the same inputs: L (fp32) and A (bf16) go through HBM."""
    elems = w.B * w.H * w.Nq * w.Nk
    L = torch.empty((w.B, w.H, w.Nq, w.Nk), dtype=torch.float32, device=bench.dev)
    A = torch.empty((w.B, w.H, w.Nq, w.Nk), dtype=torch.bfloat16, device=bench.dev)
    O2 = torch.empty_like(d["Q"])
    naive = lambda: api.flat_attn_naive_fwd_ex(d["Q"], d["K"], d["V"], O2, L, A, w.scale, k_valid_len=d["vl"])
    naive()
    n_ms, _ = bench.timed(naive, 3, flush=False)
    n_ms /= 3
    return {"ms_per_step": n_ms, "value": float(w.flops) / (n_ms * 1e-3) / 1e12, "unit": UNIT,
            "kernels_per_step": 3, "materialised_bytes": 6 * elems,
            "bytes_model": 12 * elems + w.qkvo_bytes(),
            "hbm_gbs_on_model": (12 * elems + w.qkvo_bytes()) / (n_ms * 1e-3) / 1e9,
            "max_abs_diff_vs_fused": float((O2.float() - d["O"].float()).abs().max())}


def run_backward(bench, torch, api, w, d, data, seed, args, peaks):
    """The backward pass (dQ, dK, dV from dO, recomputing the weights from the forward's lse) on the same
    workload: 10 B H Nq Nk d FLOP per call (five contractions), two kernels per step."""
    from paper_2107_06419_b200 import inputs
    if w.d not in (64, 128):
        return None
    time.sleep(1.0)
    dev = bench.dev
    n = w.B * w.H * w.Nq * w.d
    dOb = inputs.f32_to_bf16_bits(inputs.normal_f32(seed, 5, 0, n)).reshape(w.B, w.H, w.Nq, w.d)
    dO = torch.from_numpy(dOb.view(np.int16)).view(torch.bfloat16).to(dev)
    lse = torch.empty((w.B, w.H, w.Nq), dtype=torch.float32, device=dev)
    delta = torch.empty_like(lse)
    dQ, dK, dV = torch.empty_like(d["Q"]), torch.empty_like(d["K"]), torch.empty_like(d["K"])
    api.flat_attn_fwd_ex(d["Q"], d["K"], d["V"], d["O"], w.scale, k_valid_len=d["vl"], status=d["status"], lse=lse)
    step = lambda: api.flat_attn_bwd_ex(d["Q"], d["K"], d["V"], d["O"], dO, lse, dQ, dK, dV, delta, w.scale,
                                        k_valid_len=d["vl"], status=d["status"])
    sampler = ClockSampler(dev.index).start()
    time.sleep(0.3)
    for _ in range(3):
        step()
    steps = int(max(3, min(args.steps, 10)))
    sampler.mark()
    total_ms, per = bench.timed(step, steps, flush=False)
    clocks = sampler.stop()
    assert int(d["status"].item()) == 0
    ms = float(np.mean(per))
    flops = 2.5 * float(w.flops)
    val = flops / (ms * 1e-3) / 1e12
    e = {"workload": w.name, "kernel": "bwd_tc_kernel<dQ> + bwd_tc_kernel<dK,dV>", "kernels_per_step": 2, "steps": steps,
         "ms": ms, "ms_min": float(np.min(per)), "flops_per_step": flops, "value": val, "unit": UNIT,
         "frac": val / peaks["bf16_tflops"], "frac_of_sustained": val / peaks["bf16_tflops_sustained"],
         "flops_executed_per_step": 3.5 * float(w.flops), "clocks": clocks}
    if not args.no_cpu_baseline:
        import oracle
        Qb, Kb, Vb, vl = data
        heads = np.array([0, (w.B * w.H) // 2 + 1], dtype=np.int64)
        ref = oracle.attention_bwd(Qb, Kb, Vb, dOb, w.scale, valid_len=vl, heads=heads)
        par = {}
        for name, got in (("dQ", dQ), ("dK", dK), ("dV", dV)):
            g = got.view(w.B * w.H, -1, w.d)[torch.from_numpy(heads).to(dev)].float().cpu().numpy().astype(np.float64)
            err = np.abs(g - ref[name])
            par[name] = {"max_rel_to_max": float(err.max() / np.abs(ref[name]).max()),
                         "mean_rel_to_mean": float(err.mean() / np.abs(ref[name]).mean())}
        e["parity_on_sample"] = {"heads": [int(h) for h in heads], **par}
    return e


def run_fp32(bench, torch, api, w, seed, args, peaks, dev):
    """The fp32 path on one configuration widened to fp32 tensors (the same seeded values, exactly representable):
    every contraction runs as three tf32 products, so the kernel executes 3 x the metric's FLOP on the tensor
    cores; `frac` is the metric's FLOP rate over the tf32 peak, `frac_executed` counts the three products."""
    time.sleep(1.0)
    data, host, d = bench.load(w, seed)
    Q, K, V = d["Q"].float(), d["K"].float(), d["V"].float()
    O = torch.full(Q.shape, float("nan"), dtype=torch.float32, device=dev)
    del host
    d["Q"] = d["K"] = d["V"] = d["O"] = None
    step = lambda: api.flat_attn_fwd_ex(Q, K, V, O, w.scale, k_valid_len=d["vl"], status=d["status"])
    sampler = ClockSampler(dev.index).start()
    time.sleep(0.3)
    for _ in range(3):
        step()
    kernel = KERNEL_OF_VARIANT.get(api.flat_attn_last_variant(), "?")
    steps = int(max(3, min(args.steps, 5)))
    sampler.mark()
    total_ms, per = bench.timed(step, steps, flush=False)
    clocks = sampler.stop()
    assert int(d["status"].item()) == 0
    ms = float(np.mean(per))
    val = float(w.flops) / (ms * 1e-3) / 1e12
    peak = peaks["bf16_tflops"] * TF32_OVER_BF16
    cfg = workload_config(w)
    cfg["inputs"] = "the workload's seeded bf16 values widened to fp32"
    cfg["l2"] = "inputs (%d MiB) larger than the 126 MB L2; no flush between steps" % (2 * w.qkvo_bytes() >> 20)
    e = {"workload": w.name + " as fp32", "config": cfg, "dtype": "f32 (3 x tf32 products, fp32 sums)",
         "kernel": kernel, "steps": steps, "ms": ms, "ms_min": float(np.min(per)), "value": val, "unit": UNIT,
         "peak": peak, "peak_source": "measured bf16 peak x nominal tf32/bf16 ratio", "frac": val / peak,
         "frac_executed": 3.0 * val / peak, "clocks": clocks}
    if not args.no_cpu_baseline:
        _, e["parity_on_sample"] = parity_on_sample(torch, w, data, O, dev, per_head=8)
        e["parity_on_sample"]["bar_max_abs"] = 1e-4
    del data, d, Q, K, V, O
    torch.cuda.empty_cache()
    return e


def run_underfilled(torch, api, w, seed, args, dev):
    """A launch with far fewer query tiles than SMs: GPU time per launch in a replay of a CUDA graph of 20 launches,
    the dispatcher's choice (keys of a tile split over a thread-block cluster) beside the unsplit kernel, and parity
    of the dispatcher's output on every row."""
    from paper_2107_06419_b200 import inputs
    Qb, Kb, Vb = inputs.make_qkv_bf16(w, seed)
    as_t = lambda bits: torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(dev)
    Q, K, V = as_t(Qb), as_t(Kb), as_t(Vb)
    O = torch.empty_like(Q)
    status = torch.zeros(1, dtype=torch.int32, device=dev)

    def replay_us(variant):
        s = torch.cuda.Stream(device=dev)
        with torch.cuda.stream(s):
            for _ in range(3):
                api.flat_attn_fwd_ex(Q, K, V, O, w.scale, status=status, variant=variant, stream=s.cuda_stream)
            ran = api.flat_attn_last_variant()
            s.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=s):
                for _ in range(20):
                    api.flat_attn_fwd_ex(Q, K, V, O, w.scale, status=status, variant=variant, stream=s.cuda_stream)
            g.replay()
            s.synchronize()
            best = None
            for _ in range(5):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(s); g.replay(); e1.record(s); s.synchronize()
                t = e0.elapsed_time(e1) / 20 * 1e3
                best = t if best is None or t < best else best
        return best, ran

    unsplit_us, unsplit_variant = replay_us(api.FLAT_VARIANT_TC2_SINGLE if w.d == 64 else api.FLAT_VARIANT_TC2)
    auto_us, auto_variant = replay_us(api.FLAT_VARIANT_AUTO)           # (last: O holds the dispatcher's result)
    assert int(status.item()) == 0
    e = {"workload": w.name, "config": {"B": w.B, "H": w.H, "Nq": w.Nq, "Nk": w.Nk, "d": w.d},
         "timing": "CUDA-graph replay of 20 launches, best of 5, microseconds per launch",
         "kernel": KERNEL_OF_VARIANT.get(auto_variant, "?"), "us": auto_us, "value": float(w.flops) / auto_us / 1e6, "unit": UNIT,
         "unsplit_kernel": KERNEL_OF_VARIANT.get(unsplit_variant, "?"), "unsplit_us": unsplit_us}
    if not args.no_cpu_baseline:
        import oracle
        ref = oracle.attention(Qb, Kb, Vb, w.scale)["O"]
        err = np.abs(O.float().cpu().numpy().astype(np.float64) - ref)
        e["parity_all_rows"] = {"max_abs": float(err.max()), "mean_abs": float(err.mean())}
    return e


def run_other(bench, torch, api, w, seed, args, peaks, dev):
    """One more benchmark configuration: fewer steps, a parity check on 64 seeded rows per (b,h)."""
    time.sleep(2.0)                                      # let the power window of the previous workload pass
    data, host, d = bench.load(w, seed)
    ms1 = float(w.flops) / 0.9e15 * 1e3                  # a rough guess of one launch, to bound the timed region
    # (about 40 ms of launches: the 1 kW cap cuts in after roughly that much back-to-back work at d = 64, and the
    # headline run before this one has already shown the capped rate; `steps` and `clocks` are in the entry)
    steps = int(max(3, min(args.steps, 20, 40.0 / ms1)))
    total_ms, per, kernel, clocks = bench.measure(w, d, steps, max(3, min(args.warmup, 5)), sample_clocks=True)
    ms = float(np.mean(per))
    val = float(w.flops) / (ms * 1e-3) / 1e12
    e = {"workload": w.name, "config": workload_config(w), "kernel": kernel, "steps": steps, "ms": ms,
         "ms_min": float(np.min(per)), "value": val, "unit": UNIT, "frac": val / peaks["bf16_tflops"],
         "frac_of_sustained": val / peaks["bf16_tflops_sustained"], "clocks": clocks}
    if data[3] is not None:
        useful = 4.0 * w.H * w.Nq * w.d * float(np.sum(data[3])) / float(w.flops)
        e["useful_work"] = {"value": val * useful, "unit": UNIT, "valid_key_fraction": useful,
                            "frac": val * useful / peaks["bf16_tflops"]}
    if bench.schedule:
        e["schedule"] = bench.schedule
    e.update(traffic_fields(kernel, w.name))
    if not args.no_cpu_baseline:
        _, e["parity_on_sample"] = parity_on_sample(torch, w, data, d["O"], dev, per_head=64)
    del data, host, d
    torch.cuda.empty_cache()
    return e


if __name__ == "__main__":
    main()
