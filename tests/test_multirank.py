"""The N > 1 path of the benchmark on CPU: two gloo ranks agree on the slowest timing, get distinct
seeds and disjoint, complete shards.  No data-path collective exists to test: units are independent."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2107_06419_b200 import inputs, shard


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = inputs.Workload("mr", 2, 3, 64, 96, 16)
        seed = shard.rank_seed(inputs.DEFAULT_SEED, rank)
        q, _, _ = inputs.make_qkv_bf16(w, seed)
        ms = [1.0 + rank, 10.0 - rank]                      # rank 1 is slower on the first, faster on the second
        mx = shard.max_over_ranks(ms, torch.device("cpu"))
        units = list(shard.shard_units(w.B * w.H, rank, world))
        gathered = [None] * world
        dist.all_gather_object(gathered, {"rank": rank, "seed": seed, "q0": int(q.ravel()[0]), "max": mx, "units": units})
        if rank == 0:
            out.put(gathered)
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_agree():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r["rank"] for r in res] == [0, 1]
    assert res[0]["seed"] != res[1]["seed"] and res[0]["q0"] != res[1]["q0"]
    assert res[0]["max"] == res[1]["max"] == [2.0, 10.0]
    units = res[0]["units"] + res[1]["units"]
    assert sorted(units) == list(range(6)) and len(res[0]["units"]) == 3


def test_shard_units_balanced_and_complete():
    for n in (1, 7, 8, 96, 256):
        for world in (1, 2, 3, 8):
            parts = [shard.shard_units(n, r, world) for r in range(world)]
            flat = [u for p in parts for u in p]
            assert flat == list(range(n))
            sizes = [len(p) for p in parts]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        shard.shard_units(4, 2, 2)


def test_whole_job_rate_and_single_process_identity():
    assert shard.whole_job_rate(1e12, 8, 2.0) == 8e12 / 2e-3
    assert shard.max_over_ranks([1.5, 2.5], torch.device("cpu")) == [1.5, 2.5]
    assert shard.rank_seed(7, 0) == 7 and shard.rank_seed(7, 3) != shard.rank_seed(7, 2)


def test_bench_gpus_flag_starts_the_ranks_itself():
    """`bench.py --gpus 2` without a launcher must create two ranks (here: gloo, no CUDA call) and
    report them; run the way the driver runs the single-command form."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--steps", "2", "--warmup", "3",
                        "--dry-run", "--backend", "gloo", "--workload", "c1_bert_base_512"],
                       capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, r.stdout
    out = json.loads(lines[0])
    assert out["n_gpus"] == 2 and out["dry_run"] is True
    assert out["ms_per_step"] == 2.0                    # the slower rank's fake step time
    assert out["value"] == 2 * inputs.WORKLOADS["c1_bert_base_512"].flops / 2e-3 / 1e12
