"""Multi-GPU plumbing for the benchmark: how work is split over ranks and how timings are combined.

The hot path has no exchange step: (batch, head) pairs -- and query rows inside them -- are
independent (paper Section 5.1, the B/H/R granularities), so ranks only ever agree on a timing.
One process per GPU; `torch.distributed` (NCCL on GPUs, gloo in the CPU tests) carries the
max-reduction, nothing on the data path.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def rank_seed(base_seed: int, rank: int) -> int:
    """Each rank generates its own batch (weak scaling): distinct, reproducible seeds."""
    return int(base_seed) + 1000003 * int(rank)


def shard_units(n_units: int, rank: int, world: int) -> range:
    """Contiguous, balanced split of `n_units` independent units ((b,h) pairs) over `world` ranks:
    the first n_units % world ranks get one extra unit.  Used when total work is fixed."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    base, extra = divmod(int(n_units), int(world))
    lo = rank * base + min(rank, extra)
    return range(lo, lo + base + (1 if rank < extra else 0))


def max_over_ranks(values, device) -> list:
    """Element-wise maximum of a short list of floats over all ranks (identity when not distributed)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def whole_job_rate(units_per_rank: float, world: int, ms_max: float) -> float:
    """Aggregate throughput: what all ranks processed divided by the slowest rank's time (per second)."""
    return units_per_rank * world / (ms_max * 1e-3)
