"""Host-side logic for running independent GEMM replicas on several GPUs.

A GEMM partitions into independent output blocks, so several GPUs never need to
exchange operand or result data: each rank multiplies its own problem (or its
own row block of C) and only the timing is combined.  The rule is: every rank
times its steps on the device, the slowest rank defines the step time, and the
whole-job rate counts the work of all ranks.
"""
from __future__ import annotations

from typing import Sequence


def replica_seed(base_seed: int, rank: int) -> int:
    """Each rank draws its own operands."""
    return base_seed + 1000 * rank


def row_block(M: int, rank: int, world: int, align: int = 256):
    """Row range [lo, hi) of C owned by `rank` when one GEMM is split by rows
    over `world` GPUs (B replicated): blocks are multiples of `align` rows
    except the last, and cover [0, M) exactly."""
    if world < 1 or not (0 <= rank < world):
        raise ValueError("bad rank/world")
    units = (M + align - 1) // align
    base, extra = divmod(units, world)
    lo_u = rank * base + min(rank, extra)
    hi_u = lo_u + base + (1 if rank < extra else 0)
    return min(lo_u * align, M), min(hi_u * align, M)


def max_over_ranks(values_ms: Sequence[float], dist=None, device=None):
    """Element-wise maximum over ranks of a few device-measured durations."""
    import torch
    t = torch.tensor(list(values_ms), dtype=torch.float64, device=device or "cpu")
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.tolist()]


def whole_job_rate(ops_per_rank: float, world: int, ms: float) -> float:
    """Aggregate rate in 1e12 ops/s: all ranks' work over the slowest rank's time."""
    return world * ops_per_rank / (ms * 1e-3) / 1e12
