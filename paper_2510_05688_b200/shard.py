"""Host-side helpers for running the decode step on several GPUs of one node.

The step has no exchange between (batch row, KV-head group) units: every query head has its own
index sets, budget and sample, and K/V are per KV head.  Ranks therefore take disjoint slices of the
batch (or run replicas of one layer) with no collective on the data path; the only communication is
the barrier and the max-over-ranks reduction of the measured time.
"""
from __future__ import annotations


def shard_batch(batch: int, rank: int, world: int):
    """Contiguous slice [lo, hi) of the batch rows owned by `rank`; sizes differ by at most one."""
    if world <= 0 or not (0 <= rank < world) or batch < 0:
        raise ValueError("bad shard arguments")
    base, extra = divmod(batch, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def max_over_ranks(value: float, world: int) -> float:
    """MAX all-reduce of a host scalar over the default process group (any backend)."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())
