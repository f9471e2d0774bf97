"""Multi-GPU use of the library: independent replicas, one process per GPU.

The (sequence, KV head, layer) units of the path never exchange data, and the paper's method is
single-GPU, so N GPUs run N independent copies of the workload; the only cross-rank step is the
bookkeeping of a measurement: a barrier around the timed region, the slowest rank's time, and the
sum of the bytes all ranks moved.  Works with any torch.distributed backend (NCCL on GPUs, gloo on
CPU) or with no process group at all (single process).
"""
from __future__ import annotations

import torch


def _dist():
    import torch.distributed as dist
    return dist if dist.is_available() and dist.is_initialized() else None


def barrier() -> None:
    d = _dist()
    if d is not None:
        d.barrier()


def aggregate_step(ms_local: float, bytes_local: int, device="cpu"):
    """(slowest rank's time in ms, bytes summed over ranks, world size)."""
    d = _dist()
    if d is None:
        return float(ms_local), int(bytes_local), 1
    t = torch.tensor([float(ms_local)], dtype=torch.float64, device=device)
    b = torch.tensor([int(bytes_local)], dtype=torch.int64, device=device)
    d.all_reduce(t, op=d.ReduceOp.MAX)
    d.all_reduce(b, op=d.ReduceOp.SUM)
    return float(t.item()), int(b.item()), d.get_world_size()


def replica_seed(base_seed: int, rank: int) -> int:
    """Every rank draws its own synthetic workload."""
    return int(base_seed) + 1000 * int(rank)
