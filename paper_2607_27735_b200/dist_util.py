"""Multi-GPU plumbing.  The hot path is independent per (layer, sequence, KV head), so ranks
never exchange data on it: each GPU serves its own sequences (weak scaling) and the only
communication is the barrier and the max-over-ranks of the measured time."""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def init_process_group(backend: str, device=None) -> None:
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29511")
    kwargs = {}
    if backend == "nccl" and device is not None:
        kwargs["device_id"] = device
    dist.init_process_group(backend=backend, **kwargs)


def max_over_ranks(value: float, world: int, device=None) -> float:
    """Max of a host scalar over all ranks (identity for world == 1)."""
    if world <= 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64,
                     device=device if dist.get_backend() == "nccl" else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def shard_sequences(n_sequences: int, world: int, rank: int) -> range:
    """Contiguous, balanced share of a batch of sequences for `rank` (remainder to low ranks)."""
    base, rem = divmod(n_sequences, world)
    lo = rank * base + min(rank, rem)
    return range(lo, lo + base + (1 if rank < rem else 0))
