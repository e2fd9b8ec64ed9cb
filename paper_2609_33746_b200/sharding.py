"""Multi-GPU plumbing: the decode operator shards over sequences with no exchange step.

Every (sequence, KV head) is independent from the LUT build to the output (Sec. 3.3: one
index per KV head, one score row per query head), so N GPUs each take a contiguous slice of
the batch and run the same single-GPU call; nothing crosses NVLink on the data path.  The
helpers here are host-side only: which sequences a rank owns, and the max-over-ranks timing
reduction the benchmark needs."""
from __future__ import annotations

import dataclasses
from typing import Tuple

import torch

from .workload import DecodeConfig


def rank_slice(n_items: int, world: int, rank: int) -> Tuple[int, int]:
    """Contiguous [lo, hi) share of n_items for `rank`; shares differ by at most one item."""
    if world <= 0 or not 0 <= rank < world:
        raise ValueError("bad world / rank")
    base, extra = divmod(n_items, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def shard_config(cfg: DecodeConfig, world: int, rank: int) -> Tuple[DecodeConfig, int]:
    """The sub-workload (a slice of the sequences) that `rank` runs, and its first sequence."""
    lo, hi = rank_slice(cfg.batch, world, rank)
    sub = dataclasses.replace(cfg, name=f"{cfg.name}[{lo}:{hi}]", batch=hi - lo,
                              seq_lens=tuple(cfg.seq_lens[lo:hi]))
    return sub, lo


def max_over_ranks(value: float, device="cpu") -> float:
    """Largest `value` over all ranks (the benchmark's step time); identity without a group."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())
