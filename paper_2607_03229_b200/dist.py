"""Multi-GPU plumbing of the benchmark: the hot path shards by microbatch (the paper's Replicated
layout with a ByMicrobatch owner, Section 4.2), so ranks exchange nothing on the data path; only the
benchmark's timing is reduced (max over ranks) and its work counters summed."""
from __future__ import annotations

import os
from typing import Sequence, Tuple

import torch
import torch.distributed as dist


def env_world() -> Tuple[int, int, int]:
    """(rank, local_rank, world_size) from the torchrun environment; (0, 0, 1) when launched plainly."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str) -> Tuple[int, int, int]:
    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29511")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local_rank, world


def barrier() -> None:
    if dist.is_initialized():
        dist.barrier()


def rank_seed(base_seed: int, rank: int) -> int:
    """Every rank draws its own microbatch: same recipe, different seed (weak scaling)."""
    return base_seed + 1000 * rank


def reduce_max_sum(max_vals: Sequence[float], sum_vals: Sequence[float], device="cpu"):
    """Element-wise max over ranks of `max_vals` and sum over ranks of `sum_vals` (float64)."""
    mx = torch.tensor(list(max_vals), dtype=torch.float64, device=device)
    sm = torch.tensor(list(sum_vals), dtype=torch.float64, device=device)
    if dist.is_initialized():
        dist.all_reduce(mx, op=dist.ReduceOp.MAX)
        dist.all_reduce(sm, op=dist.ReduceOp.SUM)
    return mx.tolist(), sm.tolist()


def shutdown() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()
