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


def seam_targets(owner: Sequence[int], first_stage_rank: int = 0):
    """For the Replicated -> Sharded seam (Table 2): which microbatches rank r must ship, per rank.  `owner[m]` is the
    ByMicrobatch owner of microbatch m (0-based); every microbatch goes to `first_stage_rank`, and a microbatch that
    is already there needs no transfer (its merge is local)."""
    world = (max(owner) + 1) if len(owner) else 1
    world = max(world, first_stage_rank + 1)
    ship = {r: [] for r in range(world)}
    local = []
    for m, r in enumerate(owner):
        (local if r == first_stage_rank else ship[r]).append(m)
    return ship, local


def share_rows(t: "torch.Tensor", src_rank: int):
    """Export `t` ([rows, hidden] bf16 CUDA tensor owned by `src_rank`, alone in its allocation) to every other rank of
    the default process group.  Returns the tensor itself on `src_rank` and a binding.PeerRows elsewhere."""
    from . import binding as B
    rank = dist.get_rank() if dist.is_initialized() else 0
    payload = [None]
    if rank == src_rank:
        payload = [(B.ipc_export(t), int(t.shape[0]), int(t.shape[1]), int(t.stride(0)))]
    if dist.is_initialized():
        dist.broadcast_object_list(payload, src=src_rank)
    if rank == src_rank:
        return t
    handle, rows, hidden, stride = payload[0]
    return B.PeerRows(handle, rows, hidden, stride)


LAYER_PARAM_SHAPES = (("ln1_gamma", lambda h, f: (h,)), ("ln1_beta", lambda h, f: (h,)), ("w_qkv", lambda h, f: (3 * h, h)),
                      ("b_qkv", lambda h, f: (3 * h,)), ("w_o", lambda h, f: (h, h)), ("b_o", lambda h, f: (h,)),
                      ("ln2_gamma", lambda h, f: (h,)), ("ln2_beta", lambda h, f: (h,)), ("w_fc1", lambda h, f: (f, h)),
                      ("b_fc1", lambda h, f: (f,)), ("w_fc2", lambda h, f: (h, f)), ("b_fc2", lambda h, f: (h,)))


def alloc_grad_bucket(n_layers: int, hidden: int, ffn: int, device="cuda"):
    """One flat fp32 buffer for the gradients of the whole encoder and, per layer, a dict of views into it (the twelve
    tensors mpipe_encoder_layer_bwd accumulates into).  One buffer = one all-reduce per step: a bucket sized for launch
    latency rather than per-tensor collectives.  Every view starts on a 16-byte boundary."""
    sizes, offs, total = [], [], 0
    for _ in range(n_layers):
        for name, shape in LAYER_PARAM_SHAPES:
            shp = shape(hidden, ffn)
            n = 1
            for d in shp:
                n *= d
            offs.append(total)
            sizes.append((name, shp, n))
            total += (n + 3) // 4 * 4
    flat = torch.zeros(total, dtype=torch.float32, device=device)
    layers, i = [], 0
    for _ in range(n_layers):
        views = {}
        for _name in LAYER_PARAM_SHAPES:
            name, shp, n = sizes[i]
            views[name] = flat[offs[i]:offs[i] + n].view(shp)
            i += 1
        layers.append(views)
    return flat, layers


def dp_reduce(flat_grads: "torch.Tensor", group=None) -> None:
    """DpReduce(enc, ReplicaGroup) (Section 4.1): the trainable, transposed encoder is replicated on every rank of the
    replica group and each rank saw only its own microbatches, so the accumulated fp32 gradients are summed over the
    group -- one all-reduce of the bucket (NCCL on GPUs, NVLS inside the switch when available).  A no-op for one rank."""
    if dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(flat_grads, op=dist.ReduceOp.SUM, group=group)


def shutdown() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()
