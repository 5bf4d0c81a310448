"""One pass of the encoder hot path through the C ABI: plan -> attention forward -> (trained only)
attention backward -> merge into the LLM embedding buffer.  Buffer management and call order only;
every arithmetic step runs inside libmpipe_enc."""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional

import numpy as np
import torch

from . import binding as B
from .workloads import Workload


def bits_to_dev(bits: np.ndarray, device="cuda") -> torch.Tensor:
    """uint16 bf16 bit patterns -> bf16 tensor on `device` (same bits)."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).to(device)


def dev_to_bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)


@dataclass
class StepBuffers:
    """Device tensors of one microbatch.  q/k/v/dout are inputs; everything else is written by the path."""
    q: torch.Tensor
    k: torch.Tensor
    v: torch.Tensor
    dout: Optional[torch.Tensor]
    o: torch.Tensor
    lse: Optional[torch.Tensor]
    dq: Optional[torch.Tensor]
    dk: Optional[torch.Tensor]
    dv: Optional[torch.Tensor]
    workspace: Optional[torch.Tensor]
    merge_src: Optional[torch.Tensor]     # [T, hidden] rows to merge (o viewed as [T, H*D] when hidden == H*D)
    llm_embeds: Optional[torch.Tensor]    # [n_llm, hidden]
    positions: Optional[torch.Tensor]     # int32 [T]
    status: torch.Tensor


def allocate(w: Workload, device="cuda", q=None, k=None, v=None, dout=None, llm_embeds=None,
             merge_src=None) -> StepBuffers:
    """Allocate the outputs (and, if not given, random-normal inputs drawn on the device)."""
    T, H, D = w.total_tokens, w.n_heads, w.head_dim
    mode = B.TRAINED if w.trained else B.FROZEN

    def rnd(shape, seed):
        g = torch.Generator(device=device)
        g.manual_seed(seed)
        return torch.randn(shape, device=device, generator=g, dtype=torch.float32).to(torch.bfloat16)

    q = rnd((T, H, D), w.seed + 1) if q is None else q
    k = rnd((T, H, D), w.seed + 2) if k is None else k
    v = rnd((T, H, D), w.seed + 3) if v is None else v
    o = torch.empty((T, H, D), dtype=torch.bfloat16, device=device)
    lse = dq = dk = dv = ws = None
    if w.trained:
        dout = rnd((T, H, D), w.seed + 4) if dout is None else dout
        lse = torch.empty((H, T), dtype=torch.float32, device=device)
        dq, dk, dv = (torch.empty((T, H, D), dtype=torch.bfloat16, device=device) for _ in range(3))
        ws = torch.empty(max(B.attn_workspace_bytes(T, H, D, mode), 256), dtype=torch.uint8, device=device)
    pos = emb = None
    if w.merge_hidden is not None:
        pos = torch.from_numpy(np.ascontiguousarray(w.positions, dtype=np.int32)).to(device)
        emb = rnd((w.n_llm_tokens, w.merge_hidden), w.seed + 5) if llm_embeds is None else llm_embeds
        if merge_src is None:
            merge_src = o.view(T, H * D) if w.merge_hidden == H * D else rnd((T, w.merge_hidden), w.seed + 6)
    return StepBuffers(q, k, v, dout, o, lse, dq, dk, dv, ws, merge_src, emb, pos,
                       torch.zeros(4, dtype=torch.int32, device=device))


def run_step(w: Workload, buf: StepBuffers, plan: Optional[B.SegPlan] = None, stream=None) -> B.SegPlan:
    """plan (host, + upload) -> fwd -> bwd (trained) -> merge.  Enqueues on the current stream."""
    mode = B.TRAINED if w.trained else B.FROZEN
    if plan is None:
        plan = B.seg_plan(w.patch_counts, mode).to_device(buf.q.device)
    scale = w.softmax_scale
    B.varlen_attn_fwd(buf.q, buf.k, buf.v, buf.o, buf.lse, plan, scale, buf.status, stream)
    if w.trained:
        B.varlen_attn_bwd(buf.dout, buf.q, buf.k, buf.v, buf.o, buf.lse, buf.dq, buf.dk, buf.dv, plan, scale,
                          buf.workspace, buf.status, stream)
    if w.merge_hidden is not None:
        B.merge_tokens(buf.merge_src, buf.llm_embeds, buf.positions, mode, buf.status, stream)
    return plan


def kernels_per_step(w: Workload) -> int:
    """Kernels of this library launched by one run_step (forward 1, backward 3, merge 1)."""
    if w.total_tokens == 0:
        return 0
    return 1 + (3 if w.trained else 0) + (1 if w.merge_hidden is not None else 0)
