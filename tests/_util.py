"""Helpers shared by the GPU parity tests: bf16 marshalling and the parity metrics."""
import numpy as np
import torch

from paper_2607_03229_b200 import workloads as W

# Tolerances of the hot path (bf16 inputs/outputs, fp32 accumulation) against the unrounded fp64 oracle.
O_MAX_ABS = 1e-2
O_REL_L2 = 5e-3
GRAD_REL_L2 = 1e-2
LSE_MAX_ABS = 1e-3


def to_dev(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns -> bf16 CUDA tensor (same bits)."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).cuda()


def to_bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)


def to_f64(t: torch.Tensor) -> np.ndarray:
    if t.dtype == torch.bfloat16:
        return W.bf16_bits_to_f64(to_bits(t))
    return t.detach().cpu().double().numpy()


def max_abs(x: np.ndarray, ref: np.ndarray) -> float:
    return float(np.abs(x - ref).max()) if ref.size else 0.0


def rel_l2(x: np.ndarray, ref: np.ndarray) -> float:
    den = float(np.linalg.norm(ref.ravel()))
    num = float(np.linalg.norm((x - ref).ravel()))
    return num / den if den > 0 else (0.0 if num == 0 else float("inf"))


def status_buf() -> torch.Tensor:
    return torch.zeros(4, dtype=torch.int32, device="cuda")
