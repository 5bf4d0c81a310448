"""CPU oracle for the packed encoder layer -- TEST INFRASTRUCTURE, not product code.

The paper names the relocated computation only as a "ViT-style encoder" (Section 2, "From LLM to
MLLM Training"); the layer stated here is the pre-norm Transformer block of that family, over a
packed varlen token matrix x[T, hidden]:

    a  = LayerNorm(x; g1, b1)
    qkv = a Wqkv^T + bqkv                      -> q, k, v as [T, H, D]   (column block order q | k | v)
    q, k = rope(q), rope(k)                    optional rotate-half rotary encoding, angles given per token and pair
    o  = per-image softmax attention (oracle.attn_fwd, block-diagonal over cu_seqlens)
    x1 = x + o Wo^T + bo
    m  = LayerNorm(x1; g2, b2)
    y  = x1 + GELU(m W1^T + bb1) W2^T + bb2    GELU(u) = u * Phi(u)  (erf form)

Everything is fp64 numpy with no blocking or reordering; weights are nn.Linear-style [out, in].
Inputs that are bf16 on the GPU side are passed as uint16 bit patterns and widened exactly.
The GPU path rounds every stored intermediate to bf16; this oracle does not (the tolerance of
the parity tests covers that, as it does for the attention output).

Pins: ``tests/test_oracle_layer.py`` (torch fp64 functional ops, closed forms, identity cases).
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np

from . import _f64, attn_bwd, attn_fwd


def widen(a) -> np.ndarray:
    """bf16 bit patterns (uint16) -> fp64, exactly; fp64 passes through."""
    return _f64(a)


def layernorm(x: np.ndarray, gamma: np.ndarray, beta: np.ndarray, eps: float) -> np.ndarray:
    """Row-wise (x - mean) / sqrt(var + eps) * gamma + beta with the biased variance."""
    x = np.asarray(x, dtype=np.float64)
    mean = x.mean(axis=-1, keepdims=True)
    var = ((x - mean) ** 2).mean(axis=-1, keepdims=True)
    return (x - mean) / np.sqrt(var + eps) * gamma + beta


def layernorm_bwd(x: np.ndarray, dy: np.ndarray, gamma: np.ndarray, eps: float):
    """Gradients of y = xhat * gamma + beta, xhat = (x - mean) / sqrt(var + eps), per row:
    dx = rstd (g - mean(g) - xhat mean(g xhat)) with g = dy gamma;  dgamma = sum_t dy xhat;  dbeta = sum_t dy."""
    x, dy = np.asarray(x, dtype=np.float64), np.asarray(dy, dtype=np.float64)
    mean = x.mean(axis=-1, keepdims=True)
    rstd = 1.0 / np.sqrt(((x - mean) ** 2).mean(axis=-1, keepdims=True) + eps)
    xhat = (x - mean) * rstd
    g = dy * gamma
    dx = rstd * (g - g.mean(axis=-1, keepdims=True) - xhat * (g * xhat).mean(axis=-1, keepdims=True))
    return dx, (dy * xhat).sum(axis=0), dy.sum(axis=0)


def linear(x: np.ndarray, w: np.ndarray, b=None) -> np.ndarray:
    """y = x w^T + b, w as [out, in]."""
    y = np.asarray(x, dtype=np.float64) @ np.asarray(w, dtype=np.float64).T
    return y if b is None else y + np.asarray(b, dtype=np.float64)


try:   # a library erf as one step of the definition; the fallback is the C library's, element by element
    from scipy.special import erf as _erf
except ImportError:   # pragma: no cover
    _erf = np.vectorize(math.erf, otypes=[np.float64])


def gelu(u: np.ndarray) -> np.ndarray:
    """u * Phi(u) with Phi the standard normal CDF: 0.5 u (1 + erf(u / sqrt 2))."""
    u = np.asarray(u, dtype=np.float64)
    return 0.5 * u * (1.0 + _erf(u / math.sqrt(2.0)))


def gelu_grad(u: np.ndarray) -> np.ndarray:
    """d/du [u Phi(u)] = Phi(u) + u phi(u) with phi the standard normal density."""
    u = np.asarray(u, dtype=np.float64)
    return 0.5 * (1.0 + _erf(u / math.sqrt(2.0))) + u * np.exp(-0.5 * u * u) / math.sqrt(2.0 * math.pi)


def linear_dgrad(dy: np.ndarray, w: np.ndarray) -> np.ndarray:
    """Input gradient of y = x w^T: dx = dy w."""
    return np.asarray(dy, dtype=np.float64) @ np.asarray(w, dtype=np.float64)


def linear_wgrad(dy: np.ndarray, x: np.ndarray):
    """Parameter gradients of y = x w^T + b: dw = dy^T x, db = column sums of dy."""
    dy = np.asarray(dy, dtype=np.float64)
    return dy.T @ np.asarray(x, dtype=np.float64), dy.sum(axis=0)


def rope(x: np.ndarray, cos: np.ndarray, sin: np.ndarray) -> np.ndarray:
    """Rotate-half rotary encoding.  x: [T, H, D]; cos, sin: [T, D/2] (angle of pair j of token t).  The pair is
    (x[..., j], x[..., j + D/2]) and it is rotated by that angle: a plain 2-D rotation per pair."""
    x = np.asarray(x, dtype=np.float64)
    half = x.shape[-1] // 2
    x1, x2 = x[..., :half], x[..., half:]
    c, s = np.asarray(cos, dtype=np.float64)[:, None, :], np.asarray(sin, dtype=np.float64)[:, None, :]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


@dataclass
class LayerWeights:
    """fp64 views of the layer's parameters (nn.Linear layout [out, in])."""
    g1: np.ndarray
    b1: np.ndarray
    wqkv: np.ndarray   # [3*hidden, hidden], rows ordered q | k | v, each head-major
    bqkv: np.ndarray
    wo: np.ndarray     # [hidden, hidden]
    bo: np.ndarray
    g2: np.ndarray
    b2: np.ndarray
    w1: np.ndarray     # [ffn, hidden]
    bb1: np.ndarray
    w2: np.ndarray     # [hidden, ffn]
    bb2: np.ndarray


def encoder_layer_fwd(x, w: LayerWeights, cu_seqlens, n_heads: int, scale: float, eps: float, rope_tables=None):
    """The whole block.  x: [T, hidden] (uint16 bf16 bits or fp64).  Returns (y, parts) with parts a dict of
    the intermediates (a, qkv, o, x1, m, f) in fp64 for stage-wise comparisons."""
    x = widen(x)
    T, hidden = x.shape
    D = hidden // n_heads
    a = layernorm(x, w.g1, w.b1, eps)
    qkv = linear(a, w.wqkv, w.bqkv)
    q, k, v = (np.ascontiguousarray(qkv[:, i * hidden:(i + 1) * hidden].reshape(T, n_heads, D)) for i in range(3))
    if rope_tables is not None:   # (cos, sin) [T, D/2]: q and k are rotated, v is not
        q, k = rope(q, *rope_tables), rope(k, *rope_tables)
    o, lse = attn_fwd(q, k, v, cu_seqlens, scale)
    x1 = x + linear(o.reshape(T, hidden), w.wo, w.bo)
    m = layernorm(x1, w.g2, w.b2, eps)
    f = gelu(linear(m, w.w1, w.bb1))
    y = x1 + linear(f, w.w2, w.bb2)
    return y, {"a": a, "qkv": qkv, "o": o, "lse": lse, "x1": x1, "m": m, "f": f}


def encoder_layer_bwd(x, w: LayerWeights, cu_seqlens, n_heads: int, scale: float, eps: float, dy, rope_tables=None):
    """Gradient of the whole block by the chain rule, stage by stage in reverse (each stage's own gradient is one of the
    functions above or oracle.attn_bwd).  Returns dx [T, hidden] and a dict of the twelve parameter gradients."""
    x, dy = widen(x), np.asarray(widen(dy), dtype=np.float64)
    T, hidden = x.shape
    D = hidden // n_heads
    _, p = encoder_layer_fwd(x, w, cu_seqlens, n_heads, scale, eps, rope_tables)
    u = linear(p["m"], w.w1, w.bb1)
    g = {}
    # y = x1 + f W2^T + bb2
    g["w_fc2"], g["b_fc2"] = linear_wgrad(dy, p["f"])
    du = linear_dgrad(dy, w.w2) * gelu_grad(u)
    g["w_fc1"], g["b_fc1"] = linear_wgrad(du, p["m"])
    dm = linear_dgrad(du, w.w1)
    dln, g["ln2_gamma"], g["ln2_beta"] = layernorm_bwd(p["x1"], dm, w.g2, eps)
    dx1 = dy + dln
    # x1 = x + o Wo^T + bo
    o2 = p["o"].reshape(T, hidden)
    g["w_o"], g["b_o"] = linear_wgrad(dx1, o2)
    do = linear_dgrad(dx1, w.wo).reshape(T, n_heads, D)
    qkv = p["qkv"]
    q, k, v = (np.ascontiguousarray(qkv[:, i * hidden:(i + 1) * hidden].reshape(T, n_heads, D)) for i in range(3))
    if rope_tables is not None:
        q, k = rope(q, *rope_tables), rope(k, *rope_tables)
    dq, dk, dv = attn_bwd(np.ascontiguousarray(do), q, k, v, cu_seqlens, scale)
    if rope_tables is not None:   # the transpose of a rotation is the rotation by the opposite angle
        c, s_ = rope_tables
        dq, dk = rope(dq, c, -np.asarray(s_)), rope(dk, c, -np.asarray(s_))
    dqkv = np.concatenate([t.reshape(T, hidden) for t in (dq, dk, dv)], axis=1)
    g["w_qkv"], g["b_qkv"] = linear_wgrad(dqkv, p["a"])
    da = linear_dgrad(dqkv, w.wqkv)
    dln, g["ln1_gamma"], g["ln1_beta"] = layernorm_bwd(x, da, w.g1, eps)
    return dx1 + dln, g
