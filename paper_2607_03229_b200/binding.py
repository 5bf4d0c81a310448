"""ctypes binding of libmpipe_enc.so: argument marshalling only.

Every function has the name of the C entry point without the ``mpipe_`` prefix and forwards
to it; all arithmetic of the hot path runs in the CUDA kernels behind the C ABI
(``include/mpipe_enc.h``).  torch is used for device memory and streams only.  There is no
CPU fallback: if the shared library is missing the import of this module's functions fails.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import List, Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmpipe_enc.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT, ERR_INDEX = range(7)
FROZEN, TRAINED = 0, 1

_lib = None


class WorkItem(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("seg", "tile", "row_start", "row_len", "kv_start", "kv_len")]


ITEM_DTYPE = np.dtype([(n, np.int32) for n in ("seg", "tile", "row_start", "row_len", "kv_start", "kv_len")])

_i32, _i64, _vp, _f32, _sz = ctypes.c_int32, ctypes.c_int64, ctypes.c_void_p, ctypes.c_float, ctypes.c_size_t
_SIGNATURES = {
    "mpipe_encoder_workspace_bytes": (_sz, [_i32, _i32, _i32, _i32, _i32]),
    "mpipe_encoder_bwd_workspace_bytes": (_sz, [_i32, _i32, _i32, _i32]),
    "mpipe_encoder_fwd": (_i32, [_vp, _vp, _vp, _i32, _i32, _i32, _i32, _i32, _vp, _i32, _i32, _vp, _i32, _f32, _f32, _vp, _vp,
                                 _i32, _vp, _vp, _sz, _vp, _vp]),
    "mpipe_encoder_bwd": (_i32, [_vp, _vp, _vp, _vp, _vp, _i32, _i32, _i32, _i32, _i32, _vp, _i32, _i32, _vp, _i32, _f32, _f32,
                                 _vp, _vp, _i32, _vp, _vp, _vp, _sz, _vp, _vp]),
    "mpipe_encoder_layer_bwd_workspace_bytes": (_sz, [_i32, _i32, _i32, _i32]),
    "mpipe_encoder_layer_bwd": (_i32, [_vp, _vp, _vp, _vp, _vp, _i32, _i32, _i32, _i32, _vp, _i32, _i32, _vp, _i32, _f32, _f32,
                                       _vp, _vp, _i32, _vp, _vp, _vp, _sz, _vp, _vp]),
    "mpipe_rope_apply_bwd": (_i32, [_vp, _i64, _i64, _vp, _vp, _i32, _i32, _i32, _vp]),
    "mpipe_layernorm_bwd": (_i32, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _i32, _i32, _i64, _i64, _i64, _i64, _f32, _vp]),
    "mpipe_colsum_accumulate": (_i32, [_vp, _vp, _i32, _i32, _i64, _vp]),
    "mpipe_linear_wgrad": (_i32, [_vp, _vp, _vp, _i32, _i32, _i32, _i64, _i64, _i64, _vp, _vp]),
    "mpipe_linear_dgrad": (_i32, [_vp, _vp, _vp, _vp, _vp, _i32, _i32, _i32, _i64, _i64, _i64, _i64, _i64, _vp, _vp]),
    "mpipe_ipc_handle_bytes": (_i32, []),
    "mpipe_ipc_export": (_i32, [_vp, _vp]),
    "mpipe_ipc_open": (_i32, [_vp, _vp]),
    "mpipe_ipc_close": (_i32, [_vp]),
    "mpipe_stage_index": (_i32, [_i32, _i32, _i32]),
    "mpipe_schedule_valid": (_i32, [_vp, _vp, _i32, _i32]),
    "mpipe_schedule_normalize": (_i32, [_vp, _vp, _i32, _i32, _vp, _vp, _vp]),
    "mpipe_derive": (_i32, [_vp, _vp, _i32, _i32, _vp, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i32, _vp, _vp, _i32,
                            _vp, _vp, _vp]),
    "mpipe_order_makespan": (_i32, [_vp, _i32, _vp, _i32, _vp, _i32, _vp, _vp, _vp]),
    "mpipe_linear_fwd": (_i32, [_vp, _vp, _vp, _vp, _vp, _i32, _i32, _i32, _i64, _i64, _i64, _i64, _i32, _vp, _vp]),
    "mpipe_layernorm_fwd": (_i32, [_vp, _vp, _vp, _vp, _i32, _i32, _i64, _i64, _f32, _vp]),
    "mpipe_encoder_layer_workspace_bytes": (_sz, [_i32, _i32, _i32]),
    "mpipe_encoder_layer_fwd": (_i32, [_vp, _vp, _vp, _i32, _i32, _i32, _i32, _vp, _i32, _i32, _vp, _i32, _f32, _f32,
                                       _vp, _vp, _i32, _vp, _vp, _sz, _vp, _vp]),
    "mpipe_rope_apply": (_i32, [_vp, _i64, _i64, _vp, _vp, _i32, _i32, _i32, _vp]),
    "mpipe_fwd_tile_rows": (_i32, []),
    "mpipe_bwd_tile_rows": (_i32, []),
    "mpipe_seg_plan": (_i32, [_vp, _i32, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "mpipe_attn_workspace_bytes": (_sz, [_i32, _i32, _i32, _i32]),
    "mpipe_varlen_attn_fwd": (_i32, [_vp, _vp, _vp, _vp, _vp, _i64, _i64, _i64, _i64, _vp, _i32, _i32, _i32, _vp,
                                     _i32, _i32, _i32, _f32, _i32, _vp, _vp]),
    "mpipe_varlen_attn_bwd": (_i32, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i64, _i64, _i64, _i64, _i64, _i64,
                                     _vp, _i32, _i32, _i32, _vp, _i32, _i32, _i32, _f32, _i32, _vp, _sz, _vp, _vp]),
    "mpipe_attn_bwd_static_scratch_bytes": (_sz, []),
    "mpipe_varlen_attn_bwd_static": (_i32, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _i64, _i64, _i64, _i64, _i64,
                                            _i64, _vp, _i32, _i32, _i32, _vp, _i32, _i32, _i32, _f32, _i32, _vp, _vp]),
    "mpipe_merge_tokens": (_i32, [_vp, _i64, _vp, _i64, _vp, _i32, _i32, _i32, _i32, _vp, _vp]),
    "mpipe_merge_tokens_bwd": (_i32, [_vp, _i64, _vp, _i64, _vp, _i32, _i32, _i32, _i32, _vp, _vp]),
    "mpipe_validate_positions": (_i32, [_vp, _i32, _i32]),
    "mpipe_set_profile_events": (_i32, [_i32, _vp, _vp]),
    "mpipe_selftest_wait_timeout": (_i32, [_i64, _vp, _vp]),
    "mpipe_event_cost": (_i32, [ctypes.c_double] * 4 + [_vp]),
    "mpipe_coll_cost": (_i32, [ctypes.c_double] * 3 + [_vp]),
    "mpipe_encoder_attn_work": (_i32, [_vp, _i32, _i32, _i32, _i32, _vp, _vp, _vp, _vp]),
    "mpipe_warmup_slack_1f1b": (_i32, [_i32, ctypes.c_double, ctypes.c_double, _vp]),
    "mpipe_owner_map": (_i32, [_vp, _i32, _vp, _i32, _vp, _vp, _vp, _vp]),
    "mpipe_status_str": (ctypes.c_char_p, [_i32]),
    "mpipe_version": (_i32, []),
}
EXPORTED_SYMBOLS = tuple(_SIGNATURES)


def load() -> ctypes.CDLL:
    """Load the shared library (built in-tree by ``build.py``); raises if it is not there."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2607_03229_b200.build` "
                "(there is no fallback path)")
        lib = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


class MpipeError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {load().mpipe_status_str(status).decode()} (status {status})")


def _check(status: int, where: str) -> None:
    if status != OK:
        raise MpipeError(status, where)


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        return t.data_ptr() if t.numel() else None
    if isinstance(t, np.ndarray):
        return t.ctypes.data if t.size else None
    return int(t)


def _stream(stream) -> Optional[int]:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream or None
    return getattr(stream, "cuda_stream", stream) or None


def fwd_tile_rows() -> int:
    return load().mpipe_fwd_tile_rows()


def bwd_tile_rows() -> int:
    return load().mpipe_bwd_tile_rows()


def version() -> int:
    return load().mpipe_version()


def status_str(status: int) -> str:
    return load().mpipe_status_str(status).decode()


@dataclass
class SegPlan:
    """Host result of ``seg_plan`` plus (after ``to_device``) the device copies the kernels read."""
    mode: int
    cu_seqlens: np.ndarray          # int32 [n_seg + 1]
    total_tokens: int
    max_seqlen: int
    fwd_items: np.ndarray           # ITEM_DTYPE [n_fwd]
    bwd_items: np.ndarray           # ITEM_DTYPE [n_bwd]
    cu_seqlens_dev: Optional[torch.Tensor] = None
    fwd_items_dev: Optional[torch.Tensor] = None
    bwd_items_dev: Optional[torch.Tensor] = None
    _host_staging: Optional[torch.Tensor] = None

    @property
    def n_seg(self) -> int:
        return self.cu_seqlens.size - 1

    def to_device(self, device="cuda") -> "SegPlan":
        """Upload cu_seqlens and both item lists with ONE asynchronous copy from a pinned staging buffer
        (stream-ordered on the current stream; the host does not wait for the device)."""
        parts = [np.ascontiguousarray(self.cu_seqlens).view(np.int32).reshape(-1),
                 np.ascontiguousarray(self.fwd_items).view(np.int32).reshape(-1),
                 np.ascontiguousarray(self.bwd_items).view(np.int32).reshape(-1)]
        sizes = [x.size for x in parts]
        offs = np.concatenate([[0], np.cumsum([(n + 3) // 4 * 4 for n in sizes])])   # 16-byte aligned sections
        total = int(offs[-1])
        host = torch.empty(max(total, 4), dtype=torch.int32)
        if torch.device(device).type == "cuda":
            host = host.pin_memory()
        hv = host.numpy()
        for x, o, n in zip(parts, offs[:-1], sizes):
            hv[o:o + n] = x
        dev = host.to(device, non_blocking=True)
        self._host_staging = host     # keep the pinned buffer alive until the copy has run
        self.cu_seqlens_dev = dev[offs[0]:offs[0] + sizes[0]]
        self.fwd_items_dev = dev[offs[1]:offs[1] + sizes[1]].view(-1, 6)
        self.bwd_items_dev = dev[offs[2]:offs[2] + sizes[2]].view(-1, 6)
        return self


def seg_plan(patch_counts, mode: int, fwd_rows: Optional[int] = None, bwd_rows: Optional[int] = None) -> SegPlan:
    """mpipe_seg_plan with the two-call pattern (count, then fill).  Host only."""
    lib = load()
    counts = np.ascontiguousarray(np.asarray(patch_counts, dtype=np.int32).reshape(-1))
    n_seg = counts.size
    fwd_rows = fwd_tile_rows() if fwd_rows is None else fwd_rows
    bwd_rows = bwd_tile_rows() if bwd_rows is None else bwd_rows
    cu = np.zeros(n_seg + 1, dtype=np.int32)
    total, mx, nf, nb = (ctypes.c_int32() for _ in range(4))
    args = (_ptr(counts), n_seg, fwd_rows, bwd_rows, mode, _ptr(cu), ctypes.addressof(total), ctypes.addressof(mx))
    _check(lib.mpipe_seg_plan(*args, None, ctypes.addressof(nf), None, ctypes.addressof(nb)), "mpipe_seg_plan")
    fwd = np.zeros(nf.value, dtype=ITEM_DTYPE)
    bwd = np.zeros(nb.value, dtype=ITEM_DTYPE)
    _check(lib.mpipe_seg_plan(*args, _ptr(fwd), ctypes.addressof(nf), _ptr(bwd), ctypes.addressof(nb)),
           "mpipe_seg_plan")
    return SegPlan(mode, cu, total.value, mx.value, fwd, bwd)


def attn_workspace_bytes(total_tokens: int, n_heads: int, head_dim: int, mode: int) -> int:
    return load().mpipe_attn_workspace_bytes(total_tokens, n_heads, head_dim, mode)


def _thd_strides(t: torch.Tensor):
    assert t.dim() == 3 and t.stride(2) == 1, "expected [tokens, heads, head_dim] with contiguous head_dim"
    return t.stride(0), t.stride(1)


def _check_plan(plan: SegPlan, T: int, items_dev, n_items: int, what: str) -> None:
    """The plan must have been made for these tensors and uploaded: the kernels index the tensors with the
    rows its items name."""
    assert plan.total_tokens == T, f"{what}: plan was made for {plan.total_tokens} tokens, tensors hold {T}"
    if T > 0 and n_items > 0:
        assert items_dev is not None and plan.cu_seqlens_dev is not None, f"{what}: plan.to_device() first"
        assert items_dev.numel() == 6 * n_items and items_dev.dtype == torch.int32


def varlen_attn_fwd(q, k, v, o, lse, plan: SegPlan, softmax_scale: float, status_buf=None, stream=None) -> None:
    """mpipe_varlen_attn_fwd.  q,k,v,o: bf16 CUDA tensors [T,H,D]; lse: fp32 [H,T] or None (frozen)."""
    T, H, D = q.shape
    assert k.shape == q.shape and v.shape == q.shape and o.shape == q.shape
    assert q.dtype == k.dtype == v.dtype == o.dtype == torch.bfloat16
    _check_plan(plan, T, plan.fwd_items_dev, int(plan.fwd_items.size), "varlen_attn_fwd")
    ts, hs = _thd_strides(q)
    assert _thd_strides(k) == (ts, hs) and _thd_strides(v) == (ts, hs), "q, k, v must share strides"
    tso, hso = _thd_strides(o)
    if lse is not None:
        assert lse.dtype == torch.float32 and lse.is_contiguous() and tuple(lse.shape) == (H, T)
    st = load().mpipe_varlen_attn_fwd(
        _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), ts, hs, tso, hso, _ptr(plan.cu_seqlens_dev), plan.n_seg,
        plan.total_tokens, plan.max_seqlen, _ptr(plan.fwd_items_dev), int(plan.fwd_items.size), H, D,
        softmax_scale, plan.mode, _ptr(status_buf), _stream(stream))
    _check(st, "mpipe_varlen_attn_fwd")


def _bwd_args(what, dout, q, k, v, o, lse, dq, dk, dv, plan: SegPlan, softmax_scale: float):
    """Shape / dtype / stride checks and argument marshalling shared by the two backward entry points."""
    T, H, D = q.shape
    ts, hs = _thd_strides(q)
    tso, hso = _thd_strides(o)
    if plan.mode == TRAINED:
        for name, t in (("k", k), ("v", v), ("o", o), ("dout", dout), ("dq", dq), ("dk", dk), ("dv", dv)):
            assert tuple(t.shape) == (T, H, D) and t.dtype == torch.bfloat16, f"{what}: {name} must be bf16 {(T, H, D)}"
        assert lse.dtype == torch.float32 and lse.is_contiguous() and tuple(lse.shape) == (H, T)
        _check_plan(plan, T, plan.bwd_items_dev, int(plan.bwd_items.size), what)
        assert _thd_strides(k) == (ts, hs) and _thd_strides(v) == (ts, hs), "q, k, v must share strides"
        assert _thd_strides(dout) == (tso, hso), "dout must share o's strides"
        tsg, hsg = _thd_strides(dq)
        assert _thd_strides(dk) == (tsg, hsg) and _thd_strides(dv) == (tsg, hsg), "dq, dk, dv must share strides"
    else:
        tsg, hsg = ts, hs
    return (_ptr(dout), _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _ptr(dq), _ptr(dk), _ptr(dv), ts, hs, tso, hso,
            tsg, hsg, _ptr(plan.cu_seqlens_dev), plan.n_seg, plan.total_tokens, plan.max_seqlen,
            _ptr(plan.bwd_items_dev), int(plan.bwd_items.size), H, D, softmax_scale, plan.mode)


def varlen_attn_bwd(dout, q, k, v, o, lse, dq, dk, dv, plan: SegPlan, softmax_scale: float, workspace,
                    status_buf=None, stream=None) -> None:
    """mpipe_varlen_attn_bwd.  A frozen plan returns at once (nothing is launched)."""
    args = _bwd_args("varlen_attn_bwd", dout, q, k, v, o, lse, dq, dk, dv, plan, softmax_scale)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    st = load().mpipe_varlen_attn_bwd(*args, _ptr(workspace), ws_bytes, _ptr(status_buf), _stream(stream))
    _check(st, "mpipe_varlen_attn_bwd")


LINEAR_GELU = 1


def _rows(t):
    assert t.dim() == 2 and t.stride(1) == 1 and t.dtype == torch.bfloat16
    return t.stride(0)


def linear_fwd(a, w, c, bias=None, residual=None, gelu: bool = False, status_buf=None, stream=None) -> None:
    """mpipe_linear_fwd: c[M,N] = act(a[M,K] w[N,K]^T + bias) + residual (bf16 CUDA tensors, rows contiguous)."""
    M, K = a.shape
    N = w.shape[0]
    assert w.shape[1] == K and tuple(c.shape) == (M, N)
    if bias is not None:
        assert bias.dtype == torch.bfloat16 and bias.is_contiguous() and bias.numel() == N
    st = load().mpipe_linear_fwd(_ptr(a), _ptr(w), _ptr(bias), _ptr(residual), _ptr(c), M, N, K, _rows(a), _rows(w),
                                 0 if residual is None else _rows(residual), _rows(c), LINEAR_GELU if gelu else 0,
                                 _ptr(status_buf), _stream(stream))
    _check(st, "mpipe_linear_fwd")


def linear_dgrad(dy, w, dx, gelu_input=None, residual=None, status_buf=None, stream=None) -> None:
    """mpipe_linear_dgrad: dx[M,K] = (dy[M,N] w[N,K]) o GELU'(gelu_input) + residual (bf16 CUDA tensors)."""
    M, N = dy.shape
    K = w.shape[1]
    assert w.shape[0] == N and tuple(dx.shape) == (M, K)
    st = load().mpipe_linear_dgrad(_ptr(dy), _ptr(w), _ptr(gelu_input), _ptr(residual), _ptr(dx), M, N, K, _rows(dy), _rows(w),
                                   0 if gelu_input is None else _rows(gelu_input), 0 if residual is None else _rows(residual),
                                   _rows(dx), _ptr(status_buf), _stream(stream))
    _check(st, "mpipe_linear_dgrad")


def linear_wgrad(dy, x, dw, status_buf=None, stream=None) -> None:
    """mpipe_linear_wgrad: dw[N,K] (fp32, accumulated in place) += dy[T,N]^T x[T,K]."""
    T, N = dy.shape
    K = x.shape[1]
    assert x.shape[0] == T and tuple(dw.shape) == (N, K) and dw.dtype == torch.float32 and dw.stride(1) == 1
    st = load().mpipe_linear_wgrad(_ptr(dy), _ptr(x), _ptr(dw), T, N, K, _rows(dy), _rows(x), dw.stride(0), _ptr(status_buf),
                                   _stream(stream))
    _check(st, "mpipe_linear_wgrad")


def layernorm_fwd(x, gamma, beta, y, eps: float, stream=None) -> None:
    """mpipe_layernorm_fwd over the rows of x [T, hidden] (bf16 CUDA tensors)."""
    T, hidden = x.shape
    assert tuple(y.shape) == (T, hidden) and gamma.numel() == hidden and beta.numel() == hidden
    assert gamma.dtype == beta.dtype == torch.bfloat16 and gamma.is_contiguous() and beta.is_contiguous()
    st = load().mpipe_layernorm_fwd(_ptr(x), _ptr(gamma), _ptr(beta), _ptr(y), T, hidden, _rows(x), _rows(y), eps,
                                    _stream(stream))
    _check(st, "mpipe_layernorm_fwd")


def rope_apply_bwd(dqkv, cos, sin, n_heads: int, head_dim: int, stream=None) -> None:
    """mpipe_rope_apply_bwd in place on the dq and dk column blocks of a packed gradient dqkv [T, 3*hidden]."""
    T = dqkv.shape[0]
    hidden = n_heads * head_dim
    assert dqkv.shape[1] == 3 * hidden and dqkv.dtype == torch.bfloat16 and dqkv.stride(1) == 1
    st = load().mpipe_rope_apply_bwd(_ptr(dqkv), dqkv.stride(0), hidden, _ptr(cos), _ptr(sin), T, n_heads, head_dim, _stream(stream))
    _check(st, "mpipe_rope_apply_bwd")


def layernorm_bwd(x, dy, gamma, dx, dgamma, dbeta, eps: float, dres=None, stream=None) -> None:
    """mpipe_layernorm_bwd; dgamma, dbeta: fp32 [hidden] CUDA tensors that are accumulated into."""
    T, hidden = x.shape
    assert dgamma.dtype == dbeta.dtype == torch.float32 and dgamma.numel() == dbeta.numel() == hidden
    st = load().mpipe_layernorm_bwd(_ptr(x), _ptr(dy), _ptr(gamma), _ptr(dres), _ptr(dx), _ptr(dgamma), _ptr(dbeta), T, hidden,
                                    _rows(x), _rows(dy), 0 if dres is None else _rows(dres), _rows(dx), eps, _stream(stream))
    _check(st, "mpipe_layernorm_bwd")


def colsum_accumulate(a, out, stream=None) -> None:
    """mpipe_colsum_accumulate: out[j] (fp32) += sum over rows of a[:, j] (bf16)."""
    T, N = a.shape
    assert out.dtype == torch.float32 and out.numel() == N
    _check(load().mpipe_colsum_accumulate(_ptr(a), _ptr(out), T, N, _rows(a), _stream(stream)), "mpipe_colsum_accumulate")


class LayerWeights(ctypes.Structure):
    """mpipe_layer_weights_t: twelve device pointers.  ``from_tensors`` keeps the tensors alive."""
    _fields_ = [(n, ctypes.c_void_p) for n in ("ln1_gamma", "ln1_beta", "w_qkv", "b_qkv", "w_o", "b_o", "ln2_gamma",
                                               "ln2_beta", "w_fc1", "b_fc1", "w_fc2", "b_fc2")]

    @classmethod
    def from_tensors(cls, **tensors) -> "LayerWeights":
        w = cls()
        for name, _ in cls._fields_:
            t = tensors[name]
            assert t.dtype == torch.bfloat16 and t.is_cuda and t.is_contiguous(), name
            setattr(w, name, t.data_ptr())
        w._keep = tensors
        return w


class LayerGrads(ctypes.Structure):
    """mpipe_layer_grads_t: twelve fp32 device pointers, same order and shapes as LayerWeights; accumulated into."""
    _fields_ = LayerWeights._fields_

    @classmethod
    def from_tensors(cls, **tensors) -> "LayerGrads":
        g = cls()
        for name, _ in cls._fields_:
            t = tensors[name]
            assert t.dtype == torch.float32 and t.is_cuda and t.is_contiguous(), name
            setattr(g, name, t.data_ptr())
        g._keep = tensors
        return g


def encoder_layer_bwd_workspace_bytes(n_tokens: int, hidden: int, n_heads: int, ffn: int) -> int:
    return load().mpipe_encoder_layer_bwd_workspace_bytes(n_tokens, hidden, n_heads, ffn)


def encoder_layer_bwd(dy, x, dx, weights: LayerWeights, grads: LayerGrads, n_heads: int, ffn: int, plan: SegPlan,
                      softmax_scale: float, ln_eps: float, lse, fwd_workspace, workspace, status_buf=None, stream=None,
                      rope=None) -> None:
    """mpipe_encoder_layer_bwd: dy, x, dx bf16 [T, hidden] contiguous; fwd_workspace untouched since the matching forward."""
    T, hidden = x.shape
    assert dy.is_contiguous() and x.is_contiguous() and dx.is_contiguous()
    st = load().mpipe_encoder_layer_bwd(
        _ptr(dy), _ptr(x), _ptr(dx), ctypes.addressof(weights), ctypes.addressof(grads), T, hidden, n_heads, ffn,
        _ptr(plan.cu_seqlens_dev), plan.n_seg, plan.max_seqlen, _ptr(plan.bwd_items_dev), int(plan.bwd_items.size), softmax_scale,
        ln_eps, _ptr(None if rope is None else rope[0]), _ptr(None if rope is None else rope[1]), plan.mode, _ptr(lse),
        _ptr(fwd_workspace), _ptr(workspace), 0 if workspace is None else workspace.numel() * workspace.element_size(),
        _ptr(status_buf), _stream(stream))
    _check(st, "mpipe_encoder_layer_bwd")


def _struct_array(items):
    arr = (type(items[0]) * len(items))()
    for i, it in enumerate(items):
        ctypes.memmove(ctypes.addressof(arr) + i * ctypes.sizeof(it), ctypes.addressof(it), ctypes.sizeof(it))
    arr._keep = items
    return arr


def encoder_workspace_bytes(n_layers: int, n_tokens: int, hidden: int, ffn: int, mode: int) -> int:
    return load().mpipe_encoder_workspace_bytes(n_layers, n_tokens, hidden, ffn, mode)


def encoder_bwd_workspace_bytes(n_tokens: int, hidden: int, n_heads: int, ffn: int) -> int:
    return load().mpipe_encoder_bwd_workspace_bytes(n_tokens, hidden, n_heads, ffn)


def encoder_fwd(x, y, layers, n_heads: int, ffn: int, plan: SegPlan, softmax_scale: float, ln_eps: float, workspace, lse=None,
                status_buf=None, stream=None, rope=None) -> None:
    """mpipe_encoder_fwd: `layers` is a list of LayerWeights; lse fp32 [L, H, T] for a trained plan."""
    T, hidden = x.shape
    arr = _struct_array(layers)
    st = load().mpipe_encoder_fwd(
        _ptr(x), _ptr(y), ctypes.addressof(arr), len(layers), T, hidden, n_heads, ffn, _ptr(plan.cu_seqlens_dev), plan.n_seg,
        plan.max_seqlen, _ptr(plan.fwd_items_dev), int(plan.fwd_items.size), softmax_scale, ln_eps,
        _ptr(None if rope is None else rope[0]), _ptr(None if rope is None else rope[1]), plan.mode, _ptr(lse), _ptr(workspace),
        workspace.numel() * workspace.element_size(), _ptr(status_buf), _stream(stream))
    _check(st, "mpipe_encoder_fwd")


def encoder_bwd(dy, x, dx, layers, grads, n_heads: int, ffn: int, plan: SegPlan, softmax_scale: float, ln_eps: float, lse,
                fwd_workspace, workspace, status_buf=None, stream=None, rope=None) -> None:
    """mpipe_encoder_bwd: `layers` / `grads` are lists of LayerWeights / LayerGrads."""
    T, hidden = x.shape
    la, ga = _struct_array(layers), _struct_array(grads)
    st = load().mpipe_encoder_bwd(
        _ptr(dy), _ptr(x), _ptr(dx), ctypes.addressof(la), ctypes.addressof(ga), len(layers), T, hidden, n_heads, ffn,
        _ptr(plan.cu_seqlens_dev), plan.n_seg, plan.max_seqlen, _ptr(plan.bwd_items_dev), int(plan.bwd_items.size), softmax_scale,
        ln_eps, _ptr(None if rope is None else rope[0]), _ptr(None if rope is None else rope[1]), plan.mode, _ptr(lse),
        _ptr(fwd_workspace), _ptr(workspace), 0 if workspace is None else workspace.numel() * workspace.element_size(),
        _ptr(status_buf), _stream(stream))
    _check(st, "mpipe_encoder_bwd")


def encoder_layer_workspace_bytes(n_tokens: int, hidden: int, ffn: int) -> int:
    return load().mpipe_encoder_layer_workspace_bytes(n_tokens, hidden, ffn)


def rope_apply(qkv, cos, sin, n_heads: int, head_dim: int, stream=None) -> None:
    """mpipe_rope_apply in place on the q and k column blocks of a packed projection qkv [T, 3*hidden] (bf16, CUDA);
    cos, sin: fp32 [T, head_dim/2] contiguous CUDA tensors."""
    T = qkv.shape[0]
    hidden = n_heads * head_dim
    assert qkv.shape[1] == 3 * hidden and qkv.dtype == torch.bfloat16 and qkv.stride(1) == 1
    for t in (cos, sin):
        assert t.dtype == torch.float32 and t.is_contiguous() and tuple(t.shape) == (T, head_dim // 2)
    st = load().mpipe_rope_apply(_ptr(qkv), qkv.stride(0), hidden, _ptr(cos), _ptr(sin), T, n_heads, head_dim, _stream(stream))
    _check(st, "mpipe_rope_apply")


def encoder_layer_fwd(x, y, weights: LayerWeights, n_heads: int, ffn: int, plan: SegPlan, softmax_scale: float,
                      ln_eps: float, workspace, lse=None, status_buf=None, stream=None, rope=None) -> None:
    """mpipe_encoder_layer_fwd: x, y bf16 [T, hidden] contiguous CUDA tensors; lse fp32 [H, T] for a trained plan;
    rope = (cos, sin) fp32 [T, head_dim/2] CUDA tensors or None."""
    T, hidden = x.shape
    assert x.is_contiguous() and y.is_contiguous() and tuple(y.shape) == (T, hidden) and x.dtype == y.dtype == torch.bfloat16
    st = load().mpipe_encoder_layer_fwd(
        _ptr(x), _ptr(y), ctypes.addressof(weights), T, hidden, n_heads, ffn, _ptr(plan.cu_seqlens_dev), plan.n_seg,
        plan.max_seqlen, _ptr(plan.fwd_items_dev), int(plan.fwd_items.size), softmax_scale, ln_eps,
        _ptr(None if rope is None else rope[0]), _ptr(None if rope is None else rope[1]), plan.mode, _ptr(lse),
        _ptr(workspace), workspace.numel() * workspace.element_size(), _ptr(status_buf), _stream(stream))
    _check(st, "mpipe_encoder_layer_fwd")


def attn_bwd_static_scratch_bytes() -> int:
    return load().mpipe_attn_bwd_static_scratch_bytes()


def varlen_attn_bwd_static(dout, q, k, v, o, lse, dq, dk, dv, plan: SegPlan, softmax_scale: float, status_buf=None,
                           stream=None) -> None:
    """mpipe_varlen_attn_bwd_static: the backward with the library's built-in 32 MiB scratch, for callers
    that may not allocate device memory.  Same tensors as varlen_attn_bwd, no workspace argument; problems
    whose scratch would not fit are refused with ERR_WORKSPACE.  Calls sharing a device must not overlap."""
    args = _bwd_args("varlen_attn_bwd_static", dout, q, k, v, o, lse, dq, dk, dv, plan, softmax_scale)
    st = load().mpipe_varlen_attn_bwd_static(*args, _ptr(status_buf), _stream(stream))
    _check(st, "mpipe_varlen_attn_bwd_static")


def merge_tokens(enc_tokens, llm_embeds, positions_dev, mode: int = TRAINED, status_buf=None, stream=None) -> None:
    """mpipe_merge_tokens: llm_embeds[positions[i], :] = enc_tokens[i, :], in place."""
    n_enc = int(positions_dev.numel())
    n_llm, hidden = llm_embeds.shape
    assert enc_tokens.dtype == llm_embeds.dtype == torch.bfloat16 and positions_dev.dtype == torch.int32
    assert enc_tokens.shape[0] == n_enc and (n_enc == 0 or enc_tokens.shape[1] == hidden)
    assert llm_embeds.stride(1) == 1 and (n_enc == 0 or enc_tokens.stride(1) == 1)
    st = load().mpipe_merge_tokens(_ptr(enc_tokens), enc_tokens.stride(0) if n_enc else hidden, _ptr(llm_embeds),
                                   llm_embeds.stride(0), _ptr(positions_dev), n_enc, n_llm, hidden, mode,
                                   _ptr(status_buf), _stream(stream))
    _check(st, "mpipe_merge_tokens")


def merge_tokens_bwd(d_llm_embeds, d_enc, positions_dev, mode: int, status_buf=None, stream=None) -> None:
    """mpipe_merge_tokens_bwd: d_enc[i, :] = d_llm_embeds[positions[i], :]; no-op when frozen."""
    n_enc = int(positions_dev.numel())
    n_llm, hidden = d_llm_embeds.shape
    assert d_llm_embeds.dtype == torch.bfloat16 and positions_dev.dtype == torch.int32
    st = load().mpipe_merge_tokens_bwd(_ptr(d_llm_embeds), d_llm_embeds.stride(0), _ptr(d_enc),
                                       d_enc.stride(0) if n_enc else hidden, _ptr(positions_dev), n_enc, n_llm,
                                       hidden, mode, _ptr(status_buf), _stream(stream))
    _check(st, "mpipe_merge_tokens_bwd")


class PeerRows:
    """A [n_rows, hidden] bf16 matrix in ANOTHER process's device memory (opened from an IPC handle), usable as the
    `llm_embeds` of merge_tokens / the `d_llm_embeds` of merge_tokens_bwd: the cross-rank seam as one kernel."""

    def __init__(self, handle: bytes, n_rows: int, hidden: int, row_stride: int):
        self.n_rows, self.hidden, self.row_stride = n_rows, hidden, row_stride
        ptr = ctypes.c_void_p()
        buf = ctypes.create_string_buffer(handle, len(handle))
        _check(load().mpipe_ipc_open(ctypes.addressof(buf), ctypes.addressof(ptr)), "mpipe_ipc_open")
        self.ptr = ptr.value

    def close(self) -> None:
        if self.ptr:
            _check(load().mpipe_ipc_close(self.ptr), "mpipe_ipc_close")
            self.ptr = None


def ipc_export(t) -> bytes:
    """IPC handle of the allocation behind CUDA tensor t (which must start at the allocation's base: allocate it with
    `torch.empty` of at least 1 MiB or through a dedicated allocation so that it is not packed into a shared block)."""
    n = load().mpipe_ipc_handle_bytes()
    buf = ctypes.create_string_buffer(n)
    _check(load().mpipe_ipc_export(_ptr(t), ctypes.addressof(buf)), "mpipe_ipc_export")
    return buf.raw


def merge_tokens_peer(enc_tokens, peer: PeerRows, positions_dev, mode: int = TRAINED, status_buf=None, stream=None) -> None:
    """mpipe_merge_tokens with the destination in a peer's memory: the Gather seam (Table 2) as one kernel."""
    n_enc = int(positions_dev.numel())
    assert enc_tokens.dtype == torch.bfloat16 and enc_tokens.shape[1] == peer.hidden and enc_tokens.stride(1) == 1
    st = load().mpipe_merge_tokens(_ptr(enc_tokens), enc_tokens.stride(0), peer.ptr, peer.row_stride, _ptr(positions_dev),
                                   n_enc, peer.n_rows, peer.hidden, mode, _ptr(status_buf), _stream(stream))
    _check(st, "mpipe_merge_tokens")


def merge_tokens_bwd_peer(peer: PeerRows, d_enc, positions_dev, mode: int, status_buf=None, stream=None) -> None:
    """mpipe_merge_tokens_bwd reading the gradient rows from a peer's memory: the reverse (Scatter) seam."""
    n_enc = int(positions_dev.numel())
    st = load().mpipe_merge_tokens_bwd(peer.ptr, peer.row_stride, _ptr(d_enc), d_enc.stride(0), _ptr(positions_dev), n_enc,
                                       peer.n_rows, peer.hidden, mode, _ptr(status_buf), _stream(stream))
    _check(st, "mpipe_merge_tokens_bwd")


def event_cost(flops: float, nbytes: float, peak_flops: float, peak_bw: float) -> float:
    out = ctypes.c_double()
    _check(load().mpipe_event_cost(flops, nbytes, peak_flops, peak_bw, ctypes.addressof(out)), "mpipe_event_cost")
    return out.value


def coll_cost(alpha: float, beta: float, payload_bytes: float) -> float:
    out = ctypes.c_double()
    _check(load().mpipe_coll_cost(alpha, beta, payload_bytes, ctypes.addressof(out)), "mpipe_coll_cost")
    return out.value


def encoder_attn_work(patch_counts, n_heads: int, head_dim: int, mode: int):
    """(fwd_flops, fwd_bytes, bwd_flops, bwd_bytes) of one microbatch's attention events."""
    counts = np.ascontiguousarray(np.asarray(patch_counts, dtype=np.int32).reshape(-1))
    out = [ctypes.c_double() for _ in range(4)]
    _check(load().mpipe_encoder_attn_work(_ptr(counts), counts.size, n_heads, head_dim, mode,
                                          *[ctypes.addressof(x) for x in out]), "mpipe_encoder_attn_work")
    return tuple(x.value for x in out)


def warmup_slack_1f1b(n_ranks: int, stage_fwd_cost: float, seam_cost: float) -> np.ndarray:
    w = np.zeros(max(n_ranks, 0), dtype=np.float64)
    _check(load().mpipe_warmup_slack_1f1b(n_ranks, stage_fwd_cost, seam_cost, _ptr(w) if w.size else None),
           "mpipe_warmup_slack_1f1b")
    return w


def owner_map(enc_cost, warmup_slack):
    """mpipe_owner_map.  Returns (owner int32[M], E float64[P], spill float64[P], max_spill)."""
    cost = np.ascontiguousarray(np.asarray(enc_cost, dtype=np.float64).reshape(-1))
    slack = np.ascontiguousarray(np.asarray(warmup_slack, dtype=np.float64).reshape(-1))
    owner = np.zeros(cost.size, dtype=np.int32)
    work = np.zeros(slack.size, dtype=np.float64)
    spill = np.zeros(slack.size, dtype=np.float64)
    mx = ctypes.c_double()
    _check(load().mpipe_owner_map(_ptr(cost), cost.size, _ptr(slack), slack.size, _ptr(owner), _ptr(work), _ptr(spill),
                                  ctypes.addressof(mx)), "mpipe_owner_map")
    return owner, work, spill, mx.value


def selftest_wait_timeout(budget_cycles: int, status_buf, stream=None) -> None:
    """mpipe_selftest_wait_timeout: a wait that nothing satisfies must end with ERR_TIMEOUT in status_buf."""
    _check(load().mpipe_selftest_wait_timeout(int(budget_cycles), _ptr(status_buf), _stream(stream)),
           "mpipe_selftest_wait_timeout")


PROFILE_FWD, PROFILE_BWD_MAIN, PROFILE_MERGE = 0, 1, 2


def set_profile_events(which: int, start: Optional[torch.cuda.Event], stop: Optional[torch.cuda.Event]) -> None:
    """mpipe_set_profile_events: record two CUDA events around one kernel of the next calls (None = off)."""
    def handle(ev):
        if ev is None:
            return None
        ev.record()  # torch creates the underlying cudaEvent_t lazily, on the first record
        return ev.cuda_event
    _check(load().mpipe_set_profile_events(which, handle(start), handle(stop)), "mpipe_set_profile_events")


def validate_positions(positions, n_llm_tokens: int) -> int:
    pos = np.ascontiguousarray(np.asarray(positions, dtype=np.int32))
    return load().mpipe_validate_positions(_ptr(pos), pos.size, n_llm_tokens)


# ------------------------------------------------------------------------------------------------
# derive (Section 4.1) and the makespan read off its order graph (Section 4.3): host only
# ------------------------------------------------------------------------------------------------
SK_1F1B, SK_GPIPE, SK_TRANSPOSE = 0, 1, 2
LAYOUT_SHARDED, LAYOUT_REPLICATED = 0, 1
COMM_NONE, COMM_GATHER, COMM_SCATTER, COMM_SEND, COMM_RECVGRAD = range(5)
GROUP_REPLICA, GROUP_DATA = 0, 1
EV_FWD, EV_BWD, EV_COLL, EV_DPREDUCE, EV_LOSS, EV_STEPBARRIER = range(6)
EDGE_ACTIVATION, EDGE_GRADIENT, EDGE_TURNAROUND, EDGE_ACCUMULATE, EDGE_SEQUENCE = range(5)


def _i32arr(x):
    return np.ascontiguousarray(np.asarray(x, dtype=np.int32).reshape(-1))


def stage_index(rank: int, region: int, n_ranks: int) -> int:
    return load().mpipe_stage_index(rank, region, n_ranks)


def schedule_valid(skeletons, cut, n_layers: int) -> bool:
    sk, c = _i32arr(skeletons), _i32arr(cut)
    assert c.size == max(sk.size - 1, 0)
    return load().mpipe_schedule_valid(sk.ctypes.data, c.ctypes.data if c.size else None, sk.size, n_layers) == OK


def schedule_normalize(skeletons, cut, n_layers: int):
    """-> (skeletons, cut) with runs of adjacent transpose regions collapsed into one."""
    sk, c = _i32arr(skeletons), _i32arr(cut)
    out_sk, out_c, out_k = np.zeros(sk.size, np.int32), np.zeros(max(sk.size - 1, 1), np.int32), ctypes.c_int32(0)
    st = load().mpipe_schedule_normalize(sk.ctypes.data, c.ctypes.data if c.size else None, sk.size, n_layers,
                                         out_sk.ctypes.data, out_c.ctypes.data, ctypes.addressof(out_k))
    _check(st, "mpipe_schedule_normalize")
    return out_sk[:out_k.value].tolist(), out_c[:out_k.value - 1].tolist()


@dataclass
class Derived:
    """Output of mpipe_derive as numpy arrays (column meaning as in the header's structs)."""
    regions: np.ndarray       # [k, 4]  layout, first_layer, n_layers, skeleton
    slabs: np.ndarray         # [k, P, 2]
    seams: np.ndarray         # [k-1, 3] left_region, fwd_comm, bwd_comm
    reduces: np.ndarray       # [n, 2]  region, group
    events: np.ndarray        # [n, 6]  kind, region, rank, mb, comm, group
    edges: np.ndarray         # [n, 3]  src, dst, type
    nodes: List[List[int]]    # per rank, event indices in execution order


def derive(skeletons, cut, n_layers: int, trainable, n_ranks: int, n_microbatches: int, owner=None) -> Derived:
    sk, c, tr = _i32arr(skeletons), _i32arr(cut), _i32arr(trainable)
    k, P = sk.size, n_ranks
    assert tr.size == k and c.size == max(k - 1, 0)
    ow = None if owner is None else _i32arr(owner)
    regions, slabs = np.zeros((k, 4), np.int32), np.zeros((k, max(P, 1), 2), np.int32)
    seams, reduces = np.zeros((max(k - 1, 1), 3), np.int32), np.zeros((k, 2), np.int32)
    n_red, n_ev, n_ed = ctypes.c_int32(0), ctypes.c_int32(0), ctypes.c_int32(0)
    offsets = np.zeros(max(P, 1) + 1, np.int32)
    lib = load()

    def call(events, edges, order, ecap, dcap):
        return lib.mpipe_derive(sk.ctypes.data, c.ctypes.data if c.size else None, k, n_layers, tr.ctypes.data, P,
                                n_microbatches, None if ow is None else ow.ctypes.data, regions.ctypes.data,
                                slabs.ctypes.data, seams.ctypes.data, reduces.ctypes.data, ctypes.addressof(n_red),
                                None if events is None else events.ctypes.data, ecap, ctypes.addressof(n_ev),
                                None if edges is None else edges.ctypes.data, dcap, ctypes.addressof(n_ed),
                                None if order is None else order.ctypes.data, offsets.ctypes.data)
    st = call(None, None, None, 0, 0)          # first pass: sizes
    if st != ERR_WORKSPACE:
        _check(st, "mpipe_derive")
    events, edges = np.zeros((max(n_ev.value, 1), 6), np.int32), np.zeros((max(n_ed.value, 1), 3), np.int32)
    order = np.zeros(max(n_ev.value, 1), np.int32)
    _check(call(events, edges, order, n_ev.value, n_ed.value), "mpipe_derive")
    nodes = [order[offsets[r]:offsets[r + 1]].tolist() for r in range(P)]
    return Derived(regions, slabs, seams[:k - 1], reduces[:n_red.value], events[:n_ev.value], edges[:n_ed.value], nodes)


def order_makespan(events: np.ndarray, edges: np.ndarray, cost, n_ranks: int):
    """-> (T, start[n_events], bubble[n_ranks])."""
    ev, ed = np.ascontiguousarray(events, dtype=np.int32), np.ascontiguousarray(edges, dtype=np.int32)
    cs = np.ascontiguousarray(cost, dtype=np.float64)
    assert cs.size == ev.shape[0]
    T, start, bub = ctypes.c_double(0.0), np.zeros(ev.shape[0], np.float64), np.zeros(n_ranks, np.float64)
    st = load().mpipe_order_makespan(ev.ctypes.data, ev.shape[0], ed.ctypes.data if ed.size else None, ed.shape[0],
                                     cs.ctypes.data, n_ranks, ctypes.addressof(T), start.ctypes.data, bub.ctypes.data)
    _check(st, "mpipe_order_makespan")
    return T.value, start, bub
