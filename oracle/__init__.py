"""CPU oracle for the encoder hot path -- TEST INFRASTRUCTURE, not product code.

Only ``tests/``, ``__graft_entry__.smoke()`` and the CPU-baseline / reference legs of
``bench.py`` may import this package.  It never imports the CUDA package and shares no
code with it.

What it states, in fp64 and without any tiling or reordering:

* ``attn_fwd`` / ``attn_bwd``: per-image (block-diagonal) multi-head softmax attention over a
  packed token sequence and its exact gradient -- the computation the transpose schedule
  moves into the pipeline bubbles (Section 4.2, instantiation <transpose,1f1b>; the backward
  exists only when the encoder is trainable, Lemma 1).  The arithmetic lives in
  ``mpipe_oracle.c`` (plain C, compiled on first use with gcc).
* ``merge_tokens`` / ``merge_tokens_bwd``: the local half of the Replicated->Sharded seam of
  Table 2 ("Gather" forward, gated "Scatter" backward): a row scatter / row gather on raw
  16-bit words.
* ``seg_plan``: the integer planning rule (prefix sum of patch counts, longest-segment-first
  tile list), restated with Python's stable sort.

Pins: ``tests/test_oracle_attention.py``, ``tests/test_oracle_merge_plan.py``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import List, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mpipe_oracle.c")
_SO = os.path.join(_HERE, "libmpipe_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (-O2, OpenMP, no fast-math).  Returns the .so path."""
    stale = (not os.path.exists(_SO)) or os.path.getmtime(_SO) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _SO + f".{os.getpid()}.tmp"
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-ffp-contract=off",
               "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
    return _lib


def n_threads() -> int:
    """Threads the C oracle uses (OpenMP default = cores in the affinity mask, or OMP_NUM_THREADS)."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env.split(",")[0])
    return len(os.sched_getaffinity(0))


def _u16(a: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, "bf16 tensors are passed as uint16 bit patterns"
    return a


def _f64(a: np.ndarray) -> np.ndarray:
    """Attention inputs: bf16 bit patterns (uint16) are widened exactly; fp64 arrays pass through
    (used by the finite-difference pin, whose perturbed inputs are not bf16 numbers)."""
    a = np.asarray(a)
    if a.dtype == np.uint16:
        return (np.ascontiguousarray(a).astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    assert a.dtype == np.float64
    return np.ascontiguousarray(a)


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _cu(cu) -> np.ndarray:
    cu = np.ascontiguousarray(np.asarray(cu, dtype=np.int32))
    assert cu.ndim == 1 and cu.size >= 1 and cu[0] == 0 and np.all(np.diff(cu) >= 0)
    return cu


def attn_fwd(q, k, v, cu_seqlens, scale: float) -> Tuple[np.ndarray, np.ndarray]:
    """Full forward.  q,k,v: bf16 bits (uint16) or fp64, [T,H,D].  Returns O fp64 [T,H,D] and LSE fp64 [H,T]."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    T, H, D = q.shape
    cu = _cu(cu_seqlens)
    assert cu[-1] == T
    O = np.zeros((T, H, D), dtype=np.float64)
    LSE = np.zeros((H, T), dtype=np.float64)
    rc = _load().mo_attn_fwd(_p(q), _p(k), _p(v), ctypes.c_int64(T), H, D, _p(cu), cu.size - 1,
                             ctypes.c_float(scale), _p(O), _p(LSE))
    assert rc == 0
    return O, LSE


def attn_bwd(dout, q, k, v, cu_seqlens, scale: float):
    """Full backward.  Returns dQ, dK, dV fp64 [T,H,D]."""
    dout, q, k, v = _f64(dout), _f64(q), _f64(k), _f64(v)
    T, H, D = q.shape
    cu = _cu(cu_seqlens)
    assert cu[-1] == T
    dQ = np.zeros((T, H, D), dtype=np.float64)
    dK = np.zeros_like(dQ)
    dV = np.zeros_like(dQ)
    rc = _load().mo_attn_bwd(_p(dout), _p(q), _p(k), _p(v), ctypes.c_int64(T), H, D, _p(cu),
                             cu.size - 1, ctypes.c_float(scale), _p(dQ), _p(dK), _p(dV))
    assert rc == 0
    return dQ, dK, dV


def attn_fwd_rows(q, k, v, cu_seqlens, scale: float, rows, heads):
    """Forward for sampled (token row, head) pairs.  Returns O [n,D], LSE [n]."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    T, H, D = q.shape
    cu = _cu(cu_seqlens)
    rows = np.ascontiguousarray(np.asarray(rows, dtype=np.int64))
    heads = np.ascontiguousarray(np.asarray(heads, dtype=np.int32))
    n = rows.size
    assert heads.size == n
    O = np.zeros((n, D), dtype=np.float64)
    LSE = np.zeros((n,), dtype=np.float64)
    rc = _load().mo_attn_fwd_rows(_p(q), _p(k), _p(v), ctypes.c_int64(T), H, D, _p(cu), cu.size - 1,
                                  ctypes.c_float(scale), _p(rows), _p(heads), ctypes.c_int64(n),
                                  _p(O), _p(LSE))
    assert rc == 0, "a sampled row lies in no segment"
    return O, LSE


def attn_bwd_dq_rows(dout, q, k, v, cu_seqlens, scale: float, rows, heads):
    """dQ for sampled (token row, head) pairs.  Returns [n,D]."""
    dout, q, k, v = _f64(dout), _f64(q), _f64(k), _f64(v)
    T, H, D = q.shape
    cu = _cu(cu_seqlens)
    rows = np.ascontiguousarray(np.asarray(rows, dtype=np.int64))
    heads = np.ascontiguousarray(np.asarray(heads, dtype=np.int32))
    n = rows.size
    dQ = np.zeros((n, D), dtype=np.float64)
    rc = _load().mo_attn_bwd_dq_rows(_p(dout), _p(q), _p(k), _p(v), ctypes.c_int64(T), H, D, _p(cu),
                                     cu.size - 1, ctypes.c_float(scale), _p(rows), _p(heads),
                                     ctypes.c_int64(n), _p(dQ))
    assert rc == 0
    return dQ


def attn_bwd_dkv_rows(dout, q, k, v, cu_seqlens, scale: float, seg: int, head: int, rows):
    """dK, dV for sampled key rows of one (segment, head).  Returns two [n,D] arrays."""
    dout, q, k, v = _f64(dout), _f64(q), _f64(k), _f64(v)
    T, H, D = q.shape
    cu = _cu(cu_seqlens)
    rows = np.ascontiguousarray(np.asarray(rows, dtype=np.int64))
    n = rows.size
    dK = np.zeros((n, D), dtype=np.float64)
    dV = np.zeros((n, D), dtype=np.float64)
    rc = _load().mo_attn_bwd_dkv_rows(_p(dout), _p(q), _p(k), _p(v), ctypes.c_int64(T), H, D, _p(cu),
                                      cu.size - 1, ctypes.c_float(scale), int(seg), int(head),
                                      _p(rows), ctypes.c_int64(n), _p(dK), _p(dV))
    assert rc == 0
    return dK, dV


def merge_tokens(enc, llm_embeds, positions) -> np.ndarray:
    """out = copy(llm_embeds); out[positions[i], :] = enc[i, :]  (uint16 words, bit-exact)."""
    enc, emb = _u16(enc), _u16(llm_embeds)
    pos = np.ascontiguousarray(np.asarray(positions, dtype=np.int32))
    n_enc = pos.size
    n_llm, hidden = emb.shape
    assert enc.shape == (n_enc, hidden)
    out = np.empty_like(emb)
    rc = _load().mo_merge_tokens(_p(enc), _p(emb), _p(out), _p(pos), ctypes.c_int64(n_enc),
                                 ctypes.c_int64(n_llm), ctypes.c_int64(hidden))
    assert rc == 0, "position out of range"
    return out


def merge_tokens_bwd(d_emb, positions) -> np.ndarray:
    """d_enc[i, :] = d_emb[positions[i], :]  (uint16 words, bit-exact)."""
    d_emb = _u16(d_emb)
    pos = np.ascontiguousarray(np.asarray(positions, dtype=np.int32))
    n_llm, hidden = d_emb.shape
    d_enc = np.zeros((pos.size, hidden), dtype=np.uint16)
    rc = _load().mo_merge_tokens_bwd(_p(d_emb), _p(d_enc), _p(pos), ctypes.c_int64(pos.size),
                                     ctypes.c_int64(n_llm), ctypes.c_int64(hidden))
    assert rc == 0
    return d_enc


WorkItem = Tuple[int, int, int, int, int, int]  # seg, tile, row_start, row_len, kv_start, kv_len


def _tile_items(counts: Sequence[int], cu: Sequence[int], tile_rows: int) -> List[WorkItem]:
    order = sorted(range(len(counts)), key=lambda i: -counts[i])  # stable: ties keep index order
    items: List[WorkItem] = []
    for i in order:
        n = counts[i]
        if n == 0:
            continue
        for t in range((n + tile_rows - 1) // tile_rows):
            items.append((i, t, cu[i] + t * tile_rows, min(tile_rows, n - t * tile_rows), cu[i], n))
    return items


def seg_plan(patch_counts: Sequence[int], fwd_tile_rows: int, bwd_tile_rows: int, trained: bool):
    """The planning rule: cu = exclusive prefix sum; segments longest first (ties by index);
    one item per tile of each non-empty segment.  Forward items tile the query rows, backward
    items tile the key/value rows; a frozen encoder has no backward items (Lemma 1).

    Returns (cu_seqlens, total_tokens, max_seqlen, fwd_items, bwd_items) as Python ints/lists.
    """
    counts = [int(c) for c in patch_counts]
    assert all(c >= 0 for c in counts)
    cu = [0]
    for c in counts:
        cu.append(cu[-1] + c)
    fwd = _tile_items(counts, cu, fwd_tile_rows)
    bwd = _tile_items(counts, cu, bwd_tile_rows) if trained else []
    return cu, cu[-1], (max(counts) if counts else 0), fwd, bwd


# ---------------------------------------------------------------------------------------------------
# Cost model of the transpose schedule (Section 4.3), restated plainly
# ---------------------------------------------------------------------------------------------------

def event_cost(flops: float, nbytes: float, peak_flops: float, peak_bw: float) -> float:
    """cost(Fwd) = cost(Bwd) = max(W / F, D / B)."""
    return max(flops / peak_flops, nbytes / peak_bw)


def coll_cost(alpha: float, beta: float, payload_bytes: float) -> float:
    """cost(Coll) = alpha + beta * n."""
    return alpha + beta * payload_bytes


def encoder_attn_work(patch_counts: Sequence[int], n_heads: int, head_dim: int, trained: bool):
    """FLOPs and HBM bytes of the attention events of one encoder microbatch."""
    n1 = sum(int(c) for c in patch_counts)
    n2 = sum(int(c) * int(c) for c in patch_counts)
    fwd_flops = 4 * n_heads * head_dim * n2
    fwd_bytes = n1 * n_heads * (8 * head_dim + (4 if trained else 0))
    bwd_flops = 10 * n_heads * head_dim * n2 if trained else 0
    bwd_bytes = n1 * n_heads * (16 * head_dim + 16) if trained else 0
    return float(fwd_flops), float(fwd_bytes), float(bwd_flops), float(bwd_bytes)


def spills(owner: Sequence[int], enc_cost: Sequence[float], warmup_slack: Sequence[float]):
    """E_r = sum of the encoder costs rank r owns; spill_r = max(0, E_r - w_r)."""
    work = [0.0] * len(warmup_slack)
    for m, r in enumerate(owner):
        work[r] += enc_cost[m]
    sp = [max(0.0, e - w) for e, w in zip(work, warmup_slack)]
    return work, sp, (max(sp) if sp else 0.0)


def owner_map_greedy(enc_cost: Sequence[float], warmup_slack: Sequence[float]):
    """Heaviest encode first, each to the rank with the most warm-up slack left (ties: lower index / rank)."""
    work = [0.0] * len(warmup_slack)
    owner = [0] * len(enc_cost)
    for m in sorted(range(len(enc_cost)), key=lambda i: -enc_cost[i]):
        left = [w - e for w, e in zip(warmup_slack, work)]
        r = max(range(len(left)), key=lambda i: (left[i], -i))
        owner[m] = r
        work[r] += enc_cost[m]
    return owner


def owner_map_optimal(enc_cost: Sequence[float], warmup_slack: Sequence[float]):
    """Brute force over all assignments (tiny inputs only): the smallest achievable max_r spill_r."""
    import itertools
    best = None
    for owner in itertools.product(range(len(warmup_slack)), repeat=len(enc_cost)):
        mx = spills(owner, enc_cost, warmup_slack)[2]
        best = mx if best is None or mx < best else best
    return 0.0 if best is None else best
