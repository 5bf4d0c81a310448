"""Seeded synthetic inputs shaped like the paper's image/video mixes.

This module holds NO arithmetic of the method: only a counter-based random generator
(a 64-bit integer mixer -> uniforms -> Box-Muller normals -> bf16 bit patterns) and the
recipes that turn a seed into patch counts, placeholder positions and tensors.  Both the
CUDA path's tests/benchmark and the CPU oracle's tests take their inputs from here, so that
the two sides see bit-identical data.  Everything is numpy on the host; bf16 tensors are
returned as ``uint16`` bit patterns.

The paper trains on an internal multimodal set and on CapsFusion (Section 5); neither their
data nor their resolution statistics are available, so these recipes stand in for them:
variable-resolution images (Section 2: resolutions, video lengths and pure-text samples all
vary), log-uniform patch counts, a video-heavy tail, and a swept image-token fraction.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional

import numpy as np

BASE_SEED = 260703229
_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)


def _mix64(x: np.ndarray) -> np.ndarray:
    """splitmix64 finaliser on uint64 arrays (wrap-around arithmetic)."""
    x = x.astype(np.uint64, copy=True)
    with np.errstate(over="ignore"):
        x += np.uint64(0x9E3779B97F4A7C15)
        x ^= x >> np.uint64(30)
        x *= np.uint64(0xBF58476D1CE4E5B9)
        x ^= x >> np.uint64(27)
        x *= np.uint64(0x94D049BB133111EB)
        x ^= x >> np.uint64(31)
    return x


def _stream_key(seed: int, stream: int) -> np.uint64:
    k = _mix64(np.array([seed & 0xFFFFFFFFFFFFFFFF], dtype=np.uint64))
    with np.errstate(over="ignore"):
        k = _mix64(k ^ np.uint64((stream * 0xD1342543DE82EF95) & 0xFFFFFFFFFFFFFFFF))
    return k[0]


def rand_u64(seed: int, stream: int, n: int, start: int = 0) -> np.ndarray:
    """n hashed 64-bit words: word i depends only on (seed, stream, start + i)."""
    key = _stream_key(seed, stream)
    idx = np.arange(start, start + n, dtype=np.uint64)
    with np.errstate(over="ignore"):
        return _mix64(idx * np.uint64(0x2545F4914F6CDD1D) + key)


def rand_int(seed: int, stream: int, n: int, lo: int, hi: int) -> np.ndarray:
    """n integers uniform in [lo, hi] (modulo bias < 2^-40 for the ranges used here)."""
    span = np.uint64(hi - lo + 1)
    return (rand_u64(seed, stream, n) % span).astype(np.int64) + lo


def rand_unit(seed: int, stream: int, n: int) -> np.ndarray:
    """n doubles uniform in [0, 1)."""
    return (rand_u64(seed, stream, n) >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float32 -> bf16, returned as uint16 bit patterns (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(b).astype(np.float64)


def normal_bf16(seed: int, stream: int, shape) -> np.ndarray:
    """i.i.d. N(0,1) values rounded to bf16 (uint16 bits), Box-Muller on hashed uniforms.

    Element 2p and 2p+1 of the flattened tensor come from hashed word p.
    """
    n = int(np.prod(shape)) if len(shape) else 1
    out = np.empty(n + (n & 1), dtype=np.uint16)
    n_pairs = out.size // 2
    chunk = 1 << 22
    for p0 in range(0, n_pairs, chunk):
        m = min(chunk, n_pairs - p0)
        w = rand_u64(seed, stream, m, start=p0)
        u1 = ((w >> np.uint64(40)).astype(np.float32) + np.float32(1.0)) * np.float32(1.0 / 16777216.0)  # (0,1]
        u2 = ((w & np.uint64(0xFFFFFF)).astype(np.float32)) * np.float32(1.0 / 16777216.0)             # [0,1)
        r = np.sqrt(np.float32(-2.0) * np.log(u1))
        ang = np.float32(2.0 * np.pi) * u2
        out[2 * p0:2 * (p0 + m):2] = f32_to_bf16_bits(r * np.cos(ang))
        out[2 * p0 + 1:2 * (p0 + m):2] = f32_to_bf16_bits(r * np.sin(ang))
    return out[:n].reshape(shape)


def scaled_normal_bf16(seed: int, stream: int, shape, std: float, mean: float = 0.0) -> np.ndarray:
    """mean + std * N(0,1), rounded to bf16 bits (for synthetic weights, biases and norm parameters)."""
    z = bf16_bits_to_f32(normal_bf16(seed, stream, shape))
    return f32_to_bf16_bits((np.float32(mean) + np.float32(std) * z).astype(np.float32))


LAYER_PARAMS = ("ln1_gamma", "ln1_beta", "w_qkv", "b_qkv", "w_o", "b_o", "ln2_gamma", "ln2_beta", "w_fc1", "b_fc1",
                "w_fc2", "b_fc2")


def layer_params_bf16(seed: int, hidden: int, ffn: int) -> dict:
    """Random-init parameters of one encoder layer as bf16 bits: weights N(0, 1/fan_in) so that activations stay
    O(1), biases N(0, 0.1^2), norm scales 1 + N(0, 0.1^2).  Streams 100.. keep them apart from the activations."""
    shapes = {"ln1_gamma": (hidden,), "ln1_beta": (hidden,), "w_qkv": (3 * hidden, hidden), "b_qkv": (3 * hidden,),
              "w_o": (hidden, hidden), "b_o": (hidden,), "ln2_gamma": (hidden,), "ln2_beta": (hidden,),
              "w_fc1": (ffn, hidden), "b_fc1": (ffn,), "w_fc2": (hidden, ffn), "b_fc2": (hidden,)}
    out = {}
    for i, name in enumerate(LAYER_PARAMS):
        shp = shapes[name]
        if name.startswith("w_"):
            out[name] = scaled_normal_bf16(seed, 100 + i, shp, std=float(shp[1]) ** -0.5)
        elif name.endswith("gamma"):
            out[name] = scaled_normal_bf16(seed, 100 + i, shp, std=0.1, mean=1.0)
        else:
            out[name] = scaled_normal_bf16(seed, 100 + i, shp, std=0.1)
    return out


def rope2d_tables(patch_counts, head_dim: int, theta: float = 10000.0):
    """cos / sin tables fp32 [T, head_dim/2] of a 2-D rotary encoding for packed images: image i is laid out as a
    grid of width ceil(sqrt(n_i)) (row-major, last row ragged); the first head_dim/4 pairs turn with the row
    index, the other head_dim/4 with the column index, frequencies theta^(-k / (head_dim/4)).  Input recipe only:
    the tables are inputs of both the kernel and the oracle."""
    quarter = head_dim // 4
    inv = (theta ** (-np.arange(quarter, dtype=np.float64) / quarter))
    rows, cols = [], []
    for n in patch_counts:
        wdt = int(np.ceil(np.sqrt(n)))
        idx = np.arange(n)
        rows.append(idx // wdt)
        cols.append(idx % wdt)
    r = np.concatenate(rows).astype(np.float64)[:, None] * inv[None, :]
    c = np.concatenate(cols).astype(np.float64)[:, None] * inv[None, :]
    ang = np.concatenate([r, c], axis=1)
    return np.cos(ang).astype(np.float32), np.sin(ang).astype(np.float32)


# --------------------------------------------------------------------------------------
# Structure recipes
# --------------------------------------------------------------------------------------

@dataclass
class Workload:
    """One microbatch of encoder work (and, optionally, its merge into LLM sequences)."""
    name: str
    seed: int
    patch_counts: List[int]
    n_heads: int
    head_dim: int
    trained: bool
    # merge part (None when the config has no merge)
    merge_hidden: Optional[int] = None
    n_llm_tokens: Optional[int] = None
    positions: Optional[np.ndarray] = None  # int32 [T]
    meta: Dict = field(default_factory=dict)

    @property
    def total_tokens(self) -> int:
        return int(sum(self.patch_counts))

    @property
    def sum_n2(self) -> int:
        return int(sum(int(c) * int(c) for c in self.patch_counts))

    @property
    def cu_seqlens(self) -> np.ndarray:
        return np.concatenate([[0], np.cumsum(np.asarray(self.patch_counts, dtype=np.int64))]).astype(np.int32)

    @property
    def softmax_scale(self) -> float:
        return float(np.float32(1.0 / np.sqrt(np.float32(self.head_dim))))

    def flops(self, fwd: bool = True, bwd: bool = True) -> float:
        """4*H*D*sum n^2 forward, 10*H*D*sum n^2 backward (five contractions, no causal halving)."""
        per = (4.0 if fwd else 0.0) + (10.0 if bwd else 0.0)
        return per * self.n_heads * self.head_dim * float(self.sum_n2)

    def qkv(self):
        """q, k, v as uint16 bf16 bits, [T, H, D], N(0,1)."""
        shape = (self.total_tokens, self.n_heads, self.head_dim)
        return tuple(normal_bf16(self.seed, 10 + i, shape) for i in range(3))

    def dout(self):
        return normal_bf16(self.seed, 13, (self.total_tokens, self.n_heads, self.head_dim))

    def merge_source(self):
        """[T, merge_hidden] bf16 bits standing for the projector output."""
        return normal_bf16(self.seed, 20, (self.total_tokens, self.merge_hidden))

    def llm_embeds(self):
        """[n_llm_tokens, merge_hidden] bf16 bits standing for the text embeddings."""
        return normal_bf16(self.seed, 21, (self.n_llm_tokens, self.merge_hidden))


def _runs_with_gaps(seed: int, stream: int, run_lens: List[int], n_total: int) -> np.ndarray:
    """Place contiguous runs (in order) inside [0, n_total), text gaps = a seeded random
    composition of the remaining tokens into len(run_lens)+1 parts."""
    n_img = int(sum(run_lens))
    n_text = n_total - n_img
    assert n_text >= 0
    k = len(run_lens) + 1
    if k == 1:
        return np.zeros((0,), dtype=np.int32)
    # composition: sort k-1 seeded cut points in [0, n_text]
    cuts = np.sort(rand_int(seed, stream, k - 1, 0, n_text)) if n_text > 0 else np.zeros(k - 1, dtype=np.int64)
    gaps = np.diff(np.concatenate([[0], cuts, [n_text]]))
    pos = []
    cursor = 0
    for g, r in zip(gaps[:-1], run_lens):
        cursor += int(g)
        pos.append(np.arange(cursor, cursor + r, dtype=np.int64))
        cursor += r
    return np.concatenate(pos).astype(np.int32) if pos else np.zeros((0,), dtype=np.int32)


def tiny(seed: int = BASE_SEED + 1, shuffled_positions: bool = False) -> Workload:
    """Four images of 16, 49, 64 and 100 patches (229 tokens), 4 heads of 64, trained; merge of the
    229 tokens (hidden 256) into one 512-token sequence."""
    counts = [16, 49, 64, 100]
    if shuffled_positions:
        keys = rand_u64(seed, 31, 512)
        pos = np.argsort(keys, kind="stable")[:229].astype(np.int32)  # unique, unsorted
    else:
        pos = _runs_with_gaps(seed, 30, counts, 512)
    return Workload("tiny", seed, counts, 4, 64, True, merge_hidden=256, n_llm_tokens=512, positions=pos)


def vit_l(seed: int = BASE_SEED + 2, n_images: int = 32, n_llm_tokens: int = 131072) -> Workload:
    """32 images, height and width independently uniform in 16..64 patches (224-896 px at patch
    14), 16 heads of 64, trained.  For the whole-path benchmark the encoder output (hidden 1024 =
    heads x head_dim, one LLM token per patch) is merged into 16 LLM sequences of 8192 tokens at
    hidden 1024: every image one contiguous placeholder run, seeded text gaps in between."""
    h = rand_int(seed, 1, n_images, 16, 64)
    w = rand_int(seed, 2, n_images, 16, 64)
    counts = [int(a * b) for a, b in zip(h, w)]
    pos = _runs_with_gaps(seed, 30, counts, n_llm_tokens)
    return Workload("vit_l", seed, counts, 16, 64, True, merge_hidden=1024, n_llm_tokens=n_llm_tokens,
                    positions=pos)


def qwen2vl(seed: int = BASE_SEED + 3, trained: bool = True, total: int = 65536) -> Workload:
    """Patch counts log-uniform in [64, 16384] drawn until the packed length reaches 65536; the last
    draw is clipped so the total is exact.  16 heads of 80."""
    u = rand_unit(seed, 1, 4096)
    counts: List[int] = []
    acc = 0
    for x in u:
        n = int(round(float(np.exp(np.log(64.0) + x * (np.log(16384.0) - np.log(64.0))))))
        n = min(n, total - acc)
        counts.append(n)
        acc += n
        if acc >= total:
            break
    return Workload("qwen2vl", seed, counts, 16, 80, trained)


def video_tail(seed: int = BASE_SEED + 4, n_small: int = 200, n_clips: int = 4) -> Workload:
    """200 small images (64-256 patches) and 4 clips of 16 frames x 1024 patches, each clip one
    16384-token segment, clips at seeded slots among the images.  16 heads of 80, trained."""
    small = [int(x) for x in rand_int(seed, 1, n_small, 64, 256)]
    slots = sorted(int(x) for x in rand_int(seed, 2, n_clips, 0, n_small))
    counts: List[int] = []
    si = 0
    for i in range(n_small + 1):
        while si < n_clips and slots[si] == i:
            counts.append(16 * 1024)
            si += 1
        if i < n_small:
            counts.append(small[i])
    return Workload("video_tail", seed, counts, 16, 80, True)


def modality_mix(fraction: float, seed: int = BASE_SEED + 5, trained: bool = True, n_seq: int = 8,
                 seq_len: int = 8192, llm_hidden: int = 4096) -> Workload:
    """8 LLM sequences of 8192 tokens at hidden 4096; each gets round(fraction*8192) image tokens made
    of images of 16..64 x 16..64 patches (clipped to the remaining budget; a remainder under 256 is
    absorbed by the current image); images sit in contiguous placeholder runs separated by seeded
    text gaps.  The encoder microbatch packs all sequences' images: 16 heads of 64."""
    budget = int(round(fraction * seq_len))
    counts: List[int] = []
    positions = []
    for s in range(n_seq):
        h = rand_int(seed, 100 + 2 * s, 64, 16, 64)
        w = rand_int(seed, 101 + 2 * s, 64, 16, 64)
        remaining = budget
        runs: List[int] = []
        i = 0
        while remaining > 0:
            n = min(int(h[i] * w[i]), remaining)
            if remaining - n < 256:
                n = remaining
            runs.append(n)
            remaining -= n
            i += 1
        counts += runs
        positions.append(_runs_with_gaps(seed, 200 + s, runs, seq_len).astype(np.int64) + s * seq_len)
    pos = np.concatenate(positions).astype(np.int32) if positions else np.zeros((0,), dtype=np.int32)
    return Workload(f"modality_mix_{int(round(fraction * 100))}", seed, counts, 16, 64, trained,
                    merge_hidden=llm_hidden, n_llm_tokens=n_seq * seq_len, positions=pos,
                    meta={"fraction": fraction})


MIX_FRACTIONS = (0.0, 0.10, 0.25, 0.50, 0.75)
