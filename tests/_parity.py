"""Parity tiers for the benchmark-size configurations.

FULL tier: every element of O, LSE, dQ, dK, dV against the fp64 oracle.  The oracle is called once per (segment,
head) on contiguous single-head slices -- the packed computation is per image and per head by definition (the
oracle's own pins check packed == per image), and contiguous rows are what lets the plain row loops run at
their speed on 16 384-token segments.

SAMPLED tier (for configurations whose full pass takes many minutes of CPU):
  * every segment of at most `long_threshold` tokens: the FULL tier;
  * every longer segment: `rows_per_head` seeded query rows (plus the first and last row) of EVERY head for
    O, LSE and dQ (each needs only its own row), and `dkv_heads` seeded heads compared in full for dK and dV
    (a key row's gradient sums over all query rows of the segment).
Both tiers print exactly what was compared.
"""
import numpy as np
import torch

import oracle
from paper_2607_03229_b200 import binding as B
from paper_2607_03229_b200 import workloads as W
from _util import GRAD_REL_L2, LSE_MAX_ABS, O_MAX_ABS, O_REL_L2, status_buf, to_dev, to_f64


class Acc:
    """Running max-abs and relative-L2 error of one tensor over several pieces."""

    def __init__(self, name):
        self.name, self.max_abs, self.num, self.den, self.count = name, 0.0, 0.0, 0.0, 0

    def add(self, got, ref):
        d = got - ref
        assert not np.isnan(got).any(), self.name
        if d.size:
            self.max_abs = max(self.max_abs, float(np.abs(d).max()))
        self.num += float((d * d).sum())
        self.den += float((ref * ref).sum())
        self.count += d.size

    @property
    def rel_l2(self):
        return (self.num / self.den) ** 0.5 if self.den > 0 else (0.0 if self.num == 0 else float("inf"))

    def __repr__(self):
        return f"{self.name}: n={self.count} max_abs={self.max_abs:.3e} rel_l2={self.rel_l2:.3e}"


def run_gpu(w, mode=B.TRAINED):
    """Forward (+ backward when trained) of a workload through the C ABI.  Returns host inputs and device outputs."""
    q, k, v = w.qkv()
    do = w.dout() if mode == B.TRAINED else None
    T, H, D = q.shape
    plan = B.seg_plan(w.patch_counts, mode).to_device()
    qd, kd, vd = to_dev(q), to_dev(k), to_dev(v)
    o = torch.empty_like(qd)
    lse = torch.empty((H, T), dtype=torch.float32, device="cuda") if mode == B.TRAINED else None
    st = status_buf()
    B.varlen_attn_fwd(qd, kd, vd, o, lse, plan, w.softmax_scale, st)
    dq = dk = dv = None
    if mode == B.TRAINED:
        dod = to_dev(do)
        dq, dk, dv = (torch.empty_like(qd) for _ in range(3))
        ws = torch.empty(max(B.attn_workspace_bytes(T, H, D, mode), 1), dtype=torch.uint8, device="cuda")
        B.varlen_attn_bwd(dod, qd, kd, vd, o, lse, dq, dk, dv, plan, w.softmax_scale, ws, st)
    torch.cuda.synchronize()
    assert st.cpu().tolist()[0] == 0, f"device status {st.cpu().tolist()}"
    return dict(q=q, k=k, v=v, do=do, o=o, lse=lse, dq=dq, dk=dk, dv=dv)


def _new_accs():
    return {n: Acc(n) for n in ("o", "lse", "dq", "dk", "dv")}


def full_segments(w, res, segs, accs):
    """FULL tier on the listed segments: one oracle call per (segment, head) on contiguous slices."""
    cu, H = w.cu_seqlens, w.n_heads
    for s in segs:
        a, b = int(cu[s]), int(cu[s + 1])
        if b <= a:
            continue
        one = np.array([0, b - a], dtype=np.int32)
        got = {n: to_f64(res[n][a:b]) for n in ("o", "dq", "dk", "dv")}
        got_lse = to_f64(res["lse"][:, a:b])
        for h in range(H):
            sl = [np.ascontiguousarray(res[n][a:b, h:h + 1]) for n in ("q", "k", "v", "do")]
            O_ref, L_ref = oracle.attn_fwd(sl[0], sl[1], sl[2], one, w.softmax_scale)
            g_ref = oracle.attn_bwd(sl[3], sl[0], sl[1], sl[2], one, w.softmax_scale)
            accs["o"].add(got["o"][:, h], O_ref[:, 0])
            accs["lse"].add(got_lse[h], L_ref[0])
            for n, r in zip(("dq", "dk", "dv"), g_ref):
                accs[n].add(got[n][:, h], r[:, 0])


def sampled_long_segments(w, res, segs, accs, rows_per_head, dkv_heads, seed):
    """SAMPLED tier on the listed (long) segments."""
    cu, H, D = w.cu_seqlens, w.n_heads, w.head_dim
    for s in segs:
        a, b = int(cu[s]), int(cu[s + 1])
        n = b - a
        one = np.array([0, n], dtype=np.int32)
        wide = [W.bf16_bits_to_f64(res[x][a:b]) for x in ("q", "k", "v", "do")]      # widened once per segment
        rows_l, heads_l = [], []
        for h in range(H):
            r = (W.rand_u64(seed + s, 100 + h, rows_per_head) % np.uint64(n)).astype(np.int64)
            r = np.unique(np.concatenate([r, [0, n - 1]]))
            rows_l.append(r)
            heads_l.append(np.full(r.size, h, dtype=np.int32))
        rows, heads = np.concatenate(rows_l), np.concatenate(heads_l)
        O_ref, L_ref = oracle.attn_fwd_rows(wide[0], wide[1], wide[2], one, w.softmax_scale, rows, heads)
        dQ_ref = oracle.attn_bwd_dq_rows(wide[3], wide[0], wide[1], wide[2], one, w.softmax_scale, rows, heads)
        ridx = torch.from_numpy(rows + a).cuda()
        hidx = torch.from_numpy(heads.astype(np.int64)).cuda()
        accs["o"].add(to_f64(res["o"][ridx, hidx]), O_ref)
        accs["lse"].add(to_f64(res["lse"][hidx, ridx]), L_ref)
        accs["dq"].add(to_f64(res["dq"][ridx, hidx]), dQ_ref)
        pick = np.argsort(W.rand_u64(seed + s, 99, H), kind="stable")[:dkv_heads]
        all_rows = np.arange(n, dtype=np.int64)
        for h in (int(x) for x in pick):
            sl = [np.ascontiguousarray(x[:, h:h + 1]) for x in wide]
            rk, rv = oracle.attn_bwd_dkv_rows(sl[3], sl[0], sl[1], sl[2], one, w.softmax_scale, 0, 0, all_rows)
            accs["dk"].add(to_f64(res["dk"][a:b, h]), rk)
            accs["dv"].add(to_f64(res["dv"][a:b, h]), rv)
        print(f"  segment {s} ({n} tokens): {rows.size} (row, head) pairs for O/LSE/dQ; heads {sorted(int(x) for x in pick)} "
              f"in full for dK/dV")


def assert_bars(name, accs):
    print(name, "|", " | ".join(repr(a) for a in accs.values()))
    assert accs["o"].max_abs <= O_MAX_ABS and accs["o"].rel_l2 <= O_REL_L2, accs["o"]
    assert accs["lse"].max_abs <= LSE_MAX_ABS, accs["lse"]
    for n in ("dq", "dk", "dv"):
        assert accs[n].rel_l2 <= GRAD_REL_L2, accs[n]


def check_full(w, segs=None):
    res = run_gpu(w)
    accs = _new_accs()
    segs = range(len(w.patch_counts)) if segs is None else segs
    full_segments(w, res, segs, accs)
    assert_bars(f"{w.name} FULL tier ({len(list(segs))} segments, {w.n_heads} heads)", accs)
    return accs


def check_sampled(w, long_threshold=4096, rows_per_head=256, dkv_heads=2, seed=11):
    res = run_gpu(w)
    lens = np.diff(w.cu_seqlens)
    short = [s for s in range(lens.size) if 0 < lens[s] <= long_threshold]
    long_ = [s for s in range(lens.size) if lens[s] > long_threshold]
    accs = _new_accs()
    print(f"{w.name} SAMPLED tier: {len(short)} segments of <= {long_threshold} tokens in full, {len(long_)} longer ones sampled")
    full_segments(w, res, short, accs)
    sampled_long_segments(w, res, long_, accs, rows_per_head, dkv_heads, seed)
    for n in ("o", "dq", "dk", "dv"):
        assert not torch.isnan(res[n].float()).any(), n
    assert_bars(f"{w.name} SAMPLED tier", accs)
    return accs
