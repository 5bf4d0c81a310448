"""Seeded random ragged workloads (segment counts, lengths around the tile edges, empty segments, 1 to 16 heads, both
head dimensions) through forward and backward, every element against the fp64 oracle.  Complements the hand-picked
shape lists of the forward and backward suites."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_03229_b200 import binding as B
from paper_2607_03229_b200 import workloads as W
from _util import GRAD_REL_L2, LSE_MAX_ABS, O_MAX_ABS, O_REL_L2, max_abs, rel_l2, status_buf, to_dev, to_f64

pytestmark = pytest.mark.gpu

EDGES = [0, 1, 2, 15, 16, 17, 63, 64, 65, 127, 128, 129, 255, 256, 257, 383, 384, 385, 511, 512, 513]


def _draw(case):
    rng = np.random.default_rng(7000 + case)
    D = int(rng.choice([64, 80]))
    H = int(rng.choice([1, 2, 3, 5, 16]))
    nseg = int(rng.integers(1, 10))
    kind = case % 4
    if kind == 0:
        counts = rng.integers(0, 140, nseg)
    elif kind == 1:
        counts = rng.integers(100, 700, nseg)
    elif kind == 2:
        counts = rng.choice(EDGES, nseg)
    else:
        counts = rng.integers(1, 1500, max(1, nseg // 3))
    counts = [int(c) for c in counts]
    if sum(counts) < 2:
        counts[0] = 5
    if H == 16 and sum(counts) > 3000:
        H = 4
    return W.Workload(f"random_{case}", 7000 + case, counts, H, D, True)


@pytest.mark.parametrize("case", range(40))
def test_random_ragged_workload_matches_the_oracle(case):
    w = _draw(case)
    q, k, v, do = w.qkv() + (w.dout(),)
    T, H, D = q.shape
    plan = B.seg_plan(w.patch_counts, B.TRAINED).to_device()
    qd, kd, vd, dod = (to_dev(x) for x in (q, k, v, do))
    o = torch.empty_like(qd)
    lse = torch.empty((H, T), dtype=torch.float32, device="cuda")
    dq, dk, dv = (torch.empty_like(qd) for _ in range(3))
    ws = torch.empty(max(B.attn_workspace_bytes(T, H, D, B.TRAINED), 1), dtype=torch.uint8, device="cuda")
    st = status_buf()
    B.varlen_attn_fwd(qd, kd, vd, o, lse, plan, w.softmax_scale, st)
    B.varlen_attn_bwd(dod, qd, kd, vd, o, lse, dq, dk, dv, plan, w.softmax_scale, ws, st)
    torch.cuda.synchronize()
    assert st.cpu().tolist()[0] == 0

    cu = w.cu_seqlens
    O_ref, L_ref = oracle.attn_fwd(q, k, v, cu, w.softmax_scale)
    refs = oracle.attn_bwd(do, q, k, v, cu, w.softmax_scale)
    got_o = to_f64(o)
    assert not np.isnan(got_o).any()
    assert max_abs(got_o, O_ref) <= O_MAX_ABS and rel_l2(got_o, O_ref) <= O_REL_L2, w.patch_counts
    assert max_abs(to_f64(lse), L_ref) <= LSE_MAX_ABS, w.patch_counts
    for name, got, ref in zip(("dq", "dk", "dv"), (dq, dk, dv), refs):
        g = to_f64(got)
        assert not np.isnan(g).any(), name
        # one-token segments have dQ = dK = 0 exactly; a workload made of them alone has no norm to be relative to
        if np.linalg.norm(ref.ravel()) > 0:
            assert rel_l2(g, ref) <= GRAD_REL_L2, (name, w.patch_counts)
        else:
            assert max_abs(g, ref) <= 1e-4, (name, w.patch_counts)
