"""The attention step is stream-ordered, allocation-free and free of host synchronisation, so a caller can capture
forward + backward in a CUDA graph and replay it (the launch-bound regime of short segments).  The replay must
give what the plain launches give: O, LSE, dK and dV bit for bit (their summation orders are fixed),
dQ within the parity bar (its reduce-adds land in hardware order), all of them within the bars against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_03229_b200 import binding as B
from paper_2607_03229_b200 import workloads as W
from _util import GRAD_REL_L2, LSE_MAX_ABS, O_MAX_ABS, O_REL_L2, rel_l2, max_abs, status_buf, to_dev, to_f64

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("make", [W.tiny, lambda: W.Workload("ragged_d80", 3, [5, 130, 0, 257, 64], 4, 80, True)],
                         ids=["tiny_d64", "ragged_d80"])
def test_step_replays_from_a_cuda_graph(make):
    w = make()
    q, k, v, do = w.qkv() + (w.dout(),)
    T, H, D = q.shape
    plan = B.seg_plan(w.patch_counts, B.TRAINED).to_device()
    qd, kd, vd, dod = (to_dev(x) for x in (q, k, v, do))
    ws = torch.empty(B.attn_workspace_bytes(T, H, D, B.TRAINED), dtype=torch.uint8, device="cuda")
    st = status_buf()

    def new_out():
        return dict(o=torch.zeros_like(qd), lse=torch.zeros((H, T), dtype=torch.float32, device="cuda"),
                    dq=torch.zeros_like(qd), dk=torch.zeros_like(qd), dv=torch.zeros_like(qd))

    def step(t):
        B.varlen_attn_fwd(qd, kd, vd, t["o"], t["lse"], plan, w.softmax_scale, st)
        B.varlen_attn_bwd(dod, qd, kd, vd, t["o"], t["lse"], t["dq"], t["dk"], t["dv"], plan, w.softmax_scale, ws, st)

    eager = new_out()
    step(eager)                      # also the warm-up: per-kernel attributes are set outside the capture
    torch.cuda.synchronize()

    captured = new_out()
    g = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            step(captured)
    torch.cuda.synchronize()
    for t in captured.values():      # capture launches nothing
        assert not t.float().abs().sum().item()
    for _ in range(3):               # replays are repeatable
        g.replay()
    torch.cuda.synchronize()
    assert st.cpu().tolist()[0] == 0

    for n in ("o", "lse", "dk", "dv"):
        assert torch.equal(eager[n], captured[n]), n
    assert rel_l2(to_f64(captured["dq"]), to_f64(eager["dq"])) <= 1e-3

    cu = w.cu_seqlens
    O_ref, L_ref = oracle.attn_fwd(q, k, v, cu, w.softmax_scale)
    g_ref = oracle.attn_bwd(do, q, k, v, cu, w.softmax_scale)
    assert max_abs(to_f64(captured["o"]), O_ref) <= O_MAX_ABS and rel_l2(to_f64(captured["o"]), O_ref) <= O_REL_L2
    assert max_abs(to_f64(captured["lse"]), L_ref) <= LSE_MAX_ABS
    for n, r in zip(("dq", "dk", "dv"), g_ref):
        assert rel_l2(to_f64(captured[n]), r) <= GRAD_REL_L2, n
