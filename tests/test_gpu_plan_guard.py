"""The work items reach the kernels through device memory the host cannot inspect at launch, so the kernels clamp
them to the tensors.  These tests hand the attention calls plans that do not fit the tensors and check that nothing
outside the tensors is written, that MPIPE_ERR_INDEX is reported, and that everything that does fit is still right.

Every out-of-range row used here lies inside canary padding allocated around the outputs (and the inputs are read
through TMA, which fills out-of-range rows with zeros), so not even a missing guard could touch unowned memory."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_03229_b200 import binding as B
from paper_2607_03229_b200 import workloads as W
from _util import GRAD_REL_L2, O_MAX_ABS, O_REL_L2, LSE_MAX_ABS, max_abs, rel_l2, status_buf, to_dev, to_f64

pytestmark = pytest.mark.gpu
PAD = 128


def _run(plan, q, k, v, do, scale):
    T, H, D = q.shape
    qd, kd, vd, dod = to_dev(q), to_dev(k), to_dev(v), to_dev(do)

    def padded(fill):
        buf = torch.full((T + 2 * PAD, H, D), fill, dtype=torch.bfloat16, device="cuda")
        return buf, buf[PAD:PAD + T]

    obuf, o = padded(777.0)
    lse_buf = torch.full((H * T + 2 * PAD,), -555.0, dtype=torch.float32, device="cuda")
    lse = lse_buf[PAD:PAD + H * T].view(H, T)
    # lse must be contiguous and 4-byte aligned only; PAD floats in front keep a stray negative index inside the buffer
    st_f, st_b = status_buf(), status_buf()
    B.varlen_attn_fwd(qd, kd, vd, o, lse, plan, scale, st_f)
    gbufs = [padded(333.0) for _ in range(3)]
    ws = torch.empty(B.attn_workspace_bytes(T, H, D, B.TRAINED) + 4096, dtype=torch.uint8, device="cuda")
    B.varlen_attn_bwd(dod, qd, kd, vd, o, lse, *(g[1] for g in gbufs), plan, scale, ws, st_b)
    torch.cuda.synchronize()
    assert torch.all(obuf[:PAD] == 777.0) and torch.all(obuf[PAD + T:] == 777.0), "forward wrote outside O"
    assert torch.all(lse_buf[:PAD] == -555.0) and torch.all(lse_buf[PAD + H * T:] == -555.0), "forward wrote outside LSE"
    for buf, _ in gbufs:
        assert torch.all(buf[:PAD] == 333.0) and torch.all(buf[PAD + T:] == 333.0), "backward wrote outside a gradient"
    return o, lse, [g[1] for g in gbufs], st_f.cpu().tolist(), st_b.cpu().tolist()


@pytest.mark.parametrize("D", [64, 80])
def test_plan_made_for_more_tokens_is_clamped_and_flagged(D):
    """The plan's last segment is 40 tokens longer than the tensors: its items overrun them by 40 rows.  Clamped to
    the tensors the items describe segments of 300 and 200 tokens, so the results must be those."""
    H, T, scale = 2, 500, float(np.float32(1.0 / np.sqrt(D)))
    q, k, v, do = (W.normal_bf16(91, s, (T, H, D)) for s in (1, 2, 3, 4))
    plan = B.seg_plan([300, 240], B.TRAINED)
    assert plan.total_tokens == 540
    plan.total_tokens = T          # what the caller claims; the items still name rows up to 540
    plan.to_device()
    o, lse, (dq, dk, dv), st_f, st_b = _run(plan, q, k, v, do, scale)
    assert st_f[0] == B.ERR_INDEX and st_b[0] == B.ERR_INDEX
    cu = np.array([0, 300, 500], dtype=np.int32)
    O_ref, L_ref = oracle.attn_fwd(q, k, v, cu, scale)
    assert max_abs(to_f64(o), O_ref) <= O_MAX_ABS and rel_l2(to_f64(o), O_ref) <= O_REL_L2
    assert max_abs(to_f64(lse), L_ref) <= LSE_MAX_ABS
    for g, r in zip((dq, dk, dv), oracle.attn_bwd(do, q, k, v, cu, scale)):
        assert rel_l2(to_f64(g), r) <= GRAD_REL_L2


def test_items_outside_the_tensors_store_nothing():
    """Items that lie wholly behind the tensors' end or before their start (inside the padding) are replaced by a
    stand-in unit that stores nothing; the other items are unaffected."""
    H, D, scale = 2, 64, 0.125
    counts = [200, 150, 90]
    T = sum(counts)
    q, k, v, do = (W.normal_bf16(92, s, (T, H, D)) for s in (1, 2, 3, 4))
    plan = B.seg_plan(counts, B.TRAINED)
    # the 90-token segment's item: forward, moved 8 rows behind the tensors' end; backward, moved to end 10 rows
    # before their start
    for items, victim_seg, start in ((plan.fwd_items, 2, T + 8), (plan.bwd_items, 2, -100)):
        idx = [i for i in range(items.size) if items[i]["seg"] == victim_seg][-1]
        items[idx]["row_start"] = start
        items[idx]["kv_start"] = start
    plan.to_device()
    o, lse, (dq, dk, dv), st_f, st_b = _run(plan, q, k, v, do, scale)
    assert st_f[0] == B.ERR_INDEX and st_b[0] == B.ERR_INDEX
    a = 350                       # rows of the 90-token segment
    assert torch.all(o[a:] == 777.0) and torch.all(lse[:, a:] == -555.0)          # never stored
    assert torch.all(dk[a:] == 333.0) and torch.all(dv[a:] == 333.0)
    cu = np.array([0, 200, 350, 440], dtype=np.int32)
    O_ref, _ = oracle.attn_fwd(q, k, v, cu, scale)
    assert rel_l2(to_f64(o[:a]), O_ref[:a]) <= O_REL_L2
    ref = oracle.attn_bwd(do, q, k, v, cu, scale)
    for g, r in zip((dq, dk, dv), ref):
        assert rel_l2(to_f64(g[:a]), r[:a]) <= GRAD_REL_L2
