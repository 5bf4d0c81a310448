"""The work items reach the kernels through device memory the host cannot inspect at launch, so each kernel checks
the whole list before doing anything else and rejects a plan that does not fit the tensors.  These tests hand the
attention calls such plans and check that nothing at all is written, inside or outside the tensors, and that
MPIPE_ERR_INDEX is reported with the index of an offending item.

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


def _untouched(o, lse, grads):
    """O, LSE, dK, dV keep their fill values; dQ is all zeros (the accumulator is cleared and converted by the two
    helper kernels, which do not depend on the plan, and no item has added to it)."""
    dq, dk, dv = grads
    return bool(torch.all(o == 777.0) and torch.all(lse == -555.0) and torch.all(dk == 333.0) and torch.all(dv == 333.0)
                and torch.all(dq == 0.0))


@pytest.mark.parametrize("D", [64, 80])
def test_plan_made_for_more_tokens_is_rejected(D):
    """The plan's last segment is 40 tokens longer than the tensors: its last items overrun them by 40 rows."""
    H, T, scale = 2, 500, float(np.float32(1.0 / np.sqrt(D)))
    q, k, v, do = (W.normal_bf16(91, s, (T, H, D)) for s in (1, 2, 3, 4))
    plan = B.seg_plan([300, 240], B.TRAINED)
    assert plan.total_tokens == 540
    plan.total_tokens = T          # what the caller claims; the items still name rows up to 540
    plan.to_device()
    o, lse, grads, st_f, st_b = _run(plan, q, k, v, do, scale)
    assert st_f[0] == B.ERR_INDEX and st_b[0] == B.ERR_INDEX
    assert plan.fwd_items[st_f[1]]["seg"] == 1 and plan.bwd_items[st_b[1]]["seg"] == 1     # an item of the long segment
    assert _untouched(o, lse, grads)


def test_items_outside_the_tensors_reject_the_plan():
    """One item moved wholly behind the tensors' end (forward list) or before their start (backward list), inside
    the padding: the plan is rejected, nothing is written, the status names the item."""
    H, D, scale = 2, 64, 0.125
    counts = [200, 150, 90]
    T = sum(counts)
    q, k, v, do = (W.normal_bf16(92, s, (T, H, D)) for s in (1, 2, 3, 4))
    plan = B.seg_plan(counts, B.TRAINED)
    moved = []
    for items, start in ((plan.fwd_items, T + 8), (plan.bwd_items, -100)):
        idx = [i for i in range(items.size) if items[i]["seg"] == 2][-1]
        items[idx]["row_start"] = start
        items[idx]["kv_start"] = start
        moved.append(idx)
    plan.to_device()
    o, lse, grads, st_f, st_b = _run(plan, q, k, v, do, scale)
    assert st_f[:2] == [B.ERR_INDEX, moved[0]] and st_b[:2] == [B.ERR_INDEX, moved[1]]
    assert _untouched(o, lse, grads)


def test_a_good_plan_after_a_rejected_one_runs_normally():
    """Rejection leaves no state behind: the same tensors with the right plan give the right answer."""
    H, D, scale = 2, 64, 0.125
    counts = [200, 150, 90]
    T = sum(counts)
    q, k, v, do = (W.normal_bf16(93, s, (T, H, D)) for s in (1, 2, 3, 4))
    bad = B.seg_plan(counts, B.TRAINED)
    bad.fwd_items[0]["kv_len"] = T + 1
    bad.bwd_items[0]["row_len"] = 0
    bad.to_device()
    _, _, _, st_f, st_b = _run(bad, q, k, v, do, scale)
    assert st_f[0] == B.ERR_INDEX and st_b[0] == B.ERR_INDEX
    o, lse, (dq, dk, dv), st_f, st_b = _run(B.seg_plan(counts, B.TRAINED).to_device(), q, k, v, do, scale)
    assert st_f[0] == 0 and st_b[0] == 0
    cu = np.array([0, 200, 350, 440], dtype=np.int32)
    O_ref, L_ref = oracle.attn_fwd(q, k, v, cu, scale)
    assert max_abs(to_f64(o), O_ref) <= O_MAX_ABS and rel_l2(to_f64(o), O_ref) <= O_REL_L2
    assert max_abs(to_f64(lse), L_ref) <= LSE_MAX_ABS
    for g, r in zip((dq, dk, dv), oracle.attn_bwd(do, q, k, v, cu, scale)):
        assert rel_l2(to_f64(g), r) <= GRAD_REL_L2
