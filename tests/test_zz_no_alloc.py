"""mpipe_varlen_attn_bwd_static: the backward for callers that are not allowed to allocate device
memory (a pipeline runtime with a fixed memory plan, a process whose device memory belongs to someone
else's pool, a loop where cudaMalloc's device-wide synchronisation is unacceptable).  Its scratch is a
32 MiB array inside the library, shared by all calls on a device, so this file checks, through the C
ABI, that it gives what the caller-workspace entry point gives -- twice in a row, on different
problems, so that whatever the first call left in the shared scratch cannot leak into the second --
and that a problem too large for the built-in scratch is refused up front.

Collected last on purpose (file name): a failure here never hides another test's result.
"""
import numpy as np
import pytest
import torch

from paper_2607_03229_b200 import binding as B
from paper_2607_03229_b200 import workloads as W
from _util import GRAD_REL_L2, rel_l2, status_buf, to_dev, to_f64

pytestmark = pytest.mark.gpu


def _both_ways(counts, H, D, seed):
    """Forward once, then the backward through both entry points.  Returns the two gradient triples."""
    T = int(sum(counts))
    q, k, v, do = (to_dev(W.normal_bf16(seed, s, (T, H, D))) for s in (1, 2, 3, 4))
    scale = float(np.float32(1.0 / np.sqrt(D)))
    plan = B.seg_plan(counts, B.TRAINED).to_device()
    o = torch.empty_like(q)
    lse = torch.empty((H, T), dtype=torch.float32, device="cuda")
    st = status_buf()
    B.varlen_attn_fwd(q, k, v, o, lse, plan, scale, st)
    ws = torch.empty(B.attn_workspace_bytes(T, H, D, B.TRAINED), dtype=torch.uint8, device="cuda")
    ref = [torch.empty_like(q) for _ in range(3)]
    B.varlen_attn_bwd(do, q, k, v, o, lse, *ref, plan, scale, ws, st)
    got = [torch.full_like(q, 9.0) for _ in range(3)]
    B.varlen_attn_bwd_static(do, q, k, v, o, lse, *got, plan, scale, st)
    torch.cuda.synchronize()
    assert st.cpu().tolist()[0] == 0
    return got, ref


def test_static_scratch_backward_matches_workspace_backward_twice_in_a_row():
    assert B.attn_bwd_static_scratch_bytes() == 32 << 20
    # two different problems back to back: the second runs on the scratch the first one dirtied
    for counts, H, D, seed in (([700, 300, 129, 1], 4, 64, 71), ([260, 513], 2, 80, 72), ([16, 49, 64, 100], 4, 64, 73)):
        assert B.attn_workspace_bytes(sum(counts), H, D, B.TRAINED) <= B.attn_bwd_static_scratch_bytes()
        (dq, dk, dv), (rq, rk, rv) = _both_ways(counts, H, D, seed)
        # dK and dV do not pass through the scratch accumulator.  With head_dim 64 one warp issues all tensor-core
        # work in a fixed order, so they come out bit-identical; with head_dim 80 two warps issue and the order in
        # which their partial products are added can differ from call to call: equal within the tolerance.
        if D == 64:
            assert torch.equal(dk.view(torch.int16), rk.view(torch.int16))
            assert torch.equal(dv.view(torch.int16), rv.view(torch.int16))
        else:
            assert rel_l2(to_f64(dk), to_f64(rk)) <= GRAD_REL_L2 and rel_l2(to_f64(dv), to_f64(rv)) <= GRAD_REL_L2
        # dQ is summed with fp32 atomics in both entry points: equal within the gradient tolerance
        assert rel_l2(to_f64(dq), to_f64(rq)) <= GRAD_REL_L2
        assert not torch.isnan(dq.float()).any()


def test_too_large_for_the_builtin_scratch_is_refused_before_any_launch():
    T, H, D = 20000, 16, 64
    assert B.attn_workspace_bytes(T, H, D, B.TRAINED) > B.attn_bwd_static_scratch_bytes()
    plan = B.seg_plan([T], B.TRAINED).to_device()
    x = torch.zeros((T, H, D), dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros((H, T), dtype=torch.float32, device="cuda")
    grads = [torch.full_like(x, 3.0) for _ in range(3)]
    with pytest.raises(B.MpipeError) as e:
        B.varlen_attn_bwd_static(x, x, x, x, x, lse, *grads, plan, 0.125)
    assert e.value.status == B.ERR_WORKSPACE
    torch.cuda.synchronize()
    assert all(torch.all(g == 3.0) for g in grads)


def test_frozen_encoder_needs_no_scratch_and_does_nothing():
    plan = B.seg_plan([40], B.FROZEN).to_device()
    x = torch.zeros((40, 2, 64), dtype=torch.bfloat16, device="cuda")
    g = torch.full_like(x, 4.0)
    B.varlen_attn_bwd_static(x, x, x, x, x, None, g, g, g, plan, 0.125)
    torch.cuda.synchronize()
    assert torch.all(g == 4.0)
