"""mpipe_varlen_attn_bwd_static: the backward for callers that are not allowed to allocate device
memory (a pipeline runtime with a fixed memory plan, a process whose device memory belongs to someone
else's pool, a loop where cudaMalloc's device-wide synchronisation is unacceptable).  Its scratch is a
32 MiB array inside the library, shared by all calls on a device, so this file checks, through the C
ABI, that it gives what the caller-workspace entry point gives -- twice in a row, on different
problems, so that whatever the first call left in the shared scratch cannot leak into the second --
and that a problem too large for the built-in scratch is refused up front.

Collected last on purpose (file name): a failure here never hides another test's result.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
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
        # dK and dV do not pass through the scratch accumulator, and one warp issues all tensor-core work in a fixed
        # order at both head dimensions: they come out bit-identical
        assert torch.equal(dk.view(torch.int16), rk.view(torch.int16))
        assert torch.equal(dv.view(torch.int16), rv.view(torch.int16))
        # dQ is summed in fp32 by the copy engine in an order that is not fixed: equal within the gradient tolerance
        assert rel_l2(to_f64(dq), to_f64(rq)) <= GRAD_REL_L2
        assert not torch.isnan(dq.float()).any()


def test_static_scratch_backward_matches_the_oracle_on_the_tiny_config():
    """Not only equal to the other entry point: right.  The tiny configuration against the fp64 oracle."""
    w = W.tiny()
    q, k, v = w.qkv()
    do = w.dout()
    qd, kd, vd, dod = (to_dev(x) for x in (q, k, v, do))
    plan = B.seg_plan(w.patch_counts, B.TRAINED).to_device()
    o = torch.empty_like(qd)
    lse = torch.empty((w.n_heads, w.total_tokens), dtype=torch.float32, device="cuda")
    st = status_buf()
    B.varlen_attn_fwd(qd, kd, vd, o, lse, plan, w.softmax_scale, st)
    grads = [torch.empty_like(qd) for _ in range(3)]
    B.varlen_attn_bwd_static(dod, qd, kd, vd, o, lse, *grads, plan, w.softmax_scale, st)
    torch.cuda.synchronize()
    assert st.cpu().tolist()[0] == 0
    for g, r in zip(grads, oracle.attn_bwd(do, q, k, v, w.cu_seqlens, w.softmax_scale)):
        assert rel_l2(to_f64(g), r) <= GRAD_REL_L2


def test_a_warm_static_call_leaves_the_device_memory_as_it_found_it():
    """What the entry point promises: once the library's device code is resident (first call), a call takes no
    device memory from the driver or from torch's pool."""
    counts, H, D = [300, 129], 4, 64
    T = sum(counts)
    q, k, v, do = (to_dev(W.normal_bf16(74, s, (T, H, D))) for s in (1, 2, 3, 4))
    plan = B.seg_plan(counts, B.TRAINED).to_device()
    o = torch.empty_like(q)
    lse = torch.empty((H, T), dtype=torch.float32, device="cuda")
    grads = [torch.empty_like(q) for _ in range(3)]
    B.varlen_attn_fwd(q, k, v, o, lse, plan, 0.125)
    B.varlen_attn_bwd_static(do, q, k, v, o, lse, *grads, plan, 0.125)       # warm-up: module load, address look-up
    torch.cuda.synchronize()
    free0, alloc0, reserved0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    B.varlen_attn_bwd_static(do, q, k, v, o, lse, *grads, plan, 0.125)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0
    assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == reserved0


def test_bad_arguments_get_the_status_the_workspace_entry_point_gives():
    """Unsupported head_dim and misaligned strides are reported as by mpipe_varlen_attn_bwd, also for a problem that
    would not fit the scratch (the shared checks run before the size check).  Raw C-ABI calls: the Python wrapper's
    own assertions would stop these before the library sees them."""
    lib = B.load()
    T, H = 20000, 16
    x = torch.zeros((T, H, 128), dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros((H, T), dtype=torch.float32, device="cuda")
    ws = torch.zeros(1024, dtype=torch.uint8, device="cuda")
    plan = B.seg_plan([T], B.TRAINED).to_device()
    p = lambda t: ctypes.c_void_p(t.data_ptr())

    def both(head_dim, tok_stride, head_stride):
        common = [p(x)] * 5 + [p(lse)] + [p(x)] * 3 + [tok_stride, head_stride] * 3 + \
                 [p(plan.cu_seqlens_dev), plan.n_seg, T, plan.max_seqlen, p(plan.bwd_items_dev), int(plan.bwd_items.size),
                  H, head_dim, ctypes.c_float(0.125), B.TRAINED]
        a = lib.mpipe_varlen_attn_bwd(*common, p(ws), ctypes.c_size_t(1024), None, None)
        b = lib.mpipe_varlen_attn_bwd_static(*common, None, None)
        return a, b

    assert both(128, H * 128, 128) == (B.ERR_UNSUPPORTED, B.ERR_UNSUPPORTED)
    assert both(64, H * 128 + 4, 128) == (B.ERR_INVALID_ARG, B.ERR_INVALID_ARG)
    assert both(64, H * 128, 128) == (B.ERR_WORKSPACE, B.ERR_WORKSPACE)     # well-formed but too large / too small


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
