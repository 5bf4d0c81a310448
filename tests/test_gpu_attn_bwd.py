"""GPU parity of mpipe_varlen_attn_bwd against the fp64 oracle, and the trainability gate of
Lemma 1: a frozen encoder launches no backward and touches no gradient buffer."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_03229_b200 import binding as B
from paper_2607_03229_b200 import workloads as W
from _util import GRAD_REL_L2, max_abs, rel_l2, status_buf, to_dev, to_f64

pytestmark = pytest.mark.gpu


def gpu_fwd_bwd(q, k, v, do, counts, scale, mode=B.TRAINED):
    """Forward then backward through the C ABI.  Returns (o, lse, dq, dk, dv) device tensors."""
    T, H, D = q.shape
    plan = B.seg_plan(counts, mode).to_device()
    qd, kd, vd, dod = to_dev(q), to_dev(k), to_dev(v), to_dev(do)
    o = torch.empty_like(qd)
    lse = torch.empty((H, T), dtype=torch.float32, device="cuda") if mode == B.TRAINED else None
    st = status_buf()
    B.varlen_attn_fwd(qd, kd, vd, o, lse, plan, scale, st)
    pad = 2
    grads = [torch.full((T + 2 * pad, H, D), 333.0, dtype=torch.bfloat16, device="cuda") for _ in range(3)]
    dq, dk, dv = (g[pad:pad + T] for g in grads)
    ws_bytes = B.attn_workspace_bytes(T, H, D, mode)
    ws = torch.empty(max(ws_bytes, 1), dtype=torch.uint8, device="cuda")
    B.varlen_attn_bwd(dod, qd, kd, vd, o, lse, dq, dk, dv, plan, scale, ws, st)
    torch.cuda.synchronize()
    assert st.cpu().tolist()[0] == 0, f"device status {st.cpu().tolist()}"
    for g in grads:
        assert torch.all(g[:pad] == 333.0) and torch.all(g[pad + T:] == 333.0), "canary rows overwritten"
    return o, lse, dq, dk, dv


def check_bwd(counts, H, D, seed, scale=None):
    T = int(sum(counts))
    q, k, v, do = (W.normal_bf16(seed, s, (T, H, D)) for s in (1, 2, 3, 4))
    scale = float(np.float32(1.0 / np.sqrt(D))) if scale is None else scale
    _, _, dq, dk, dv = gpu_fwd_bwd(q, k, v, do, counts, scale)
    cu = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    ref = oracle.attn_bwd(do, q, k, v, cu, scale)
    errs = {}
    for name, g, r in zip(("dq", "dk", "dv"), (dq, dk, dv), ref):
        x = to_f64(g)
        assert not np.isnan(x).any(), name
        if np.linalg.norm(r) == 0:      # single-token segments only: dQ = dK = 0 exactly
            assert np.abs(x).max() <= 1e-2, name
            continue
        errs[name] = rel_l2(x, r)
        assert errs[name] <= GRAD_REL_L2, (counts, name, errs[name])
    return errs


def test_tiny_config():
    w = W.tiny()
    check_bwd(w.patch_counts, w.n_heads, w.head_dim, w.seed, w.softmax_scale)


@pytest.mark.parametrize("D", [64, 80])
@pytest.mark.parametrize("counts", [
    [1], [16], [127], [128], [129], [255], [256], [257], [385], [700],
    [1, 5, 0, 127, 128, 129, 0, 255, 256, 257, 300, 513],
    [1040, 3, 260],
])
def test_ragged_segments(counts, D):
    check_bwd(counts, 2, D, seed=200 + sum(counts) + D)


@pytest.mark.parametrize("D", [64, 80])
def test_many_units_per_cta(D):
    counts = [int(x) for x in W.rand_int(19, 1, 24, 40, 900)]
    check_bwd(counts, 8, D, seed=19)


def _random_mix(seed):
    """Segment lengths drawn around the tile edges (64, 128, 256 rows) and from a wide range, some empty."""
    edges = [1, 2, 15, 16, 17, 63, 64, 65, 127, 128, 129, 191, 192, 193, 255, 256, 257, 383, 384, 385, 511, 512, 513]
    n_seg = int(W.rand_int(seed, 1, 1, 3, 10)[0])
    pick = W.rand_int(seed, 2, n_seg, 0, 3)
    edge = W.rand_int(seed, 3, n_seg, 0, len(edges) - 1)
    wide = W.rand_int(seed, 4, n_seg, 1, 700)
    return [0 if pick[i] == 0 and i % 4 == 3 else (edges[int(edge[i])] if pick[i] < 2 else int(wide[i])) for i in range(n_seg)]


@pytest.mark.parametrize("D", [64, 80])
@pytest.mark.parametrize("seed", range(8))
def test_random_length_mixes_forward_and_backward(seed, D):
    """A seeded sweep over mixes of segment lengths at and around the tile edges, odd head counts included: the
    forward output, the LSE it hands to the backward and all three gradients against the oracle."""
    counts = _random_mix(1000 + seed)
    if sum(counts) == 0:
        counts = counts + [130]
    H = 1 + (seed % 3)
    T = int(sum(counts))
    q, k, v, do = (W.normal_bf16(3000 + seed, s, (T, H, D)) for s in (1, 2, 3, 4))
    scale = float(np.float32(1.0 / np.sqrt(D)))
    o, lse, dq, dk, dv = gpu_fwd_bwd(q, k, v, do, counts, scale)
    cu = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    O_ref, L_ref = oracle.attn_fwd(q, k, v, cu, scale)
    assert max_abs(to_f64(o), O_ref) <= 1e-2 and rel_l2(to_f64(o), O_ref) <= 5e-3, counts
    assert max_abs(to_f64(lse), L_ref) <= 1e-3, counts
    ref = oracle.attn_bwd(do, q, k, v, cu, scale)
    for name, g, r in zip(("dq", "dk", "dv"), (dq, dk, dv), ref):
        if np.linalg.norm(r) == 0:
            assert np.abs(to_f64(g)).max() <= 1e-2, (counts, name)
        else:
            assert rel_l2(to_f64(g), r) <= GRAD_REL_L2, (counts, name, rel_l2(to_f64(g), r))


@pytest.mark.parametrize("D", [64, 80])
def test_repeated_backward_is_stable(D):
    """The same inputs five times over: dK and dV (one issuing warp, fixed accumulation order) come out bit-identical,
    dQ (fp32 reduce-add in the copy engine, order not fixed) within a bf16 rounding step."""
    counts = [300, 129, 513, 64, 257]
    T, H = sum(counts), 4
    q, k, v, do = (W.normal_bf16(77, s, (T, H, D)) for s in (1, 2, 3, 4))
    scale = float(np.float32(1.0 / np.sqrt(D)))
    first = None
    for _ in range(5):
        _, _, dq, dk, dv = gpu_fwd_bwd(q, k, v, do, counts, scale)
        got = [x.clone() for x in (dq, dk, dv)]
        if first is None:
            first = got
            continue
        assert torch.equal(got[1], first[1]) and torch.equal(got[2], first[2])
        a, b = to_f64(got[0]), to_f64(first[0])
        assert np.abs(a - b).max() <= 2.0 ** -7 * max(1.0, np.abs(b).max())


def test_frozen_backward_is_a_noop():
    w = W.tiny()
    q, k, v = w.qkv()
    do = w.dout()
    plan = B.seg_plan(w.patch_counts, B.FROZEN).to_device()
    qd, kd, vd, dod = to_dev(q), to_dev(k), to_dev(v), to_dev(do)
    o = torch.empty_like(qd)
    B.varlen_attn_fwd(qd, kd, vd, o, None, plan, w.softmax_scale)
    grads = [torch.full_like(qd, 5.0) for _ in range(3)]
    B.varlen_attn_bwd(dod, qd, kd, vd, o, None, *grads, plan, w.softmax_scale, None)
    torch.cuda.synchronize()
    assert all(torch.all(g == 5.0) for g in grads)
    assert plan.bwd_items.size == 0 and B.attn_workspace_bytes(229, 4, 64, B.FROZEN) == 0


def test_gradient_identities_on_gpu_output():
    """Properties that hold for the exact gradient at any size: sum_j dV_j = sum_i dO_i per (segment,
    head), and <Q,dQ> = <K,dK>."""
    counts = [513, 190]
    T, H, D = sum(counts), 4, 64
    q, k, v, do = (W.normal_bf16(29, s, (T, H, D)) for s in (1, 2, 3, 4))
    _, _, dq, dk, dv = gpu_fwd_bwd(q, k, v, do, counts, 0.125)
    qf, kf, dof = (W.bf16_bits_to_f64(x) for x in (q, k, do))
    dqf, dkf, dvf = to_f64(dq), to_f64(dk), to_f64(dv)
    cu = [0, 513, 703]
    for s in range(2):
        a, b = cu[s], cu[s + 1]
        for h in range(H):
            sv, sd = dvf[a:b, h].sum(0), dof[a:b, h].sum(0)
            assert np.abs(sv - sd).max() <= 2e-2 * max(1.0, np.abs(sd).max())
            lhs, rhs = (qf[a:b, h] * dqf[a:b, h]).sum(), (kf[a:b, h] * dkf[a:b, h]).sum()
            assert abs(lhs - rhs) <= 2e-2 * max(1.0, abs(lhs))
