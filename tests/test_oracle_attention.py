"""Pins for the fp64 CPU oracle's attention forward and backward.

The paper prints no worked numerical example for this path, so each pin is mathematical and
independent of the oracle's own code: a dense masked brute force over the packed sequence,
a library (torch fp64 autograd) cross-check, central finite differences, closed forms and
invariances.  A dropped term, a wrong sign, a swapped operand or a segment leak fails at
least one of them.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_03229_b200 import workloads as W


def _inputs(counts, H, D, seed=7):
    T = int(sum(counts))
    q = W.normal_bf16(seed, 1, (T, H, D))
    k = W.normal_bf16(seed, 2, (T, H, D))
    v = W.normal_bf16(seed, 3, (T, H, D))
    do = W.normal_bf16(seed, 4, (T, H, D))
    cu = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    return q, k, v, do, cu


def _dense_masked(qf, kf, vf, cu, scale):
    """Brute force: one T x T score matrix over the packed sequence, -inf off the block diagonal."""
    T, H, D = qf.shape
    seg = np.zeros(T, dtype=np.int64)
    for s in range(len(cu) - 1):
        seg[cu[s]:cu[s + 1]] = s
    mask = seg[:, None] == seg[None, :]
    O = np.zeros_like(qf)
    LSE = np.zeros((H, T))
    P_all = np.zeros((H, T, T))
    for h in range(H):
        S = scale * (qf[:, h, :] @ kf[:, h, :].T)
        S = np.where(mask, S, -np.inf)
        E = np.exp(S - S.max(axis=1, keepdims=True))
        P = E / E.sum(axis=1, keepdims=True)
        P_all[h] = P
        O[:, h, :] = P @ vf[:, h, :]
        LSE[h] = np.log(np.exp(S).sum(axis=1))
    return O, LSE, P_all


COUNTS = [5, 1, 12, 0, 7]


def test_forward_matches_dense_masked_brute_force():
    q, k, v, _, cu = _inputs(COUNTS, 3, 8)
    scale = 0.37
    O, LSE = oracle.attn_fwd(q, k, v, cu, scale)
    Ob, Lb, _ = _dense_masked(W.bf16_bits_to_f64(q), W.bf16_bits_to_f64(k), W.bf16_bits_to_f64(v), cu,
                              float(np.float32(scale)))
    assert np.abs(O - Ob).max() < 1e-13
    assert np.abs(LSE - Lb).max() < 1e-13


def test_backward_matches_dense_masked_brute_force():
    q, k, v, do, cu = _inputs(COUNTS, 2, 8)
    scale = float(np.float32(0.41))
    qf, kf, vf, dof = (W.bf16_bits_to_f64(x) for x in (q, k, v, do))
    _, _, P = _dense_masked(qf, kf, vf, cu, scale)
    dQb, dKb, dVb = np.zeros_like(qf), np.zeros_like(qf), np.zeros_like(qf)
    for h in range(qf.shape[1]):
        dP = dof[:, h, :] @ vf[:, h, :].T
        dS = P[h] * (dP - (P[h] * dP).sum(axis=1, keepdims=True))  # softmax Jacobian, written densely
        dVb[:, h, :] = P[h].T @ dof[:, h, :]
        dQb[:, h, :] = scale * dS @ kf[:, h, :]
        dKb[:, h, :] = scale * dS.T @ qf[:, h, :]
    dQ, dK, dV = oracle.attn_bwd(do, q, k, v, cu, scale)
    for a, b in ((dQ, dQb), (dK, dKb), (dV, dVb)):
        assert np.abs(a - b).max() < 1e-12


def test_library_autograd_cross_check():
    """torch fp64 softmax(QK^T*scale)V per image, gradients from autograd."""
    q, k, v, do, cu = _inputs([9, 33, 17], 2, 16, seed=11)
    scale = float(np.float32(0.25))
    O, LSE = oracle.attn_fwd(q, k, v, cu, scale)
    dQ, dK, dV = oracle.attn_bwd(do, q, k, v, cu, scale)
    tq, tk, tv = (torch.tensor(W.bf16_bits_to_f64(x), requires_grad=True) for x in (q, k, v))
    tdo = torch.tensor(W.bf16_bits_to_f64(do))
    outs = []
    lses = []
    for s in range(len(cu) - 1):
        a, b = int(cu[s]), int(cu[s + 1])
        S = torch.einsum("ihd,jhd->hij", tq[a:b], tk[a:b]) * scale
        outs.append(torch.einsum("hij,jhd->ihd", torch.softmax(S, dim=-1), tv[a:b]))
        lses.append(torch.logsumexp(S, dim=-1))
    To = torch.cat(outs, dim=0)
    (To * tdo).sum().backward()
    assert np.abs(O - To.detach().numpy()).max() < 1e-12
    assert np.abs(LSE - torch.cat(lses, dim=1).detach().numpy()).max() < 1e-12
    assert np.abs(dQ - tq.grad.numpy()).max() < 1e-12
    assert np.abs(dK - tk.grad.numpy()).max() < 1e-12
    assert np.abs(dV - tv.grad.numpy()).max() < 1e-12


def test_gradient_by_central_finite_differences():
    """L = sum(O * dO); every input coordinate perturbed by +-h in fp64."""
    rng = np.random.default_rng(5)
    counts = [3, 6, 1]
    T, H, D = sum(counts), 2, 4
    cu = np.array([0, 3, 9, 10], dtype=np.int32)
    q, k, v, do = (rng.standard_normal((T, H, D)) for _ in range(4))
    scale = float(np.float32(0.5))
    dQ, dK, dV = oracle.attn_bwd(do, q, k, v, cu, scale)

    def loss(q_, k_, v_):
        return float((oracle.attn_fwd(q_, k_, v_, cu, scale)[0] * do).sum())

    h = 1e-6
    for name, x, g in (("q", q, dQ), ("k", k, dK), ("v", v, dV)):
        num = np.zeros_like(x)
        for idx in np.ndindex(*x.shape):
            old = x[idx]
            x[idx] = old + h
            lp = loss(q, k, v)
            x[idx] = old - h
            lm = loss(q, k, v)
            x[idx] = old
            num[idx] = (lp - lm) / (2 * h)
        rel = np.linalg.norm(num - g) / np.linalg.norm(g)
        assert rel < 1e-7, (name, rel)


def test_softmax_rows_sum_to_one_via_lse():
    q, k, v, _, cu = _inputs([20, 9], 2, 8, seed=3)
    scale = float(np.float32(0.3))
    _, LSE = oracle.attn_fwd(q, k, v, cu, scale)
    qf, kf = W.bf16_bits_to_f64(q), W.bf16_bits_to_f64(k)
    for s in range(2):
        a, b = cu[s], cu[s + 1]
        for h in range(2):
            S = scale * qf[a:b, h] @ kf[a:b, h].T
            assert np.abs(np.exp(S - LSE[h, a:b, None]).sum(axis=1) - 1.0).max() < 1e-13


def test_packed_equals_one_image_at_a_time_and_single_segment_is_full_attention():
    counts = [13, 40, 6]
    q, k, v, do, cu = _inputs(counts, 2, 8, seed=21)
    scale = float(np.float32(0.35))
    O, LSE = oracle.attn_fwd(q, k, v, cu, scale)
    dQ, dK, dV = oracle.attn_bwd(do, q, k, v, cu, scale)
    for s in range(3):
        a, b = cu[s], cu[s + 1]
        one = np.array([0, b - a], dtype=np.int32)
        Os, Ls = oracle.attn_fwd(q[a:b], k[a:b], v[a:b], one, scale)
        assert np.array_equal(Os, O[a:b]) and np.array_equal(Ls, LSE[:, a:b])
        g = oracle.attn_bwd(do[a:b], q[a:b], k[a:b], v[a:b], one, scale)
        assert np.array_equal(g[0], dQ[a:b]) and np.array_equal(g[1], dK[a:b]) and np.array_equal(g[2], dV[a:b])
        # a single segment is plain unmasked attention
        qf, kf, vf = (W.bf16_bits_to_f64(x[a:b]) for x in (q, k, v))
        for h in range(2):
            S = scale * qf[:, h] @ kf[:, h].T
            P = np.exp(S - S.max(1, keepdims=True))
            P /= P.sum(1, keepdims=True)
            assert np.abs(P @ vf[:, h] - Os[:, h]).max() < 1e-13


def test_closed_forms():
    counts = [7, 19, 1]
    q, k, v, do, cu = _inputs(counts, 2, 8, seed=33)
    scale = float(np.float32(0.2))
    vf, kf, qf, dof = (W.bf16_bits_to_f64(x) for x in (v, k, q, do))
    zero = np.zeros_like(q)  # bf16 +0.0 bits
    # Q = 0: uniform attention -> O = segment mean of V, LSE = ln n; dK = 0; dV = mean of dO rows
    O, LSE = oracle.attn_fwd(zero, k, v, cu, scale)
    dQ, dK, dV = oracle.attn_bwd(do, zero, k, v, cu, scale)
    for s, n in enumerate(counts):
        a, b = cu[s], cu[s + 1]
        assert np.abs(O[a:b] - vf[a:b].mean(axis=0, keepdims=True)).max() < 1e-14
        assert np.abs(LSE[:, a:b] - np.log(n)).max() < 1e-14
        assert np.abs(dV[a:b] - dof[a:b].sum(axis=0, keepdims=True) / n).max() < 1e-13
    assert np.abs(dK).max() == 0.0
    # all keys of a segment equal: O = mean V, LSE = scale*q.k + ln n
    keq = k.copy()
    for s in range(3):
        keq[cu[s]:cu[s + 1]] = k[cu[s]]
    O, LSE = oracle.attn_fwd(q, keq, v, cu, scale)
    for s, n in enumerate(counts):
        a, b = cu[s], cu[s + 1]
        assert np.abs(O[a:b] - vf[a:b].mean(axis=0, keepdims=True)).max() < 1e-13
        ref = scale * np.einsum("ihd,hd->hi", qf[a:b], kf[a]) + np.log(n)
        assert np.abs(LSE[:, a:b] - ref).max() < 1e-13
    # n = 1 segment: O = V, LSE = scale q.k, dV = dO, dQ = dK = 0
    O, LSE = oracle.attn_fwd(q, k, v, cu, scale)
    dQ, dK, dV = oracle.attn_bwd(do, q, k, v, cu, scale)
    i = cu[2]
    assert np.array_equal(O[i], vf[i])
    assert np.abs(LSE[:, i] - scale * (qf[i] * kf[i]).sum(-1)).max() < 1e-14
    assert np.array_equal(dV[i], dof[i]) and np.abs(dQ[i]).max() < 1e-15 and np.abs(dK[i]).max() < 1e-15
    # dO = 0 -> all gradients vanish
    g = oracle.attn_bwd(zero, q, k, v, cu, scale)
    assert all(np.abs(x).max() == 0.0 for x in g)


def test_segment_leak_detector():
    """V constant per segment (= segment id): any cross-segment weight shows as a non-integer."""
    counts = [4, 9, 2, 30]
    q, k, _, _, cu = _inputs(counts, 2, 8, seed=44)
    T = sum(counts)
    vals = np.zeros((T, 2, 8), dtype=np.float32)
    for s in range(4):
        vals[cu[s]:cu[s + 1]] = float(s + 1)
    O, _ = oracle.attn_fwd(q, k, W.f32_to_bf16_bits(vals), cu, 1.0)
    assert np.abs(O - vals).max() < 1e-14


def test_invariances():
    counts = [11, 23]
    q, k, v, do, cu = _inputs(counts, 2, 8, seed=55)
    scale = float(np.float32(0.3))
    O, LSE = oracle.attn_fwd(q, k, v, cu, scale)
    # permuting keys/values inside each segment leaves O and LSE unchanged
    perm = np.concatenate([np.random.default_rng(1).permutation(11), 11 + np.random.default_rng(2).permutation(23)])
    O2, L2 = oracle.attn_fwd(q, k[perm], v[perm], cu, scale)
    assert np.abs(O - O2).max() < 1e-13 and np.abs(LSE - L2).max() < 1e-13
    # swapping the two segments permutes rows
    sw = np.concatenate([np.arange(11, 34), np.arange(0, 11)])
    O3, L3 = oracle.attn_fwd(q[sw], k[sw], v[sw], np.array([0, 23, 34], dtype=np.int32), scale)
    assert np.array_equal(O3, O[sw]) and np.array_equal(L3, LSE[:, sw])
    # adding a vector c to every key shifts LSE_i by scale*q_i.c and leaves O unchanged
    qf, kf, vf = (W.bf16_bits_to_f64(x) for x in (q, k, v))
    c = np.random.default_rng(3).standard_normal((1, 2, 8))
    O4, L4 = oracle.attn_fwd(qf, kf + c, vf, cu, scale)
    assert np.abs(O4 - O).max() < 1e-12
    assert np.abs(L4 - (LSE + scale * np.einsum("ihd,hd->hi", qf, c[0]))).max() < 1e-12


def test_gradient_identities():
    counts = [14, 27]
    q, k, v, do, cu = _inputs(counts, 3, 8, seed=66)
    scale = float(np.float32(0.3))
    dQ, dK, dV = oracle.attn_bwd(do, q, k, v, cu, scale)
    qf, kf, dof = (W.bf16_bits_to_f64(x) for x in (q, k, do))
    for s in range(2):
        a, b = cu[s], cu[s + 1]
        for h in range(3):
            # <Q,dQ> = <K,dK> (both equal scale * sum_ij dS_ij S_ij / scale)
            assert abs((qf[a:b, h] * dQ[a:b, h]).sum() - (kf[a:b, h] * dK[a:b, h]).sum()) < 1e-11
            # columns of P sum over rows: sum_j dV_j = sum_i dO_i
            assert np.abs(dV[a:b, h].sum(0) - dof[a:b, h].sum(0)).max() < 1e-12
            # sum_j dS_ij = 0  =>  dQ_i is orthogonal to any common key offset: sum_j dS_ij (k_j + c) same
    # rows of dS sum to zero: shifting all keys by c leaves dQ unchanged
    c = np.random.default_rng(4).standard_normal((1, 3, 8))
    vf = W.bf16_bits_to_f64(v)
    dQ2, _, _ = oracle.attn_bwd(dof, qf, kf + c, vf, cu, scale)
    assert np.abs(dQ2 - dQ).max() < 1e-12


def test_sampled_entry_points_match_full():
    counts = [31, 8, 50]
    q, k, v, do, cu = _inputs(counts, 3, 16, seed=77)
    scale = float(np.float32(0.25))
    O, LSE = oracle.attn_fwd(q, k, v, cu, scale)
    dQ, dK, dV = oracle.attn_bwd(do, q, k, v, cu, scale)
    rows = np.array([0, 30, 31, 38, 39, 88, 60])
    heads = np.array([0, 1, 2, 0, 1, 2, 1])
    Or, Lr = oracle.attn_fwd_rows(q, k, v, cu, scale, rows, heads)
    assert np.array_equal(Or, O[rows, heads]) and np.array_equal(Lr, LSE[heads, rows])
    dQr = oracle.attn_bwd_dq_rows(do, q, k, v, cu, scale, rows, heads)
    assert np.array_equal(dQr, dQ[rows, heads])
    kr = np.array([39, 88, 50])
    dKr, dVr = oracle.attn_bwd_dkv_rows(do, q, k, v, cu, scale, 2, 1, kr)
    assert np.array_equal(dKr, dK[kr, 1]) and np.array_equal(dVr, dV[kr, 1])


def test_bf16_widening_is_exact():
    # 1.0, -2.0, 0.5, smallest normal-ish pattern, 3.140625 (0x4049)
    bits = np.array([0x3F80, 0xC000, 0x3F00, 0x0080, 0x4049], dtype=np.uint16)
    assert np.array_equal(W.bf16_bits_to_f64(bits), np.array([1.0, -2.0, 0.5, 2.0 ** -126, 3.140625]))
    x = np.array([1.0, 1.00390625, 1.005859375, -3.0e-3], dtype=np.float32)
    # RNE: 1 + 2^-8 is a tie -> rounds to even (1.0); 1 + 1.5*2^-8 rounds up to 1 + 2^-7
    r = W.bf16_bits_to_f32(W.f32_to_bf16_bits(x))
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == 1.0078125
    tb = torch.tensor(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(tb, W.f32_to_bf16_bits(x))
    # n = 1 attention returns V itself: the widening inside the oracle wrapper is the same map
    v = W.normal_bf16(9, 9, (1, 1, 8))
    O, _ = oracle.attn_fwd(v, v, v, np.array([0, 1], dtype=np.int32), 1.0)
    assert np.array_equal(O, W.bf16_bits_to_f64(v))
