"""Pins of the encoder-layer oracle (oracle/layer.py) against what fixes it from outside: torch's fp64
functional ops (library routines), closed forms, and cases that reduce to something simpler."""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
from oracle import layer as L


def _rand_weights(rng, hidden, ffn, scale=0.2):
    def r(*s):
        return rng.standard_normal(s) * scale
    return L.LayerWeights(g1=1 + r(hidden), b1=r(hidden), wqkv=r(3 * hidden, hidden), bqkv=r(3 * hidden),
                          wo=r(hidden, hidden), bo=r(hidden), g2=1 + r(hidden), b2=r(hidden),
                          w1=r(ffn, hidden), bb1=r(ffn), w2=r(hidden, ffn), bb2=r(hidden))


def test_layernorm_matches_torch_and_normalises():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((7, 48)) * 3 + 1.5
    g, b = rng.standard_normal(48), rng.standard_normal(48)
    ref = F.layer_norm(torch.from_numpy(x), (48,), torch.from_numpy(g), torch.from_numpy(b), 1e-6).numpy()
    np.testing.assert_allclose(L.layernorm(x, g, b, 1e-6), ref, rtol=0, atol=1e-12)
    z = L.layernorm(x, np.ones(48), np.zeros(48), 1e-6)
    np.testing.assert_allclose(z.mean(axis=1), 0, atol=1e-13)
    var = x.var(axis=1)
    np.testing.assert_allclose(z.var(axis=1), var / (var + 1e-6), rtol=1e-12)
    # shift / scale invariance of the normalised value (eps -> 0)
    np.testing.assert_allclose(L.layernorm(5 * x + 3, g, b, 0.0), L.layernorm(x, g, b, 0.0), atol=1e-11)


def test_linear_matches_torch_on_non_square_shapes():
    rng = np.random.default_rng(2)
    x, w, b = rng.standard_normal((5, 12)), rng.standard_normal((9, 12)), rng.standard_normal(9)
    ref = F.linear(torch.from_numpy(x), torch.from_numpy(w), torch.from_numpy(b)).numpy()
    np.testing.assert_allclose(L.linear(x, w, b), ref, atol=1e-13)
    # one-hot input picks a column of w (catches a transposed operand)
    e = np.zeros((1, 12)); e[0, 3] = 1
    np.testing.assert_allclose(L.linear(e, w)[0], w[:, 3], atol=0)


def test_gelu_closed_forms_and_torch():
    phi1 = 0.5 * (1 + math.erf(1 / math.sqrt(2)))   # standard normal CDF at 1 = 0.841344746...
    assert abs(phi1 - 0.8413447460685429) < 1e-15
    np.testing.assert_allclose(L.gelu(np.array([0.0, 1.0, -1.0])), [0.0, phi1, -(1 - phi1)], atol=1e-15)
    u = np.linspace(-6, 6, 241)
    np.testing.assert_allclose(L.gelu(u) - L.gelu(-u), u, atol=1e-14)          # u Phi(u) + u Phi(-u)... = u
    np.testing.assert_allclose(L.gelu(u), F.gelu(torch.from_numpy(u)).numpy(), atol=1e-14)
    assert abs(L.gelu(np.array([30.0]))[0] - 30.0) < 1e-12 and abs(L.gelu(np.array([-30.0]))[0]) < 1e-12


def _torch_layer(x, w, counts, H, scale, eps):
    """The same block from torch fp64 library ops and a dense block-diagonal mask."""
    t = lambda a: torch.from_numpy(np.asarray(a, dtype=np.float64))
    T, hidden = x.shape
    D = hidden // H
    X = t(x)
    a = F.layer_norm(X, (hidden,), t(w.g1), t(w.b1), eps)
    qkv = F.linear(a, t(w.wqkv), t(w.bqkv))
    q, k, v = (qkv[:, i * hidden:(i + 1) * hidden].reshape(T, H, D).permute(1, 0, 2) for i in range(3))
    seg = torch.repeat_interleave(torch.arange(len(counts)), torch.tensor(counts))
    mask = seg[:, None] == seg[None, :]
    s = (q @ k.transpose(1, 2)) * scale
    s = s.masked_fill(~mask, float("-inf"))
    o = (torch.softmax(s, dim=-1) @ v).permute(1, 0, 2).reshape(T, hidden)
    x1 = X + F.linear(o, t(w.wo), t(w.bo))
    m = F.layer_norm(x1, (hidden,), t(w.g2), t(w.b2), eps)
    y = x1 + F.linear(F.gelu(F.linear(m, t(w.w1), t(w.bb1))), t(w.w2), t(w.bb2))
    return y.numpy()


@pytest.mark.parametrize("counts,H,D", [([5, 1, 9], 2, 8), ([16, 7], 3, 16)])
def test_layer_matches_torch_composite(counts, H, D):
    rng = np.random.default_rng(3)
    hidden, ffn = H * D, 3 * H * D
    w = _rand_weights(rng, hidden, ffn)
    x = rng.standard_normal((sum(counts), hidden))
    cu = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    scale = float(np.float32(1 / math.sqrt(D)))   # the scale is an fp32 input of the attention oracle, as in the C ABI
    y, parts = L.encoder_layer_fwd(x, w, cu, H, scale, 1e-6)
    np.testing.assert_allclose(y, _torch_layer(x, w, counts, H, scale, 1e-6), atol=1e-11)
    assert parts["qkv"].shape == (sum(counts), 3 * hidden) and parts["f"].shape == (sum(counts), ffn)


def test_layer_special_cases():
    rng = np.random.default_rng(4)
    H, D = 2, 8
    hidden, ffn = H * D, 32
    w = _rand_weights(rng, hidden, ffn)
    x = rng.standard_normal((6, hidden))
    # zero output projections: both residual branches vanish
    w0 = L.LayerWeights(**{**w.__dict__, "wo": np.zeros_like(w.wo), "bo": np.zeros_like(w.bo),
                           "w2": np.zeros_like(w.w2), "bb2": np.zeros_like(w.bb2)})
    y, _ = L.encoder_layer_fwd(x, w0, np.array([0, 2, 6], dtype=np.int32), H, 0.3, 1e-6)
    np.testing.assert_allclose(y, x, atol=0)
    # one-token images: attention returns v, so x1 = x + Wo v + bo
    cu = np.arange(7, dtype=np.int32)
    _, parts = L.encoder_layer_fwd(x, w, cu, H, 0.3, 1e-6)
    v = parts["qkv"][:, 2 * hidden:]
    np.testing.assert_allclose(parts["x1"], x + v @ w.wo.T + w.bo, atol=1e-12)
    # bf16 bit patterns widen exactly
    bits = (np.float32(1.5).view(np.uint32) >> 16).astype(np.uint16)
    assert L.widen(np.array([[bits]], dtype=np.uint16))[0, 0] == 1.5


def test_rope_is_a_rotation_and_matches_complex_form():
    rng = np.random.default_rng(5)
    T, H, D = 9, 2, 16
    x = rng.standard_normal((T, H, D))
    ang = rng.uniform(-3, 3, (T, D // 2))
    y = L.rope(x, np.cos(ang), np.sin(ang))
    # the same thing as a complex multiplication of (x1 + i x2) by exp(i angle)
    z = (x[..., :D // 2] + 1j * x[..., D // 2:]) * np.exp(1j * ang)[:, None, :]
    np.testing.assert_allclose(y, np.concatenate([z.real, z.imag], axis=-1), atol=1e-14)
    np.testing.assert_allclose((y ** 2).sum(-1), (x ** 2).sum(-1), rtol=1e-13)          # norms are kept
    np.testing.assert_allclose(L.rope(x, np.ones((T, D // 2)), np.zeros((T, D // 2))), x, atol=0)   # angle 0
    back = L.rope(y, np.cos(-ang), np.sin(-ang))
    np.testing.assert_allclose(back, x, atol=1e-13)


def test_rope_scores_depend_on_relative_position_only():
    rng = np.random.default_rng(6)
    D = 8
    q, k = rng.standard_normal((1, 1, D)), rng.standard_normal((1, 1, D))
    inv = 10000.0 ** (-np.arange(D // 2) / (D // 2))

    def score(m, n):
        qa = L.rope(q, np.cos(m * inv)[None], np.sin(m * inv)[None])
        ka = L.rope(k, np.cos(n * inv)[None], np.sin(n * inv)[None])
        return float((qa * ka).sum())
    assert abs(score(5, 2) - score(13, 10)) < 1e-12 and abs(score(5, 2) - score(5, 3)) > 1e-6


def test_layer_with_rope_matches_manual_composition():
    rng = np.random.default_rng(7)
    H, D = 2, 8
    hidden, ffn = H * D, 24
    w = _rand_weights(rng, hidden, ffn)
    x = rng.standard_normal((7, hidden))
    cu = np.array([0, 3, 7], dtype=np.int32)
    ang = rng.uniform(-2, 2, (7, D // 2))
    tabs = (np.cos(ang), np.sin(ang))
    _, parts = L.encoder_layer_fwd(x, w, cu, H, 0.25, 1e-6, rope_tables=tabs)
    qkv = parts["qkv"]
    q, k, v = (qkv[:, i * hidden:(i + 1) * hidden].reshape(7, H, D) for i in range(3))
    o_ref, _ = oracle.attn_fwd(np.ascontiguousarray(L.rope(q, *tabs)), np.ascontiguousarray(L.rope(k, *tabs)),
                               np.ascontiguousarray(v), cu, 0.25)
    np.testing.assert_allclose(parts["o"], o_ref, atol=1e-14)


def test_gelu_grad_and_linear_grads_against_finite_differences_and_autograd():
    u = np.linspace(-5, 5, 101)
    h = 1e-6
    np.testing.assert_allclose(L.gelu_grad(u), (L.gelu(u + h) - L.gelu(u - h)) / (2 * h), atol=1e-9)
    assert L.gelu_grad(np.array([0.0]))[0] == 0.5
    rng = np.random.default_rng(8)
    x, w, b = rng.standard_normal((5, 7)), rng.standard_normal((3, 7)), rng.standard_normal(3)
    dy = rng.standard_normal((5, 3))
    xt, wt, bt = (torch.tensor(a, requires_grad=True) for a in (x, w, b))
    (F.linear(xt, wt, bt) * torch.from_numpy(dy)).sum().backward()
    np.testing.assert_allclose(L.linear_dgrad(dy, w), xt.grad.numpy(), atol=1e-13)
    dw, db = L.linear_wgrad(dy, x)
    np.testing.assert_allclose(dw, wt.grad.numpy(), atol=1e-13)
    np.testing.assert_allclose(db, bt.grad.numpy(), atol=1e-13)


def test_layernorm_bwd_matches_autograd():
    rng = np.random.default_rng(9)
    x, dy = rng.standard_normal((6, 24)) * 2 + 1, rng.standard_normal((6, 24))
    g, b = 1 + 0.2 * rng.standard_normal(24), rng.standard_normal(24)
    xt, gt, bt = (torch.tensor(a, requires_grad=True) for a in (x, g, b))
    (F.layer_norm(xt, (24,), gt, bt, 1e-6) * torch.from_numpy(dy)).sum().backward()
    dx, dg, db = L.layernorm_bwd(x, dy, g, 1e-6)
    np.testing.assert_allclose(dx, xt.grad.numpy(), atol=1e-12)
    np.testing.assert_allclose(dg, gt.grad.numpy(), atol=1e-12)
    np.testing.assert_allclose(db, bt.grad.numpy(), atol=1e-12)
    np.testing.assert_allclose(dx.sum(axis=1), 0, atol=1e-12)      # the normalised value does not see a shift of the row


@pytest.mark.parametrize("with_rope", [False, True])
def test_layer_bwd_matches_torch_autograd(with_rope):
    rng = np.random.default_rng(10)
    counts, H, D = [5, 1, 9], 2, 8
    hidden, ffn, T = H * D, 3 * H * D, 15
    w = _rand_weights(rng, hidden, ffn)
    x, dy = rng.standard_normal((T, hidden)), rng.standard_normal((T, hidden))
    cu = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    scale = float(np.float32(1 / math.sqrt(D)))
    ang = rng.uniform(-2, 2, (T, D // 2))
    tabs = (np.cos(ang), np.sin(ang)) if with_rope else None
    dx, g = L.encoder_layer_bwd(x, w, cu, H, scale, 1e-6, dy, tabs)
    # the same block from torch ops with autograd
    t = lambda a: torch.tensor(np.asarray(a, dtype=np.float64), requires_grad=True)
    names = {"ln1_gamma": "g1", "ln1_beta": "b1", "w_qkv": "wqkv", "b_qkv": "bqkv", "w_o": "wo", "b_o": "bo", "ln2_gamma": "g2",
             "ln2_beta": "b2", "w_fc1": "w1", "b_fc1": "bb1", "w_fc2": "w2", "b_fc2": "bb2"}
    P = {k_: t(getattr(w, v_)) for k_, v_ in names.items()}
    X = t(x)
    a = F.layer_norm(X, (hidden,), P["ln1_gamma"], P["ln1_beta"], 1e-6)
    qkv = F.linear(a, P["w_qkv"], P["b_qkv"])
    q, k, v = (qkv[:, i * hidden:(i + 1) * hidden].reshape(T, H, D) for i in range(3))
    if with_rope:
        c, s_ = torch.from_numpy(tabs[0])[:, None, :], torch.from_numpy(tabs[1])[:, None, :]
        rot = lambda z: torch.cat([z[..., :D // 2] * c - z[..., D // 2:] * s_, z[..., D // 2:] * c + z[..., :D // 2] * s_], dim=-1)
        q, k = rot(q), rot(k)
    seg = torch.repeat_interleave(torch.arange(len(counts)), torch.tensor(counts))
    sc = (q.permute(1, 0, 2) @ k.permute(1, 2, 0)) * scale
    sc = sc.masked_fill(~(seg[:, None] == seg[None, :]), float("-inf"))
    o = (torch.softmax(sc, dim=-1) @ v.permute(1, 0, 2)).permute(1, 0, 2).reshape(T, hidden)
    x1 = X + F.linear(o, P["w_o"], P["b_o"])
    m = F.layer_norm(x1, (hidden,), P["ln2_gamma"], P["ln2_beta"], 1e-6)
    y = x1 + F.linear(F.gelu(F.linear(m, P["w_fc1"], P["b_fc1"])), P["w_fc2"], P["b_fc2"])
    (y * torch.from_numpy(dy)).sum().backward()
    np.testing.assert_allclose(dx, X.grad.numpy(), atol=1e-10)
    for k_ in names:
        np.testing.assert_allclose(g[k_], P[k_].grad.numpy(), atol=1e-10, err_msg=k_)


def test_layer_bwd_finite_difference_on_the_input():
    rng = np.random.default_rng(11)
    H, D = 2, 8
    hidden, ffn, T = H * D, 24, 6
    w = _rand_weights(rng, hidden, ffn)
    x, dy = rng.standard_normal((T, hidden)), rng.standard_normal((T, hidden))
    cu = np.array([0, 2, 6], dtype=np.int32)
    dx, _ = L.encoder_layer_bwd(x, w, cu, H, 0.25, 1e-6, dy)
    loss = lambda z: float((L.encoder_layer_fwd(z, w, cu, H, 0.25, 1e-6)[0] * dy).sum())
    h = 1e-6
    for (i, j) in [(0, 0), (3, 5), (5, 15)]:
        e = np.zeros_like(x); e[i, j] = h
        assert abs((loss(x + e) - loss(x - e)) / (2 * h) - dx[i, j]) < 1e-6
