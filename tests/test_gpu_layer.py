"""GPU parity of the encoder-layer entry points (linear, layernorm, whole layer) against oracle/layer.py."""
import math

import numpy as np
import pytest
import torch

from oracle import layer as OL
from paper_2607_03229_b200 import binding as B, workloads as W
from _util import to_dev, to_f64, rel_l2, status_buf

pytestmark = pytest.mark.gpu

# A bf16 result of an fp32-accumulated dot product: half an ulp of bf16 (2^-9 relative) plus the accumulation error.
ELEM_REL = 2.0 ** -8
LAYER_REL_L2 = 1e-2     # several bf16-rounded stages in a row (same bound as the attention gradients)


def _check_close(got, ref, atol):
    err = np.abs(got - ref)
    bound = atol + ELEM_REL * np.abs(ref)
    assert (err <= bound).all(), f"max excess {(err - bound).max():.3e} at {np.unravel_index((err - bound).argmax(), err.shape)}"


@pytest.mark.parametrize("M,N,K", [(1, 8, 8), (300, 264, 72), (257, 512, 1024), (1000, 1024, 1280), (129, 3072, 64)])
@pytest.mark.parametrize("bias,res,gelu", [(False, False, False), (True, False, True), (True, True, False)])
def test_linear_matches_oracle(M, N, K, bias, res, gelu):
    a = W.normal_bf16(11, 0, (M, K))
    w = W.scaled_normal_bf16(11, 1, (N, K), std=K ** -0.5)
    b = W.scaled_normal_bf16(11, 2, (N,), std=0.5) if bias else None
    r = W.normal_bf16(11, 3, (M, N)) if res else None
    c = torch.full((M, N), 7.0, dtype=torch.bfloat16, device="cuda")
    st = status_buf()
    B.linear_fwd(to_dev(a), to_dev(w), c, None if b is None else to_dev(b), None if r is None else to_dev(r), gelu, st)
    torch.cuda.synchronize()
    assert st.cpu().tolist()[0] == 0
    ref = OL.linear(OL.widen(a), OL.widen(w), None if b is None else OL.widen(b))
    if gelu:
        ref = OL.gelu(ref)
    if res:
        ref = ref + OL.widen(r)
    _check_close(to_f64(c), ref, atol=2e-3)


def test_linear_strided_rows_and_untouched_padding():
    M, N, K = 200, 256, 128
    a_full = to_dev(W.normal_bf16(12, 0, (M, K + 8)))
    c_full = torch.full((M + 3, N + 16), 5.0, dtype=torch.bfloat16, device="cuda")
    w = W.scaled_normal_bf16(12, 1, (N, K), std=K ** -0.5)
    B.linear_fwd(a_full[:, :K], to_dev(w), c_full[:M, :N])
    torch.cuda.synchronize()
    ref = OL.linear(to_f64(a_full[:, :K]), OL.widen(w))
    _check_close(to_f64(c_full[:M, :N]), ref, atol=2e-3)
    assert (c_full[M:, :] == 5.0).all() and (c_full[:, N:] == 5.0).all()


@pytest.mark.parametrize("T,hidden", [(1, 8), (37, 256), (1000, 1024), (513, 1280), (9, 2048)])
def test_layernorm_matches_oracle(T, hidden):
    x = W.scaled_normal_bf16(13, 0, (T, hidden), std=2.0, mean=0.7)
    g = W.scaled_normal_bf16(13, 1, (hidden,), std=0.1, mean=1.0)
    b = W.scaled_normal_bf16(13, 2, (hidden,), std=0.1)
    y = torch.empty((T, hidden), dtype=torch.bfloat16, device="cuda")
    B.layernorm_fwd(to_dev(x), to_dev(g), to_dev(b), y, 1e-6)
    torch.cuda.synchronize()
    ref = OL.layernorm(OL.widen(x), OL.widen(g), OL.widen(b), 1e-6)
    _check_close(to_f64(y), ref, atol=1e-4)


@pytest.mark.parametrize("counts,H,D", [([5, 1, 30], 2, 64), ([300, 77], 3, 80), ([1000], 16, 64)])
def test_rope_matches_oracle(counts, H, D):
    T, hidden = sum(counts), H * D
    qkv = W.normal_bf16(14, 0, (T, 3 * hidden))
    cos, sin = W.rope2d_tables(counts, D)
    dev = to_dev(qkv)
    B.rope_apply(dev, torch.from_numpy(cos).cuda(), torch.from_numpy(sin).cuda(), H, D)
    torch.cuda.synchronize()
    got = to_f64(dev)
    ref = OL.widen(qkv).copy()
    for i in range(2):   # q and k are rotated, v stays
        blk = ref[:, i * hidden:(i + 1) * hidden].reshape(T, H, D)
        ref[:, i * hidden:(i + 1) * hidden] = OL.rope(blk, cos.astype(np.float64), sin.astype(np.float64)).reshape(T, hidden)
    _check_close(got, ref, atol=1e-6)
    assert np.array_equal(got[:, 2 * hidden:], OL.widen(qkv)[:, 2 * hidden:])


def _run_layer(counts, H, D, ffn, mode, seed=21, rope=False):
    hidden = H * D
    T = sum(counts)
    pb = W.layer_params_bf16(seed, hidden, ffn)
    x = W.normal_bf16(seed, 0, (T, hidden))
    plan = B.seg_plan(counts, mode).to_device()
    weights = B.LayerWeights.from_tensors(**{k: to_dev(v) for k, v in pb.items()})
    y = torch.empty((T, hidden), dtype=torch.bfloat16, device="cuda")
    lse = torch.empty((H, T), dtype=torch.float32, device="cuda") if mode == B.TRAINED else None
    ws = torch.empty(B.encoder_layer_workspace_bytes(T, hidden, ffn), dtype=torch.uint8, device="cuda")
    st = status_buf()
    scale = float(np.float32(1 / math.sqrt(D)))
    tabs = W.rope2d_tables(counts, D) if rope else None
    rope_dev = None if tabs is None else tuple(torch.from_numpy(t).cuda() for t in tabs)
    B.encoder_layer_fwd(to_dev(x), y, weights, H, ffn, plan, scale, 1e-6, ws, lse, st, rope=rope_dev)
    torch.cuda.synchronize()
    assert st.cpu().tolist()[0] == 0
    ow = OL.LayerWeights(g1=OL.widen(pb["ln1_gamma"]), b1=OL.widen(pb["ln1_beta"]), wqkv=OL.widen(pb["w_qkv"]),
                         bqkv=OL.widen(pb["b_qkv"]), wo=OL.widen(pb["w_o"]), bo=OL.widen(pb["b_o"]),
                         g2=OL.widen(pb["ln2_gamma"]), b2=OL.widen(pb["ln2_beta"]), w1=OL.widen(pb["w_fc1"]),
                         bb1=OL.widen(pb["b_fc1"]), w2=OL.widen(pb["w_fc2"]), bb2=OL.widen(pb["b_fc2"]))
    cu = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    ref, parts = OL.encoder_layer_fwd(x, ow, cu, H, scale, 1e-6,
                                      rope_tables=None if tabs is None else tuple(t.astype(np.float64) for t in tabs))
    return to_f64(y), ref, (None if lse is None else lse.cpu().double().numpy()), parts


@pytest.mark.parametrize("counts,H,D,ffn", [([16, 49, 64, 100], 4, 64, 1024), ([300, 1, 129], 2, 80, 328),
                                            ([1024, 256, 777], 16, 64, 4096)])
def test_layer_matches_oracle(counts, H, D, ffn):
    y, ref, lse, parts = _run_layer(counts, H, D, ffn, B.TRAINED)
    assert rel_l2(y, ref) <= LAYER_REL_L2
    assert np.abs(y - ref).max() <= 0.05 + 2.0 ** -6 * np.abs(ref).max()
    assert np.abs(lse - parts["lse"]).max() <= 2e-2   # LSE of bf16-rounded q, k (the projections are stored as bf16)


def test_layer_attention_stage_holds_the_attention_bars_on_its_own_inputs():
    """The layer's LSE differs from the fp64 layer oracle's by up to 2e-2 only because the projections q, k are stored as
    bf16.  Fed the SAME rounded q, k, v (read back from the forward's workspace: normalised rows, then the packed
    [T, 3*hidden] projection, then the attention output) the attention oracle must agree with the layer's LSE and
    attention output at the attention bars."""
    counts, H, D, ffn = [300, 1, 129, 640], 4, 64, 1024
    hidden, T = H * D, sum(counts)
    pb = W.layer_params_bf16(31, hidden, ffn)
    x = W.normal_bf16(31, 0, (T, hidden))
    plan = B.seg_plan(counts, B.TRAINED).to_device()
    weights = B.LayerWeights.from_tensors(**{k: to_dev(v) for k, v in pb.items()})
    y = torch.empty((T, hidden), dtype=torch.bfloat16, device="cuda")
    lse = torch.empty((H, T), dtype=torch.float32, device="cuda")
    ws = torch.empty(B.encoder_layer_workspace_bytes(T, hidden, ffn), dtype=torch.uint8, device="cuda")
    st = status_buf()
    scale = float(np.float32(1 / math.sqrt(D)))
    B.encoder_layer_fwd(to_dev(x), y, weights, H, ffn, plan, scale, 1e-6, ws, lse, st)
    torch.cuda.synchronize()
    assert st.cpu().tolist()[0] == 0
    a256 = lambda n: (n + 255) // 256 * 256
    off_qkv = a256(T * hidden * 2)
    off_attn = off_qkv + a256(T * 3 * hidden * 2)
    raw = ws.cpu().numpy()
    qkv = raw[off_qkv:off_qkv + T * 3 * hidden * 2].view(np.uint16).reshape(T, 3, H, D)
    attn = raw[off_attn:off_attn + T * hidden * 2].view(np.uint16).reshape(T, H, D)
    import oracle
    cu = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    O_ref, L_ref = oracle.attn_fwd(np.ascontiguousarray(qkv[:, 0]), np.ascontiguousarray(qkv[:, 1]),
                                   np.ascontiguousarray(qkv[:, 2]), cu, scale)
    assert np.abs(lse.cpu().double().numpy() - L_ref).max() <= 1e-3
    O = W.bf16_bits_to_f64(attn)
    assert np.abs(O - O_ref).max() <= 1e-2 and rel_l2(O, O_ref) <= 5e-3


def test_layer_with_rope_matches_oracle():
    y, ref, lse, parts = _run_layer([300, 1, 129, 640], 4, 80, 1280, B.TRAINED, rope=True)
    assert rel_l2(y, ref) <= LAYER_REL_L2
    assert np.abs(lse - parts["lse"]).max() <= 2e-2


@pytest.mark.parametrize("counts,H,D,ffn,rope", [([200, 56], 4, 64, 512, False), ([300, 1, 129, 640], 4, 80, 1280, True),
                                                 ([1024, 256, 777], 16, 64, 4096, False)])
def test_layer_frozen_forward_has_the_trained_forward_bits(counts, H, D, ffn, rope):
    """Corollary 1 for the whole layer: freezing the encoder changes no forward bit.  The trained forward also keeps the
    MLP pre-activation for the backward; both it and GELU(.) come from the one fp32 accumulator, so the activation the
    next projection reads is the frozen forward's."""
    y_t, ref, _, _ = _run_layer(counts, H, D, ffn, B.TRAINED, rope=rope)
    y_f, _, lse, _ = _run_layer(counts, H, D, ffn, B.FROZEN, rope=rope)
    assert lse is None and np.array_equal(y_f, y_t) and rel_l2(y_f, ref) <= LAYER_REL_L2


def test_layer_argument_checks():
    T, hidden, ffn = 64, 256, 512
    ws = torch.empty(B.encoder_layer_workspace_bytes(T, hidden, ffn) - 256, dtype=torch.uint8, device="cuda")
    pb = W.layer_params_bf16(5, hidden, ffn)
    weights = B.LayerWeights.from_tensors(**{k: to_dev(v) for k, v in pb.items()})
    x = to_dev(W.normal_bf16(5, 0, (T, hidden)))
    y = torch.empty_like(x)
    plan = B.seg_plan([T], B.FROZEN).to_device()
    with pytest.raises(B.MpipeError) as e:
        B.encoder_layer_fwd(x, y, weights, 4, ffn, plan, 0.125, 1e-6, ws)
    assert e.value.status == B.ERR_WORKSPACE
    with pytest.raises(B.MpipeError):
        B.linear_fwd(x, to_dev(W.normal_bf16(5, 1, (12, hidden))), torch.empty((T, 12), dtype=torch.bfloat16, device="cuda"))


def test_linear_full_size_sampled_rows():
    """The bench's largest projection shapes (ViT-L layer: fc1 and fc2 on the 50 439-token microbatch), checked on sampled
    output rows that the oracle computes one by one."""
    w = W.vit_l()
    T, hidden, ffn = w.total_tokens, 1024, 4096
    g = torch.Generator(device="cuda")
    g.manual_seed(3)
    a = torch.randn((T, hidden), device="cuda", generator=g).to(torch.bfloat16)
    w1 = (torch.randn((ffn, hidden), device="cuda", generator=g) * hidden ** -0.5).to(torch.bfloat16)
    b1 = (torch.randn((ffn,), device="cuda", generator=g) * 0.5).to(torch.bfloat16)
    w2 = (torch.randn((hidden, ffn), device="cuda", generator=g) * ffn ** -0.5).to(torch.bfloat16)
    res = torch.randn((T, hidden), device="cuda", generator=g).to(torch.bfloat16)
    h = torch.empty((T, ffn), dtype=torch.bfloat16, device="cuda")
    y = torch.empty((T, hidden), dtype=torch.bfloat16, device="cuda")
    st = status_buf()
    B.linear_fwd(a, w1, h, b1, None, True, st)
    B.linear_fwd(h, w2, y, None, res, False, st)
    torch.cuda.synchronize()
    assert st.cpu().tolist()[0] == 0
    rows = np.unique(np.concatenate([[0, 1, 127, 128, T - 1, T - 2, (T // 128) * 128],
                                     np.random.default_rng(0).integers(0, T, 40)]))
    idx = torch.from_numpy(rows).cuda()
    h_ref = OL.gelu(OL.linear(to_f64(a[idx]), to_f64(w1), to_f64(b1)))
    _check_close(to_f64(h[idx]), h_ref, atol=2e-3)
    y_ref = OL.linear(to_f64(h[idx]), to_f64(w2)) + to_f64(res[idx])      # from the GPU's own bf16 h: one stage at a time
    _check_close(to_f64(y[idx]), y_ref, atol=2e-3)


def test_layer_full_size_sampled_segments():
    """The bench's ViT-L layer microbatch through mpipe_encoder_layer_fwd; attention is block-diagonal, so the rows of
    any image depend on that image alone: the oracle recomputes the three shortest images and compares those rows."""
    w = W.vit_l()
    H, D = w.n_heads, w.head_dim
    hidden, ffn, T = H * D, 4 * H * D, w.total_tokens
    pb = W.layer_params_bf16(31, hidden, ffn)
    x = W.normal_bf16(31, 0, (T, hidden))
    plan = B.seg_plan(w.patch_counts, B.FROZEN).to_device()
    weights = B.LayerWeights.from_tensors(**{k: to_dev(v) for k, v in pb.items()})
    y = torch.empty((T, hidden), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(B.encoder_layer_workspace_bytes(T, hidden, ffn), dtype=torch.uint8, device="cuda")
    st = status_buf()
    B.encoder_layer_fwd(to_dev(x), y, weights, H, ffn, plan, w.softmax_scale, 1e-6, ws, None, st)
    torch.cuda.synchronize()
    assert st.cpu().tolist()[0] == 0
    ow = OL.LayerWeights(g1=OL.widen(pb["ln1_gamma"]), b1=OL.widen(pb["ln1_beta"]), wqkv=OL.widen(pb["w_qkv"]),
                         bqkv=OL.widen(pb["b_qkv"]), wo=OL.widen(pb["w_o"]), bo=OL.widen(pb["b_o"]),
                         g2=OL.widen(pb["ln2_gamma"]), b2=OL.widen(pb["ln2_beta"]), w1=OL.widen(pb["w_fc1"]),
                         bb1=OL.widen(pb["b_fc1"]), w2=OL.widen(pb["w_fc2"]), bb2=OL.widen(pb["b_fc2"]))
    got = to_f64(y)
    cu = w.cu_seqlens
    for seg in np.argsort(w.patch_counts)[:3]:
        lo, hi = int(cu[seg]), int(cu[seg + 1])
        ref, _ = OL.encoder_layer_fwd(x[lo:hi], ow, np.array([0, hi - lo], dtype=np.int32), H, w.softmax_scale, 1e-6)
        assert rel_l2(got[lo:hi], ref) <= LAYER_REL_L2, (seg, rel_l2(got[lo:hi], ref))


@pytest.mark.parametrize("M,N,K", [(1, 8, 8), (300, 72, 264), (257, 1024, 512), (1000, 1280, 1024), (129, 64, 3072)])
@pytest.mark.parametrize("gelu_in,res", [(False, False), (True, False), (False, True)])
def test_linear_dgrad_matches_oracle(M, N, K, gelu_in, res):
    dy = W.normal_bf16(15, 0, (M, N))
    w = W.scaled_normal_bf16(15, 1, (N, K), std=N ** -0.5)
    u = W.normal_bf16(15, 2, (M, K)) if gelu_in else None
    r = W.normal_bf16(15, 3, (M, K)) if res else None
    dx = torch.full((M, K), 7.0, dtype=torch.bfloat16, device="cuda")
    st = status_buf()
    B.linear_dgrad(to_dev(dy), to_dev(w), dx, None if u is None else to_dev(u), None if r is None else to_dev(r), st)
    torch.cuda.synchronize()
    assert st.cpu().tolist()[0] == 0
    ref = OL.linear_dgrad(OL.widen(dy), OL.widen(w))
    if gelu_in:
        ref = ref * OL.gelu_grad(OL.widen(u))
    if res:
        ref = ref + OL.widen(r)
    _check_close(to_f64(dx), ref, atol=2e-3)


@pytest.mark.parametrize("T,N,K", [(1, 8, 8), (300, 72, 264), (5000, 1024, 512), (777, 136, 1024), (20000, 256, 256)])
def test_linear_wgrad_matches_oracle_and_accumulates(T, N, K):
    dy = W.normal_bf16(16, 0, (T, N))
    x = W.normal_bf16(16, 1, (T, K))
    dw = torch.full((N, K), 0.5, dtype=torch.float32, device="cuda")      # accumulates on top of what is there
    st = status_buf()
    B.linear_wgrad(to_dev(dy), to_dev(x), dw, st)
    torch.cuda.synchronize()
    assert st.cpu().tolist()[0] == 0
    ref, _ = OL.linear_wgrad(OL.widen(dy), OL.widen(x))
    got = dw.cpu().double().numpy() - 0.5
    # fp32 accumulation of T exact bf16 products per element
    assert np.abs(got - ref).max() <= 1e-5 * max(1.0, np.abs(ref).max()) + 4e-7 * T ** 0.5 * 16


@pytest.mark.parametrize("T,hidden", [(1, 8), (37, 256), (3000, 1024), (513, 1280), (9, 2048)])
@pytest.mark.parametrize("with_res", [False, True])
def test_layernorm_bwd_matches_oracle(T, hidden, with_res):
    x = W.scaled_normal_bf16(17, 0, (T, hidden), std=2.0, mean=0.7)
    dy = W.normal_bf16(17, 1, (T, hidden))
    g = W.scaled_normal_bf16(17, 2, (hidden,), std=0.1, mean=1.0)
    r = W.normal_bf16(17, 3, (T, hidden)) if with_res else None
    dx = torch.empty((T, hidden), dtype=torch.bfloat16, device="cuda")
    dg = torch.full((hidden,), 0.25, dtype=torch.float32, device="cuda")
    db = torch.full((hidden,), -0.5, dtype=torch.float32, device="cuda")
    B.layernorm_bwd(to_dev(x), to_dev(dy), to_dev(g), dx, dg, db, 1e-6, None if r is None else to_dev(r))
    torch.cuda.synchronize()
    dx_ref, dg_ref, db_ref = OL.layernorm_bwd(OL.widen(x), OL.widen(dy), OL.widen(g), 1e-6)
    if with_res:
        dx_ref = dx_ref + OL.widen(r)
    _check_close(to_f64(dx), dx_ref, atol=2e-4)
    tol = 1e-5 * max(1.0, np.abs(dg_ref).max()) + 2e-6 * T ** 0.5 * 8
    assert np.abs(dg.cpu().double().numpy() - 0.25 - dg_ref).max() <= tol
    assert np.abs(db.cpu().double().numpy() + 0.5 - db_ref).max() <= tol


@pytest.mark.parametrize("T,N", [(1, 8), (777, 264), (20000, 3072)])
def test_colsum_matches_oracle(T, N):
    a = W.normal_bf16(18, 0, (T, N))
    out = torch.full((N,), 2.0, dtype=torch.float32, device="cuda")
    B.colsum_accumulate(to_dev(a), out)
    torch.cuda.synchronize()
    ref = OL.widen(a).sum(axis=0)
    assert np.abs(out.cpu().double().numpy() - 2.0 - ref).max() <= 1e-5 * max(1.0, np.abs(ref).max()) + 1e-6 * T ** 0.5 * 8


def test_rope_bwd_is_the_transpose_of_rope():
    counts, H, D = [300, 77], 3, 80
    T, hidden = sum(counts), H * D
    g = W.normal_bf16(19, 0, (T, 3 * hidden))
    cos, sin = W.rope2d_tables(counts, D)
    dev = to_dev(g)
    B.rope_apply_bwd(dev, torch.from_numpy(cos).cuda(), torch.from_numpy(sin).cuda(), H, D)
    torch.cuda.synchronize()
    ref = OL.widen(g).copy()
    for i in range(2):   # the transpose of a rotation is the rotation by the opposite angle
        blk = ref[:, i * hidden:(i + 1) * hidden].reshape(T, H, D)
        ref[:, i * hidden:(i + 1) * hidden] = OL.rope(blk, cos.astype(np.float64), -sin.astype(np.float64)).reshape(T, hidden)
    _check_close(to_f64(dev), ref, atol=1e-6)


GRAD_REL_L2 = 1.5e-2    # the backward chains ~10 bf16-rounded stages (recomputed activations included)


@pytest.mark.parametrize("counts,H,D,ffn,rope", [([16, 49, 64, 100], 4, 64, 1024, False), ([300, 1, 129, 640], 4, 80, 1280, True),
                                                  ([1024, 256, 777], 16, 64, 4096, False)])
def test_layer_bwd_matches_oracle(counts, H, D, ffn, rope):
    hidden, T = H * D, sum(counts)
    pb = W.layer_params_bf16(23, hidden, ffn)
    x, dy = W.normal_bf16(23, 0, (T, hidden)), W.normal_bf16(23, 1, (T, hidden))
    plan = B.seg_plan(counts, B.TRAINED).to_device()
    weights = B.LayerWeights.from_tensors(**{k: to_dev(v) for k, v in pb.items()})
    grads_t = {k: torch.zeros(v.shape, dtype=torch.float32, device="cuda") for k, v in pb.items()}
    grads = B.LayerGrads.from_tensors(**grads_t)
    xd, dyd = to_dev(x), to_dev(dy)
    y, dx = torch.empty_like(xd), torch.empty_like(xd)
    lse = torch.empty((H, T), dtype=torch.float32, device="cuda")
    ws_f = torch.empty(B.encoder_layer_workspace_bytes(T, hidden, ffn), dtype=torch.uint8, device="cuda")
    ws_b = torch.empty(B.encoder_layer_bwd_workspace_bytes(T, hidden, H, ffn), dtype=torch.uint8, device="cuda")
    st = status_buf()
    scale = float(np.float32(1 / math.sqrt(D)))
    tabs = W.rope2d_tables(counts, D) if rope else None
    rope_dev = None if tabs is None else tuple(torch.from_numpy(t).cuda() for t in tabs)
    B.encoder_layer_fwd(xd, y, weights, H, ffn, plan, scale, 1e-6, ws_f, lse, st, rope=rope_dev)
    for _ in range(2):      # two microbatches: parameter gradients accumulate, dx is overwritten
        B.encoder_layer_bwd(dyd, xd, dx, weights, grads, H, ffn, plan, scale, 1e-6, lse, ws_f, ws_b, st, rope=rope_dev)
    torch.cuda.synchronize()
    assert st.cpu().tolist()[0] == 0
    ow = OL.LayerWeights(g1=OL.widen(pb["ln1_gamma"]), b1=OL.widen(pb["ln1_beta"]), wqkv=OL.widen(pb["w_qkv"]),
                         bqkv=OL.widen(pb["b_qkv"]), wo=OL.widen(pb["w_o"]), bo=OL.widen(pb["b_o"]),
                         g2=OL.widen(pb["ln2_gamma"]), b2=OL.widen(pb["ln2_beta"]), w1=OL.widen(pb["w_fc1"]),
                         bb1=OL.widen(pb["b_fc1"]), w2=OL.widen(pb["w_fc2"]), bb2=OL.widen(pb["b_fc2"]))
    cu = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    dx_ref, g_ref = OL.encoder_layer_bwd(x, ow, cu, H, scale, 1e-6, dy,
                                         None if tabs is None else tuple(t.astype(np.float64) for t in tabs))
    assert rel_l2(to_f64(dx), dx_ref) <= GRAD_REL_L2, rel_l2(to_f64(dx), dx_ref)
    for name, ref in g_ref.items():
        got = grads_t[name].cpu().double().numpy() / 2.0
        assert rel_l2(got, ref.reshape(got.shape)) <= GRAD_REL_L2, (name, rel_l2(got, ref.reshape(got.shape)))


def test_layer_bwd_frozen_is_a_no_op():
    T, hidden, ffn, H = 64, 256, 512, 4
    pb = W.layer_params_bf16(5, hidden, ffn)
    weights = B.LayerWeights.from_tensors(**{k: to_dev(v) for k, v in pb.items()})
    grads_t = {k: torch.full(v.shape, 3.0, dtype=torch.float32, device="cuda") for k, v in pb.items()}
    grads = B.LayerGrads.from_tensors(**grads_t)
    x = to_dev(W.normal_bf16(5, 0, (T, hidden)))
    dx = torch.full_like(x, 7.0)
    plan = B.seg_plan([T], B.FROZEN).to_device()
    B.encoder_layer_bwd(x, x, dx, weights, grads, H, ffn, plan, 0.125, 1e-6, None, None, None)   # nothing else is needed
    torch.cuda.synchronize()
    assert (dx == 7.0).all() and all((g == 3.0).all() for g in grads_t.values())


def test_layer_bwd_full_size_sampled_segments():
    """The bench's ViT-L microbatch through forward + backward; the input gradient of an image's rows depends on that image
    alone (block-diagonal attention, row-wise everything else), so the oracle recomputes the two shortest images' dx."""
    w = W.vit_l()
    H, D = w.n_heads, w.head_dim
    hidden, ffn, T = H * D, 4 * H * D, w.total_tokens
    pb = W.layer_params_bf16(33, hidden, ffn)
    x, dy = W.normal_bf16(33, 0, (T, hidden)), W.normal_bf16(33, 1, (T, hidden))
    plan = B.seg_plan(w.patch_counts, B.TRAINED).to_device()
    weights = B.LayerWeights.from_tensors(**{k: to_dev(v) for k, v in pb.items()})
    grads_t = {k: torch.zeros(v.shape, dtype=torch.float32, device="cuda") for k, v in pb.items()}
    grads = B.LayerGrads.from_tensors(**grads_t)
    xd, dyd = to_dev(x), to_dev(dy)
    y, dx = torch.empty_like(xd), torch.empty_like(xd)
    lse = torch.empty((H, T), dtype=torch.float32, device="cuda")
    ws_f = torch.empty(B.encoder_layer_workspace_bytes(T, hidden, ffn), dtype=torch.uint8, device="cuda")
    ws_b = torch.empty(B.encoder_layer_bwd_workspace_bytes(T, hidden, H, ffn), dtype=torch.uint8, device="cuda")
    st = status_buf()
    B.encoder_layer_fwd(xd, y, weights, H, ffn, plan, w.softmax_scale, 1e-6, ws_f, lse, st)
    B.encoder_layer_bwd(dyd, xd, dx, weights, grads, H, ffn, plan, w.softmax_scale, 1e-6, lse, ws_f, ws_b, st)
    torch.cuda.synchronize()
    assert st.cpu().tolist()[0] == 0
    ow = OL.LayerWeights(g1=OL.widen(pb["ln1_gamma"]), b1=OL.widen(pb["ln1_beta"]), wqkv=OL.widen(pb["w_qkv"]),
                         bqkv=OL.widen(pb["b_qkv"]), wo=OL.widen(pb["w_o"]), bo=OL.widen(pb["b_o"]),
                         g2=OL.widen(pb["ln2_gamma"]), b2=OL.widen(pb["ln2_beta"]), w1=OL.widen(pb["w_fc1"]),
                         bb1=OL.widen(pb["b_fc1"]), w2=OL.widen(pb["w_fc2"]), bb2=OL.widen(pb["b_fc2"]))
    got = to_f64(dx)
    cu = w.cu_seqlens
    for seg in np.argsort(w.patch_counts)[:2]:
        lo, hi = int(cu[seg]), int(cu[seg + 1])
        ref, _ = OL.encoder_layer_bwd(x[lo:hi], ow, np.array([0, hi - lo], dtype=np.int32), H, w.softmax_scale, 1e-6, dy[lo:hi])
        assert rel_l2(got[lo:hi], ref) <= GRAD_REL_L2, (seg, rel_l2(got[lo:hi], ref))
    # the bias gradient of the last projection is the plain column sum of dy: an exact, full-size check of the accumulation
    ref_b = OL.widen(dy).sum(axis=0)
    assert np.abs(grads_t["b_fc2"].cpu().double().numpy() - ref_b).max() <= 1e-5 * np.abs(ref_b).max() + 1e-3


def test_encoder_stack_matches_oracle():
    """Three layers through mpipe_encoder_fwd / mpipe_encoder_bwd against the oracle's layer applied three times."""
    counts, H, D, ffn, L = [300, 1, 129], 4, 64, 512, 3
    hidden, T = H * D, sum(counts)
    pbs = [W.layer_params_bf16(40 + l, hidden, ffn) for l in range(L)]
    x, dy = W.normal_bf16(40, 0, (T, hidden)), W.normal_bf16(40, 1, (T, hidden))
    plan = B.seg_plan(counts, B.TRAINED).to_device()
    layers = [B.LayerWeights.from_tensors(**{k: to_dev(v) for k, v in pb.items()}) for pb in pbs]
    grads_t = [{k: torch.zeros(v.shape, dtype=torch.float32, device="cuda") for k, v in pb.items()} for pb in pbs]
    grads = [B.LayerGrads.from_tensors(**g) for g in grads_t]
    xd, dyd = to_dev(x), to_dev(dy)
    y, dx = torch.empty_like(xd), torch.empty_like(xd)
    lse = torch.empty((L, H, T), dtype=torch.float32, device="cuda")
    ws_f = torch.empty(B.encoder_workspace_bytes(L, T, hidden, ffn, B.TRAINED), dtype=torch.uint8, device="cuda")
    ws_b = torch.empty(B.encoder_bwd_workspace_bytes(T, hidden, H, ffn), dtype=torch.uint8, device="cuda")
    st = status_buf()
    scale = 0.125
    B.encoder_fwd(xd, y, layers, H, ffn, plan, scale, 1e-6, ws_f, lse, st)
    B.encoder_bwd(dyd, xd, dx, layers, grads, H, ffn, plan, scale, 1e-6, lse, ws_f, ws_b, st)
    torch.cuda.synchronize()
    assert st.cpu().tolist()[0] == 0
    # frozen stack: same forward result to bf16 rounding, through the small reused workspace
    plan_f = B.seg_plan(counts, B.FROZEN).to_device()
    y_f = torch.empty_like(xd)
    ws_small = torch.empty(B.encoder_workspace_bytes(L, T, hidden, ffn, B.FROZEN), dtype=torch.uint8, device="cuda")
    B.encoder_fwd(xd, y_f, layers, H, ffn, plan_f, scale, 1e-6, ws_small, None, st)
    torch.cuda.synchronize()
    cu = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    ows = [OL.LayerWeights(g1=OL.widen(pb["ln1_gamma"]), b1=OL.widen(pb["ln1_beta"]), wqkv=OL.widen(pb["w_qkv"]),
                           bqkv=OL.widen(pb["b_qkv"]), wo=OL.widen(pb["w_o"]), bo=OL.widen(pb["b_o"]),
                           g2=OL.widen(pb["ln2_gamma"]), b2=OL.widen(pb["ln2_beta"]), w1=OL.widen(pb["w_fc1"]),
                           bb1=OL.widen(pb["b_fc1"]), w2=OL.widen(pb["w_fc2"]), bb2=OL.widen(pb["b_fc2"])) for pb in pbs]
    acts = [OL.widen(x)]
    for ow in ows:
        acts.append(OL.encoder_layer_fwd(acts[-1], ow, cu, H, scale, 1e-6)[0])
    assert rel_l2(to_f64(y), acts[-1]) <= 2e-2 and rel_l2(to_f64(y_f), acts[-1]) <= 2e-2
    g = OL.widen(dy)
    for l in range(L - 1, -1, -1):
        g, pg = OL.encoder_layer_bwd(acts[l], ows[l], cu, H, scale, 1e-6, g)
        for name, ref in pg.items():
            got = grads_t[l][name].cpu().double().numpy()
            assert rel_l2(got, ref.reshape(got.shape)) <= 3e-2, (l, name, rel_l2(got, ref.reshape(got.shape)))
    assert rel_l2(to_f64(dx), g) <= 3e-2
