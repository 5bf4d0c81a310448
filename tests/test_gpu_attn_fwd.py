"""GPU parity of mpipe_varlen_attn_fwd against the fp64 oracle (element by element on small and
ragged cases; the benchmark sizes are in test_gpu_configs.py) plus the schedule-level properties the paper
states: freezing changes no forward bit (Corollary 1) and relocation changes no result."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_03229_b200 import binding as B
from paper_2607_03229_b200 import workloads as W
from _util import LSE_MAX_ABS, O_MAX_ABS, O_REL_L2, max_abs, rel_l2, status_buf, to_dev, to_f64

pytestmark = pytest.mark.gpu


def gpu_fwd(q, k, v, counts, scale, mode=B.TRAINED, canary=True):
    """Run the forward on bf16 bit arrays; returns (O bf16 tensor, LSE fp32 tensor or None, plan)."""
    T, H, D = q.shape
    plan = B.seg_plan(counts, mode).to_device()
    qd, kd, vd = to_dev(q), to_dev(k), to_dev(v)
    pad = 2 if canary else 0
    obuf = torch.full((T + 2 * pad, H, D), 777.0, dtype=torch.bfloat16, device="cuda")
    o = obuf[pad:pad + T]
    lse = torch.full((H, T), -555.0, dtype=torch.float32, device="cuda") if mode == B.TRAINED else None
    st = status_buf()
    B.varlen_attn_fwd(qd, kd, vd, o, lse, plan, scale, st)
    torch.cuda.synchronize()
    assert st.cpu().tolist()[0] == 0, f"device status {st.cpu().tolist()}"
    if canary:
        assert torch.all(obuf[:pad] == 777.0) and torch.all(obuf[pad + T:] == 777.0), "canary rows overwritten"
    return o, lse, plan


def check_fwd(counts, H, D, seed, scale=None):
    T = int(sum(counts))
    q, k, v = (W.normal_bf16(seed, s, (T, H, D)) for s in (1, 2, 3))
    scale = float(np.float32(1.0 / np.sqrt(D))) if scale is None else scale
    o, lse, _ = gpu_fwd(q, k, v, counts, scale)
    cu = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    O_ref, L_ref = oracle.attn_fwd(q, k, v, cu, scale)
    O = to_f64(o)
    assert not np.isnan(O).any()
    ma, rl = max_abs(O, O_ref), rel_l2(O, O_ref)
    la = max_abs(to_f64(lse), L_ref)
    assert ma <= O_MAX_ABS and rl <= O_REL_L2, (counts, ma, rl)
    assert la <= LSE_MAX_ABS, (counts, la)
    return ma, rl, la


def test_tiny_config():
    w = W.tiny()
    check_fwd(w.patch_counts, w.n_heads, w.head_dim, w.seed, w.softmax_scale)


@pytest.mark.parametrize("D", [64, 80])
@pytest.mark.parametrize("counts", [
    [1], [16], [127], [128], [129], [255], [256], [257], [384], [385], [700],
    [1, 5, 0, 127, 128, 129, 0, 255, 256, 257, 300, 513],
    [1040, 3, 260],
])
def test_ragged_segments(counts, D):
    check_fwd(counts, 2, D, seed=100 + sum(counts) + D)


@pytest.mark.parametrize("D", [64, 80])
def test_many_units_per_cta(D):
    """More (item, head) units than SMs, so every CTA loops over several units and ring phases wrap."""
    counts = [int(x) for x in W.rand_int(17, 1, 24, 40, 900)]
    check_fwd(counts, 8, D, seed=17)


def test_large_scores_trigger_rescale():
    """A large softmax scale makes row maxima jump by far more than the lazy-rescale threshold.
    The softmax is then nearly one-hot and |O| reaches 4 and more: the bf16 rounding of the one dominant
    probability (2^-9 relative) and of the output (2^-9 relative) both scale with |O| and alone exceed
    the absolute bar there, so the absolute check scales with |O|."""
    counts, H, D, scale = [700, 300], 2, 64, 1.5
    q, k, v = (W.normal_bf16(23, s, (1000, H, D)) for s in (1, 2, 3))
    o, lse, _ = gpu_fwd(q, k, v, counts, scale)
    O_ref, L_ref = oracle.attn_fwd(q, k, v, np.array([0, 700, 1000], dtype=np.int32), scale)
    O = to_f64(o)
    assert rel_l2(O, O_ref) <= O_REL_L2
    assert np.all(np.abs(O - O_ref) <= 5e-3 + 2.0 ** -7 * np.abs(O_ref))
    assert max_abs(to_f64(lse), L_ref) <= LSE_MAX_ABS


def test_frozen_and_trained_produce_identical_bits_and_frozen_writes_no_lse():
    w = W.tiny()
    q, k, v = w.qkv()
    o_t, lse_t, _ = gpu_fwd(q, k, v, w.patch_counts, w.softmax_scale, B.TRAINED)
    o_f, lse_f, plan_f = gpu_fwd(q, k, v, w.patch_counts, w.softmax_scale, B.FROZEN)
    assert lse_f is None and plan_f.bwd_items.size == 0
    assert torch.equal(o_t.view(torch.int16), o_f.view(torch.int16))
    o_2, lse_2, _ = gpu_fwd(q, k, v, w.patch_counts, w.softmax_scale, B.TRAINED)
    assert torch.equal(o_t.view(torch.int16), o_2.view(torch.int16)) and torch.equal(lse_t, lse_2)  # run to run


def test_relocation_invariance_packed_equals_per_image_and_segment_order():
    counts = [300, 41, 129]
    T, H, D = sum(counts), 4, 64
    q, k, v = (W.normal_bf16(31, s, (T, H, D)) for s in (1, 2, 3))
    scale = 0.125
    o, lse, _ = gpu_fwd(q, k, v, counts, scale)
    cu = np.concatenate([[0], np.cumsum(counts)])
    for s in range(3):
        a, b = cu[s], cu[s + 1]
        o_s, lse_s, _ = gpu_fwd(q[a:b], k[a:b], v[a:b], [counts[s]], scale)
        assert torch.equal(o_s.view(torch.int16), o[a:b].view(torch.int16))
        assert torch.equal(lse_s, lse[:, a:b])
    perm = np.concatenate([np.arange(cu[2], cu[3]), np.arange(cu[0], cu[1]), np.arange(cu[1], cu[2])])
    o_p, _, _ = gpu_fwd(q[perm], k[perm], v[perm], [counts[2], counts[0], counts[1]], scale)
    assert torch.equal(o_p.view(torch.int16), o[torch.from_numpy(perm).cuda()].view(torch.int16))


def test_segment_leak_detector():
    counts = [130, 257, 5, 128]
    T = sum(counts)
    q, k = (W.normal_bf16(37, s, (T, 2, 64)) for s in (1, 2))
    vals = np.zeros((T, 2, 64), dtype=np.float32)
    cu = np.concatenate([[0], np.cumsum(counts)])
    for s in range(4):
        vals[cu[s]:cu[s + 1]] = float(s + 1)
    o, _, _ = gpu_fwd(q, k, W.f32_to_bf16_bits(vals), counts, 0.125)
    assert np.abs(to_f64(o) - vals).max() <= 2.0 ** -6  # bf16 rounding of a weighted mean of one constant


def test_strided_qkv_from_a_packed_projection():
    """q, k, v as views of one [T, 3, H, D] buffer (token stride 3*H*D), output with its own strides."""
    counts = [200, 77]
    T, H, D = sum(counts), 4, 64
    qkv = W.normal_bf16(41, 1, (T, 3, H, D))
    qkv_d = to_dev(qkv)
    plan = B.seg_plan(counts, B.TRAINED).to_device()
    obuf = torch.zeros((T, H, 2 * D), dtype=torch.bfloat16, device="cuda")
    o = obuf[:, :, :D]
    lse = torch.zeros((H, T), dtype=torch.float32, device="cuda")
    st = status_buf()
    B.varlen_attn_fwd(qkv_d[:, 0], qkv_d[:, 1], qkv_d[:, 2], o, lse, plan, 0.125, st)
    torch.cuda.synchronize()
    assert int(st[0]) == 0
    O_ref, _ = oracle.attn_fwd(qkv[:, 0], qkv[:, 1], qkv[:, 2], plan.cu_seqlens, 0.125)
    assert rel_l2(to_f64(o), O_ref) <= O_REL_L2 and torch.all(obuf[:, :, D:] == 0)
