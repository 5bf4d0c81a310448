"""GPU parity of mpipe_merge_tokens / mpipe_merge_tokens_bwd against the oracle: bit-exact."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_03229_b200 import binding as B
from paper_2607_03229_b200 import workloads as W
from _util import status_buf, to_bits, to_dev

pytestmark = pytest.mark.gpu


def _run_merge(enc_bits, emb_bits, pos, pad_rows=3):
    """Merge on the GPU with canary rows around the embedding buffer; returns the merged bits."""
    n_llm, hidden = emb_bits.shape
    canary = np.full((pad_rows, hidden), 0xDEAD, dtype=np.uint16)
    buf = to_dev(np.concatenate([canary, emb_bits, canary]))
    emb = buf[pad_rows:pad_rows + n_llm]
    st = status_buf()
    B.merge_tokens(to_dev(enc_bits), emb, torch.from_numpy(pos).cuda(), B.TRAINED, st)
    torch.cuda.synchronize()
    out = to_bits(buf)
    assert np.all(out[:pad_rows] == 0xDEAD) and np.all(out[-pad_rows:] == 0xDEAD), "canary rows overwritten"
    return out[pad_rows:-pad_rows], st.cpu().numpy()


@pytest.mark.parametrize("shuffled", [False, True])
def test_tiny_merge(shuffled):
    w = W.tiny(shuffled_positions=shuffled)
    enc, emb = w.merge_source(), w.llm_embeds()
    got, st = _run_merge(enc, emb, w.positions)
    assert st[0] == 0
    assert np.array_equal(got, oracle.merge_tokens(enc, emb, w.positions))


@pytest.mark.parametrize("hidden,n_llm,n_enc", [(8, 5, 5), (24, 100, 37), (4096, 300, 111), (1280, 2049, 1000)])
def test_ragged_shapes(hidden, n_llm, n_enc):
    enc = W.normal_bf16(5, 1, (n_enc, hidden))
    emb = W.normal_bf16(5, 2, (n_llm, hidden))
    pos = np.argsort(W.rand_u64(5, 3, n_llm), kind="stable")[:n_enc].astype(np.int32)
    got, st = _run_merge(enc, emb, pos)
    assert st[0] == 0 and np.array_equal(got, oracle.merge_tokens(enc, emb, pos))


def test_empty_and_identity():
    emb = W.normal_bf16(6, 2, (16, 64))
    got, st = _run_merge(np.zeros((0, 64), np.uint16), emb, np.zeros((0,), np.int32))
    assert np.array_equal(got, emb)
    enc = W.normal_bf16(6, 1, (16, 64))
    got, _ = _run_merge(enc, emb, np.arange(16, dtype=np.int32))
    assert np.array_equal(got, enc)


def test_strided_rows():
    """Source and destination rows with a row stride larger than hidden."""
    enc_full = to_dev(W.normal_bf16(7, 1, (50, 512)))
    emb_full = to_dev(W.normal_bf16(7, 2, (80, 768)))
    enc, emb = enc_full[:, 128:384], emb_full[:, 256:512]
    pos = np.argsort(W.rand_u64(7, 3, 80), kind="stable")[:50].astype(np.int32)
    ref = oracle.merge_tokens(to_bits(enc), to_bits(emb), pos)
    before = to_bits(emb_full).copy()
    B.merge_tokens(enc, emb, torch.from_numpy(pos).cuda())
    torch.cuda.synchronize()
    after = to_bits(emb_full)
    assert np.array_equal(after[:, 256:512], ref)
    assert np.array_equal(after[:, :256], before[:, :256]) and np.array_equal(after[:, 512:], before[:, 512:])


def test_out_of_range_position_is_skipped_and_flagged():
    enc = W.normal_bf16(8, 1, (4, 64))
    emb = W.normal_bf16(8, 2, (10, 64))
    pos = np.array([2, 10, 7, -1], dtype=np.int32)
    got, st = _run_merge(enc, emb, pos)
    assert st[0] == B.ERR_INDEX and st[1] in (1, 3)
    ref = emb.copy()
    ref[2], ref[7] = enc[0], enc[2]
    assert np.array_equal(got, ref)


@pytest.mark.parametrize("fraction", W.MIX_FRACTIONS)
def test_modality_mix_merge_full_size(fraction):
    """The benchmark's merge: 8 x 8192 LLM tokens at hidden 4096, every element compared."""
    w = W.modality_mix(fraction)
    enc = w.merge_source()
    emb = w.llm_embeds()
    emb_d = to_dev(emb)
    st = status_buf()
    B.merge_tokens(to_dev(enc), emb_d, torch.from_numpy(w.positions).cuda(), B.TRAINED, st)
    torch.cuda.synchronize()
    assert int(st[0]) == 0
    assert np.array_equal(to_bits(emb_d), oracle.merge_tokens(enc, emb, w.positions))


def test_merge_bwd_gathers_rows_and_frozen_is_a_noop():
    w = W.tiny(shuffled_positions=True)
    d_emb = W.normal_bf16(9, 1, (512, 256))
    pos_d = torch.from_numpy(w.positions).cuda()
    d_enc = torch.full((229, 256), 7.0, dtype=torch.bfloat16, device="cuda")
    B.merge_tokens_bwd(to_dev(d_emb), d_enc, pos_d, B.FROZEN)
    torch.cuda.synchronize()
    assert torch.all(d_enc == 7.0)  # frozen encoder: the reverse seam does not exist
    B.merge_tokens_bwd(to_dev(d_emb), d_enc, pos_d, B.TRAINED)
    torch.cuda.synchronize()
    assert np.array_equal(to_bits(d_enc), oracle.merge_tokens_bwd(d_emb, w.positions))


@pytest.mark.parametrize("hidden,n_llm,n_enc", [(8, 5, 5), (24, 100, 37), (4096, 300, 111), (1280, 2049, 1000)])
def test_merge_bwd_ragged_shapes(hidden, n_llm, n_enc):
    d_emb = W.normal_bf16(15, 2, (n_llm, hidden))
    pos = np.argsort(W.rand_u64(15, 3, n_llm), kind="stable")[:n_enc].astype(np.int32)
    pad = 3
    buf = torch.full((n_enc + 2 * pad, hidden), 7.0, dtype=torch.bfloat16, device="cuda")
    st = status_buf()
    B.merge_tokens_bwd(to_dev(d_emb), buf[pad:pad + n_enc], torch.from_numpy(pos).cuda(), B.TRAINED, st)
    torch.cuda.synchronize()
    assert int(st[0]) == 0
    assert torch.all(buf[:pad] == 7.0) and torch.all(buf[pad + n_enc:] == 7.0), "canary rows overwritten"
    assert np.array_equal(to_bits(buf[pad:pad + n_enc]), oracle.merge_tokens_bwd(d_emb, pos))


def test_merge_bwd_strided_rows():
    """Gradient rows read from, and written into, column blocks of wider buffers."""
    d_emb_full = to_dev(W.normal_bf16(16, 2, (80, 768)))
    d_enc_full = torch.full((50, 512), 7.0, dtype=torch.bfloat16, device="cuda")
    d_emb, d_enc = d_emb_full[:, 256:512], d_enc_full[:, 128:384]
    pos = np.argsort(W.rand_u64(16, 3, 80), kind="stable")[:50].astype(np.int32)
    B.merge_tokens_bwd(d_emb, d_enc, torch.from_numpy(pos).cuda(), B.TRAINED)
    torch.cuda.synchronize()
    assert np.array_equal(to_bits(d_enc), oracle.merge_tokens_bwd(to_bits(d_emb), pos))
    assert torch.all(d_enc_full[:, :128] == 7.0) and torch.all(d_enc_full[:, 384:] == 7.0)


def test_merge_bwd_out_of_range_position_is_skipped_and_flagged():
    d_emb = W.normal_bf16(17, 2, (10, 64))
    pos = np.array([2, 10, 7, -1], dtype=np.int32)
    d_enc = torch.full((4, 64), 7.0, dtype=torch.bfloat16, device="cuda")
    st = status_buf()
    B.merge_tokens_bwd(to_dev(d_emb), d_enc, torch.from_numpy(pos).cuda(), B.TRAINED, st)
    torch.cuda.synchronize()
    st = st.cpu().numpy()
    assert st[0] == B.ERR_INDEX and st[1] in (1, 3)
    got = to_bits(d_enc)
    assert np.array_equal(got[0], d_emb[2]) and np.array_equal(got[2], d_emb[7])
    assert torch.all(d_enc[1] == 7.0) and torch.all(d_enc[3] == 7.0)      # rows with no valid source stay untouched


@pytest.mark.parametrize("fraction", [0.25, 0.75])
def test_merge_bwd_modality_mix_full_size(fraction):
    """The reverse seam at benchmark size: gradient rows of 8 x 8192 LLM tokens at hidden 4096 gathered back."""
    w = W.modality_mix(fraction)
    d_emb = w.llm_embeds()          # any bf16 matrix of the right shape stands for dL/d(embeddings)
    d_enc = torch.empty((w.total_tokens, 4096), dtype=torch.bfloat16, device="cuda")
    st = status_buf()
    B.merge_tokens_bwd(to_dev(d_emb), d_enc, torch.from_numpy(w.positions).cuda(), B.TRAINED, st)
    torch.cuda.synchronize()
    assert int(st[0]) == 0
    assert np.array_equal(to_bits(d_enc), oracle.merge_tokens_bwd(d_emb, w.positions))
