"""CPU-side checks of the C ABI: the library loads, exports what the header declares, the planner is
bit-exact against the oracle's restatement, and argument errors are caught before any launch."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
from paper_2607_03229_b200 import binding as B
from paper_2607_03229_b200 import build as build_mod
from paper_2607_03229_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_mod.build()


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "mpipe_enc.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(mpipe_[a-z_0-9]+)\s*\(", header))
    assert {"mpipe_seg_plan", "mpipe_varlen_attn_fwd", "mpipe_varlen_attn_bwd", "mpipe_merge_tokens"} <= declared
    lib = ctypes.CDLL(B.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(B.EXPORTED_SYMBOLS)
    assert B.version() >= 100 and B.status_str(0) == "ok"
    assert B.fwd_tile_rows() % 128 == 0 and B.bwd_tile_rows() == 128


def _items_as_tuples(items):
    return [tuple(int(x) for x in it) for it in items]


@pytest.mark.parametrize("mode", [B.FROZEN, B.TRAINED])
def test_plan_bit_exact_against_oracle(mode):
    rng = np.random.default_rng(3)
    cases = [[], [0], [0, 0, 5], [1], [128], [129], [256, 256, 257]]
    cases += [list(rng.integers(0, 1500, size=int(rng.integers(1, 40)))) for _ in range(30)]
    cases += [W.tiny().patch_counts, W.vit_l().patch_counts, W.qwen2vl().patch_counts, W.video_tail().patch_counts]
    cases += [W.modality_mix(f).patch_counts for f in W.MIX_FRACTIONS]
    for counts in cases:
        for fr, br in ((B.fwd_tile_rows(), B.bwd_tile_rows()), (64, 192)):
            plan = B.seg_plan(counts, mode, fr, br)
            cu, T, mx, fwd, bwd = oracle.seg_plan(counts, fr, br, mode == B.TRAINED)
            assert plan.cu_seqlens.tolist() == cu and plan.total_tokens == T and plan.max_seqlen == mx
            assert _items_as_tuples(plan.fwd_items) == fwd
            assert _items_as_tuples(plan.bwd_items) == bwd


def test_plan_rejects_bad_arguments():
    with pytest.raises(B.MpipeError) as e:
        B.seg_plan([4, -1], B.TRAINED)
    assert e.value.status == B.ERR_INVALID_ARG
    with pytest.raises(B.MpipeError):
        B.seg_plan([4], 7)
    with pytest.raises(B.MpipeError):
        B.seg_plan([4], B.TRAINED, 0, 128)
    with pytest.raises(B.MpipeError):
        B.seg_plan([2 ** 30, 2 ** 30], B.TRAINED)


def test_validate_positions():
    assert B.validate_positions([3, 1, 2], 4) == B.OK
    assert B.validate_positions([], 4) == B.OK
    assert B.validate_positions([3, 4], 4) == B.ERR_INDEX
    assert B.validate_positions([-1], 4) == B.ERR_INDEX
    assert B.validate_positions([1, 1], 4) == B.ERR_INVALID_ARG
    for f in W.MIX_FRACTIONS:
        m = W.modality_mix(f)
        assert B.validate_positions(m.positions, m.n_llm_tokens) == B.OK


def test_device_calls_validate_on_the_host_before_launching():
    """No GPU here: every one of these must return from the host-side checks."""
    lib = B.load()
    fake = 0x1000  # 16-byte aligned, never dereferenced on the host
    # empty work: OK without a launch
    assert lib.mpipe_varlen_attn_fwd(None, None, None, None, None, 1024, 64, 1024, 64, None, 0, 0, 0, None, 0, 16, 64,
                                     0.125, B.TRAINED, None, None) == B.OK
    assert lib.mpipe_merge_tokens(None, 256, None, 256, None, 0, 512, 256, B.TRAINED, None, None) == B.OK
    # frozen backward: nothing to do, whatever the pointers
    assert lib.mpipe_varlen_attn_bwd(*([None] * 9), 0, 0, 0, 0, 0, 0, None, 0, 0, 0, None, 0, 16, 64, 0.125, B.FROZEN,
                                     None, 0, None, None) == B.OK
    assert lib.mpipe_merge_tokens_bwd(None, 256, None, 256, None, 5, 512, 256, B.FROZEN, None, None) == B.OK
    # unsupported head_dim, misaligned pointer, bad stride, missing LSE in trained mode
    common = dict(ts=1024, hs=64)
    def fwd(q=fake, hd=64, ts=1024, hs=64, lse=fake, mode=B.TRAINED, scale=0.125):
        return lib.mpipe_varlen_attn_fwd(q, fake, fake, fake, lse, ts, hs, ts, hs, fake, 1, 100, 100, fake, 1, 16, hd,
                                         scale, mode, None, None)
    assert fwd(hd=128) == B.ERR_UNSUPPORTED
    assert fwd(q=fake + 2) == B.ERR_INVALID_ARG
    assert fwd(ts=1020) == B.ERR_INVALID_ARG
    assert fwd(lse=None) == B.ERR_INVALID_ARG
    assert fwd(mode=3) == B.ERR_INVALID_ARG
    assert fwd(scale=0.0) == B.ERR_INVALID_ARG
    # merge: hidden not a multiple of 8, misaligned base
    assert lib.mpipe_merge_tokens(fake, 260, fake, 260, fake, 4, 8, 260, B.TRAINED, None, None) == B.ERR_INVALID_ARG
    assert lib.mpipe_merge_tokens(fake + 4, 256, fake, 256, fake, 4, 8, 256, B.TRAINED, None, None) == B.ERR_INVALID_ARG
    assert B.attn_workspace_bytes(1000, 16, 64, B.FROZEN) == 0
    assert B.attn_workspace_bytes(1000, 16, 64, B.TRAINED) >= 1000 * 16 * 65 * 4
