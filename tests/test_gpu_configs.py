"""Parity of the attention forward + backward at the five benchmark configurations, in the tiers of `_parity.py`:
tiny, ViT-L-like and every fraction of the modality-mix sweep element by element; Qwen2-VL-like and the video tail
through the sampled tier in the routine suite and element by element when MPIPE_FULL_PARITY=1 (minutes of CPU)."""
import os

import pytest
import torch

from paper_2607_03229_b200 import binding as B
from paper_2607_03229_b200 import workloads as W
import _parity as P

pytestmark = pytest.mark.gpu

_FULL = pytest.mark.skipif(os.environ.get("MPIPE_FULL_PARITY") != "1",
                           reason="element-by-element oracle pass of the two largest configurations takes many minutes "
                                  "of CPU; set MPIPE_FULL_PARITY=1")


def test_tiny_config_every_element():
    P.check_full(W.tiny())


def test_vit_l_config_every_element():
    P.check_full(W.vit_l())


@pytest.mark.parametrize("fraction", W.MIX_FRACTIONS)
def test_modality_mix_every_element(fraction):
    w = W.modality_mix(fraction)
    if w.total_tokens == 0:     # pure-text microbatch: nothing is launched, nothing fails
        plan = B.seg_plan(w.patch_counts, B.TRAINED).to_device()
        e = torch.zeros((0, 16, 64), dtype=torch.bfloat16, device="cuda")
        B.varlen_attn_fwd(e, e, e, e, torch.zeros((16, 0), device="cuda"), plan, 0.125)
        B.varlen_attn_bwd(e, e, e, e, e, torch.zeros((16, 0), device="cuda"), e, e, e, plan, 0.125, None)
        torch.cuda.synchronize()
        return
    P.check_full(w)


def test_qwen2vl_config_sampled_tier():
    P.check_sampled(W.qwen2vl())


def test_video_tail_config_sampled_tier():
    P.check_sampled(W.video_tail())


def test_qwen2vl_frozen_forward_has_the_trained_forward_bits():
    """Corollary 1 at benchmark size: freezing the encoder changes no forward bit."""
    w = W.qwen2vl()
    o_t = P.run_gpu(w, B.TRAINED)["o"]
    o_f = P.run_gpu(w, B.FROZEN)["o"]
    assert torch.equal(o_t.view(torch.int16), o_f.view(torch.int16))


@_FULL
def test_qwen2vl_config_every_element():
    P.check_full(W.qwen2vl())


@_FULL
def test_video_tail_config_every_element():
    P.check_full(W.video_tail())
