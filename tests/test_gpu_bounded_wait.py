"""The kernels' waits are bounded: a wait that nothing satisfies ends by itself, reports MPIPE_ERR_TIMEOUT
through the status buffer and leaves the context usable (no trap, no fault, no hang)."""
import time

import numpy as np
import pytest
import torch

import oracle
from paper_2607_03229_b200 import binding as B
from paper_2607_03229_b200 import workloads as W
from _util import status_buf, to_bits, to_dev

pytestmark = pytest.mark.gpu


def test_wait_that_nothing_satisfies_times_out_and_the_context_survives():
    st = status_buf()
    t0 = time.perf_counter()
    B.selftest_wait_timeout(20_000_000, st)       # about 10 ms of SM clocks
    torch.cuda.synchronize()
    assert time.perf_counter() - t0 < 5.0
    got = st.cpu().tolist()
    assert got[0] == B.ERR_TIMEOUT and got[1] == 0
    # the same context still runs the library's kernels correctly
    w = W.tiny()
    enc, emb = w.merge_source(), w.llm_embeds()
    emb_d = to_dev(emb)
    B.merge_tokens(to_dev(enc), emb_d, torch.from_numpy(w.positions).cuda())
    torch.cuda.synchronize()
    assert np.array_equal(to_bits(emb_d), oracle.merge_tokens(enc, emb, w.positions))


def test_selftest_rejects_bad_arguments():
    with pytest.raises(B.MpipeError):
        B.selftest_wait_timeout(0, status_buf())
    with pytest.raises(B.MpipeError):
        B.selftest_wait_timeout(1000, None)
