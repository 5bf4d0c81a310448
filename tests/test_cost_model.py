"""The cost model of Section 4.3 behind the C ABI against the oracle's plain restatement, closed forms and a brute
force over all assignments on tiny instances."""
import numpy as np
import pytest

import oracle
from paper_2607_03229_b200 import binding as B
from paper_2607_03229_b200 import build as build_mod
from paper_2607_03229_b200 import workloads as W


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_mod.build()


def test_event_and_collective_costs():
    # compute-bound and bandwidth-bound sides of the roofline, and the ridge point
    assert B.event_cost(2e12, 1e9, 1e15, 1e12) == pytest.approx(2e-3)      # 2 ms of FLOPs vs 1 ms of bytes
    assert B.event_cost(1e11, 4e9, 1e15, 1e12) == pytest.approx(4e-3)      # 0.1 ms of FLOPs vs 4 ms of bytes
    assert B.event_cost(1e12, 1e9, 1e15, 1e12) == pytest.approx(1e-3)      # both 1 ms
    assert B.event_cost(3e12, 2e9, 2e15, 8e12) == oracle.event_cost(3e12, 2e9, 2e15, 8e12)
    assert B.coll_cost(5e-6, 1.25e-12, 4e8) == pytest.approx(5e-6 + 5e-4)
    assert B.coll_cost(1e-5, 2e-12, 0.0) == 1e-5
    with pytest.raises(B.MpipeError):
        B.event_cost(1.0, 1.0, 0.0, 1.0)
    with pytest.raises(B.MpipeError):
        B.coll_cost(-1.0, 0.0, 1.0)


@pytest.mark.parametrize("mode", [B.FROZEN, B.TRAINED])
def test_encoder_attention_work_matches_the_flop_and_byte_conventions(mode):
    for w in (W.tiny(), W.vit_l(), W.qwen2vl(), W.modality_mix(0.0)):
        got = B.encoder_attn_work(w.patch_counts, w.n_heads, w.head_dim, mode)
        ref = oracle.encoder_attn_work(w.patch_counts, w.n_heads, w.head_dim, mode == B.TRAINED)
        assert got == ref
        assert got[0] == w.flops(True, False)
        assert got[2] == (w.flops(False, True) if mode == B.TRAINED else 0.0)
    # hand value: one image of 10 patches, 2 heads of 8: fwd 4*2*8*100 = 6400 FLOPs, 10*2*(64+4) = 1360 bytes
    assert B.encoder_attn_work([10], 2, 8, B.TRAINED) == (6400.0, 1360.0, 16000.0, 10 * 2 * (128 + 16.0))
    assert B.encoder_attn_work([10], 2, 8, B.FROZEN) == (6400.0, 1280.0, 0.0, 0.0)


def test_warmup_slack_1f1b():
    assert B.warmup_slack_1f1b(4, 3.0, 0.5).tolist() == [0.0, 3.5, 7.0, 10.5]
    assert B.warmup_slack_1f1b(1, 3.0, 0.5).tolist() == [0.0]
    with pytest.raises(B.MpipeError):
        B.warmup_slack_1f1b(0, 1.0, 0.0)


def test_owner_map_closed_forms():
    # enough slack everywhere: nothing spills, whatever the assignment
    owner, work, spill, mx = B.owner_map([1.0, 2.0, 3.0], [10.0, 10.0])
    assert mx == 0.0 and spill.tolist() == [0.0, 0.0] and work.sum() == 6.0
    # one rank: spill = max(0, sum - w)
    _, work, spill, mx = B.owner_map([1.0, 2.0, 3.0], [4.0])
    assert work.tolist() == [6.0] and mx == 2.0
    # "heavier encodes to longer warm-up slots": the heavy one goes to the last rank of a 1F1B pipeline
    slack = B.warmup_slack_1f1b(4, 1.0, 0.0)           # 0, 1, 2, 3
    owner, work, spill, mx = B.owner_map([0.5, 3.0, 1.0, 2.0], slack)
    assert owner.tolist() == [3, 3, 1, 2] or owner[1] == 3
    assert owner[1] == 3 and owner[3] == 2
    # no microbatches
    owner, work, spill, mx = B.owner_map([], [1.0, 2.0])
    assert owner.size == 0 and mx == 0.0 and work.tolist() == [0.0, 0.0]
    with pytest.raises(B.MpipeError):
        B.owner_map([1.0, -2.0], [1.0])
    with pytest.raises(B.MpipeError):
        B.owner_map([1.0], [])


def test_owner_map_against_oracle_greedy_and_brute_force_optimum():
    rng = np.random.default_rng(11)
    for trial in range(60):
        P = int(rng.integers(1, 5))
        M = int(rng.integers(0, 8))
        cost = [float(x) for x in np.round(rng.uniform(0.1, 4.0, size=M), 3)]
        slack = [float(x) for x in np.round(np.sort(rng.uniform(0.0, 5.0, size=P)), 3)]
        owner, work, spill, mx = B.owner_map(cost, slack)
        ref_owner = oracle.owner_map_greedy(cost, slack)
        assert owner.tolist() == ref_owner
        rw, rs, rmx = oracle.spills(ref_owner, cost, slack)
        assert np.allclose(work, rw) and np.allclose(spill, rs) and mx == pytest.approx(rmx)
        opt = oracle.owner_map_optimal(cost, slack)
        assert mx >= opt - 1e-12                              # greedy can never beat the optimum ...
        assert mx <= opt + (max(cost) if cost else 0.0) + 1e-12   # ... and overshoots it by at most one microbatch


def test_cost_model_on_the_benchmark_workloads():
    """Encoder event costs of the modality-mix sweep on a measured roofline, spread over 8 pipeline ranks."""
    F, Bw = 1388.9e12, 6539.9e9
    costs = []
    for f in (0.10, 0.25, 0.50, 0.75, 0.10, 0.75, 0.25, 0.50):
        w = W.modality_mix(f)
        ff, fb, bf, bb = B.encoder_attn_work(w.patch_counts, w.n_heads, w.head_dim, B.TRAINED)
        costs.append(B.event_cost(ff, fb, F, Bw))
    assert all(c > 0 for c in costs) and costs[3] > costs[0]
    slack = B.warmup_slack_1f1b(8, 2e-4, 1e-5)
    owner, work, spill, mx = B.owner_map(costs, slack)
    assert work.sum() == pytest.approx(sum(costs))
    assert spill[0] == work[0]                                  # rank 0 has no warm-up bubble to hide anything in
    assert mx == pytest.approx(max(0.0, (work - slack).max()))
