"""derive (Section 4.1) and the makespan of Section 4.3: the oracle against what the paper prints and against
closed forms, and the library (host code behind the C ABI) against the oracle."""
import itertools
import os

import numpy as np
import pytest

from oracle import derive as OD
from paper_2607_03229_b200 import binding as B

SK = {"1f1b": B.SK_1F1B, "gpipe": B.SK_GPIPE, "transpose": B.SK_TRANSPOSE}
KIND = ["Fwd", "Bwd", "Coll", "DpReduce", "Loss", "StepBarrier"]
COMM = [None, "Gather", "Scatter", "Send", "RecvGrad"]
GROUP = {-1: None, 0: "ReplicaGroup", 1: "DataGroup"}
EDGE = ["Activation", "Gradient", "Turnaround", "Accumulate", "Sequence"]
GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "derive_transpose_1f1b.txt")


def _rank_dropped(d, names, with_local=False):
    """The order graph with the rank index and the microbatch dropped, as the paper prints it.  Edges inside one
    region's family (slab to slab), saved-activation arcs and the per-stage / per-rank Sequence edges are left out."""
    ev, out = d["events"], set()

    def label(e):
        if e.kind in ("Fwd", "Bwd"):
            return f"{e.kind}({names[e.region]})"
        if e.kind == "Coll":
            return f"Coll({e.comm},{names[e.region]})"
        if e.kind == "DpReduce":
            return f"DpReduce({names[e.region]},{e.group})"
        return e.kind
    for a, c, t in d["edges"]:
        ea, ec = ev[a], ev[c]
        if label(ea) == label(ec):
            continue                                            # slab to slab inside one region
        if t == "Activation" and ea.kind == "Fwd" and ec.kind == "Bwd":
            continue                                            # the saved activation
        if t == "Sequence" and ec.kind != "StepBarrier":
            continue                                            # local orders
        out.add((label(ea), label(ec), t))
    return out


def _golden(trainable_enc):
    want = {"placement": {}, "seams": [], "reduces": [], "edges": set()}
    for line in open(GOLDEN):
        tok = line.split()
        if not tok or tok[0] == "#":
            continue
        optional = tok[-1].endswith("?")
        if tok[0] == "placement":
            want["placement"][tok[1]] = (tok[2], tok[3])
        elif tok[0] == "seam":
            bwd = tok[4].rstrip("?")
            want["seams"].append((tok[1], tok[2], tok[3], bwd if (trainable_enc or not tok[4].endswith("?")) else None))
        elif tok[0] == "reduce":
            if trainable_enc or not optional:
                want["reduces"].append((tok[1], tok[2]))
        elif tok[0] == "edge":
            if trainable_enc or not optional:
                want["edges"].add((tok[1], tok[2], tok[3]))
    return want


@pytest.mark.parametrize("trainable_enc", [True, False])
def test_oracle_reproduces_the_printed_instantiation(trainable_enc):
    names = {1: "enc", 2: "llm"}
    d = OD.derive(["transpose", "1f1b"], [4], 12, [trainable_enc, True], P=4, M=3)
    want = _golden(trainable_enc)
    assert {names[j]: p[:2] for j, p in d["placement"].items()} == want["placement"]
    assert [(names[j], names[j + 1], f, b) for j, f, b in d["seams"]] == want["seams"]
    assert [(names[j], g) for j, g in d["reduces"]] == want["reduces"]
    assert _rank_dropped(d, names) == want["edges"]
    if not trainable_enc:   # "The same schedule, two footprints": no reverse Scatter, no Bwd(enc), no replica reduce
        assert not any(e.kind == "Bwd" and e.region == 1 for e in d["events"])
        assert not any(e.kind == "Coll" and e.comm == "Scatter" for e in d["events"])


def test_oracle_vpp3_and_validity_examples():
    d = OD.derive(["1f1b"] * 3, [4, 8], 12, [True, True, True], P=4, M=2)
    assert [p[:2] for p in d["placement"].values()] == [("Sharded", "ByLayer")] * 3
    assert d["seams"] == [(1, "Send", "RecvGrad"), (2, "Send", "RecvGrad")]
    # region 1 again sends no input-activation gradient: there is no reverse collective left of it
    assert not any(e.kind == "Coll" and e.region == 0 for e in d["events"])
    assert OD.is_valid(["transpose", "1f1b"], [3], 10) and OD.is_valid(["transpose", "1f1b", "transpose"], [3, 7], 10)
    assert not OD.is_valid(["transpose", "transpose"], [3], 10)
    assert OD.normalize(["transpose", "transpose"], [3], 10) == (["transpose"], [])
    assert OD.normalize(["transpose", "transpose", "1f1b", "transpose", "transpose"], [1, 2, 6, 8], 10) == (
        ["transpose", "1f1b", "transpose"], [2, 6])
    assert not OD.is_valid(["1f1b", "1f1b"], [0], 10) and not OD.is_valid(["1f1b", "1f1b"], [10], 10)   # the cut must tile


def test_oracle_lemma1_truth_table_and_schedule_invariance():
    for tr in itertools.product([False, True], repeat=3):
        receives, sends, reduces = OD.gates(tr)
        for j in (1, 2, 3):
            assert receives[j] == any(tr[:j]) and sends[j] == any(tr[:j - 1]) and reduces[j] == tr[j - 1]
            # the send and receive gates differ exactly at the trainable source
            assert (receives[j] and not sends[j]) == (tr[j - 1] and not any(tr[:j - 1]))
        # Corollary 1: which backward events fire does not depend on the skeletons
        foot = []
        for sk in (["1f1b", "1f1b", "1f1b"], ["transpose", "1f1b", "gpipe"], ["transpose", "gpipe", "transpose"]):
            d = OD.derive(sk, [4, 8], 12, tr, P=4, M=2)
            foot.append((sorted({e.region for e in d["events"] if e.kind == "Bwd"}),
                         sorted({e.region for e in d["events"] if e.kind == "Coll" and e.comm in ("Scatter", "RecvGrad", "Gather")
                                 and any(x.kind == "Bwd" for x in d["events"]) and _is_reverse(d, e)}),
                         sorted(j for j, _ in d["reduces"])))
        assert foot[0] == foot[1] == foot[2]


def _is_reverse(d, coll):
    """A collective event is a reverse (backward) one when an edge of kind Gradient enters it."""
    i = d["events"].index(coll)
    return any(c == i and t == "Gradient" for _, c, t in d["edges"])


@pytest.mark.parametrize("skeleton", ["gpipe", "1f1b"])
@pytest.mark.parametrize("P,M", [(1, 3), (4, 4), (4, 9), (3, 2)])
def test_oracle_makespan_closed_forms(skeleton, P, M):
    # one Sharded region, unit forward and backward cost, everything else free: T = 2 (M + P - 1) for both skeletons,
    # and every rank is busy 2 M of it
    d = OD.derive([skeleton], [], 2 * P, [True], P=P, M=M)
    cost = [1.0 if e.kind in ("Fwd", "Bwd") else 0.0 for e in d["events"]]
    T, start, bub = OD.makespan(d["events"], d["edges"], cost, P)
    assert T == 2 * (M + P - 1)
    assert bub == [T - 2 * M] * P
    if skeleton == "1f1b":   # at most P - r forwards in flight on rank r (one region: P - 1 - r stages downstream)
        for r in range(P):
            live = 0
            for i in d["nodes"][r]:
                live += {"Fwd": 1, "Bwd": -1}.get(d["events"][i].kind, 0)
                assert live <= P - r


def test_oracle_order_is_acyclic_and_nodes_respect_edges():
    d = OD.derive(["transpose", "1f1b", "transpose"], [2, 10], 12, [True, True, False], P=4, M=5, owner=[3, 3, 2, 1, 0])
    pos = {}
    for r, lst in enumerate(d["nodes"]):
        for p, i in enumerate(lst):
            pos[i] = (r, p)
    T, start, _ = OD.makespan(d["events"], d["edges"], [1.0] * len(d["events"]), 4)   # terminates: no cycle
    for a, c, _ in d["edges"]:
        assert start[c] >= start[a] + 1.0
        if a in pos and c in pos and pos[a][0] == pos[c][0]:
            assert pos[a][1] < pos[c][1]
    # the warm-up rule: a rank's encoder forwards precede its first backbone forward
    for r, lst in enumerate(d["nodes"]):
        kinds = [(d["events"][i].kind, d["events"][i].region) for i in lst]
        if ("Fwd", 1) in kinds and ("Fwd", 2) in kinds:
            assert max(i for i, x in enumerate(kinds) if x == ("Fwd", 1)) < kinds.index(("Fwd", 2))
    assert [OD.Event("Fwd", 1, 3, 1, None, None), OD.Event("Fwd", 1, 3, 2, None, None)] == [
        d["events"][i] for i in d["nodes"][3][:2]]


# ------------------------------------------------------------------------------------------ library vs oracle
def _as_oracle(d: "B.Derived"):
    ev = [OD.Event(KIND[k], int(j), int(r), int(m), COMM[c] if KIND[k] == "Coll" else None, GROUP[int(g)])
          for k, j, r, m, c, g in d.events.tolist()]
    edges = [(int(a), int(c), EDGE[t]) for a, c, t in d.edges.tolist()]
    return ev, edges


CASES = [
    (["transpose", "1f1b"], [4], 12, [True, True], 4, 3, None),
    (["transpose", "1f1b"], [4], 12, [False, True], 4, 6, [3, 2, 3, 1, 0, 3]),
    (["1f1b", "1f1b", "1f1b"], [4, 8], 12, [True, True, True], 4, 5, None),
    (["transpose", "gpipe", "transpose"], [2, 11], 13, [True, False, True], 3, 4, [0, 2, 1, 2]),
    (["gpipe"], [], 7, [True], 3, 2, None),
    (["1f1b", "transpose"], [5], 6, [False, False], 2, 3, None),
    (["transpose"], [], 3, [True], 2, 5, None),
]


@pytest.mark.parametrize("sk,cut,L,tr,P,M,owner", CASES)
def test_library_equals_oracle(sk, cut, L, tr, P, M, owner):
    want = OD.derive(sk, cut, L, tr, P, M, owner)
    got = B.derive([SK[s] for s in sk], cut, L, [int(t) for t in tr], P, M, owner)
    ev, edges = _as_oracle(got)
    assert ev == want["events"]
    assert edges == want["edges"]
    assert got.nodes == want["nodes"]
    lay = {"Sharded": B.LAYOUT_SHARDED, "Replicated": B.LAYOUT_REPLICATED}
    for j, (layout, _, slabs) in want["placement"].items():
        assert got.regions[j - 1, 0] == lay[layout] and got.regions[j - 1, 3] == SK[sk[j - 1]]
        assert got.slabs[j - 1].tolist() == [list(s) for s in slabs]
        assert got.slabs[j - 1][:, 1].sum() == (got.regions[j - 1, 2] if layout == "Sharded" else P * got.regions[j - 1, 2])
    assert [(int(a), COMM[f], COMM[b]) for a, f, b in got.seams.tolist()] == want["seams"]
    assert [(int(j), GROUP[int(g)]) for j, g in got.reduces.tolist()] == want["reduces"]
    rng = np.random.default_rng(len(ev))
    cost = rng.uniform(0.0, 2.0, len(ev))
    T, start, bub = B.order_makespan(got.events, got.edges, cost, P)
    T0, start0, bub0 = OD.makespan(want["events"], want["edges"], list(cost), P)
    assert abs(T - T0) < 1e-12 and np.allclose(start, start0, atol=1e-12) and np.allclose(bub, bub0, atol=1e-12)


def test_library_validity_normalize_stage_index_and_errors():
    T, F = SK["transpose"], SK["1f1b"]
    assert B.schedule_valid([T, F], [3], 10) and B.schedule_valid([T, F, T], [3, 7], 10)
    assert not B.schedule_valid([T, T], [3], 10) and not B.schedule_valid([F, F], [0], 10)
    assert not B.schedule_valid([F, 7], [3], 10)
    assert B.schedule_normalize([T, T], [3], 10) == ([T], [])
    assert B.schedule_normalize([T, T, F, T, T], [1, 2, 6, 8], 10) == ([T, F, T], [2, 6])
    for P in (1, 4):
        for region in (1, 2, 3):
            for rank in range(P):
                assert B.stage_index(rank, region, P) == rank + (region - 1) * P
    with pytest.raises(B.MpipeError):
        B.derive([T, T], [3], 10, [1, 1], 2, 2)                 # not in normal form
    with pytest.raises(B.MpipeError):
        B.derive([F], [], 3, [1], 4, 2)                         # a rank without a slab
    with pytest.raises(B.MpipeError) as e:
        B.derive([T, F], [2], 8, [1, 1], 2, 2, owner=[0, 2])     # owner outside [0, P)
    assert e.value.status == B.ERR_INDEX
    d = B.derive([F], [], 4, [1], 2, 2)
    bad = d.edges.copy()
    bad[0] = [bad[0][1], bad[0][0], bad[0][2]]
    with pytest.raises(B.MpipeError):                           # a cycle is not an order graph
        B.order_makespan(d.events, np.concatenate([d.edges, bad[:1]]), np.ones(len(d.events)), 2)


# ------------------------------------------------------------------------------------------ derive + makespan together
def _makespan(sk, cut, L, tr, P, M, owner, cost_of):
    d = B.derive([SK[s] for s in sk], cut, L, [int(t) for t in tr], P, M, owner)
    ev, _ = _as_oracle(d)
    T, start, bub = B.order_makespan(d.events, d.edges, [cost_of(e) for e in ev], P)
    return T, bub, ev


def test_transposed_encoder_is_free_when_it_costs_nothing_and_never_worse_than_a_pipelined_one():
    P, M = 4, 8
    unit = lambda e: 1.0 if (e.kind in ("Fwd", "Bwd") and e.region == 2) else 0.0
    # a frozen encoder that costs nothing: the step is the backbone's 1F1B step, 2 (M + P - 1) with unit stage costs
    T, bub, _ = _makespan(["transpose", "1f1b"], [4], 12, [False, True], P, M, None, unit)
    assert T == 2 * (M + P - 1) and list(bub) == [T - 2 * M] * P
    # the same model with the encoder as one more pipelined region (region 1 sharded over the same ranks, each rank's slab
    # costing e / P per microbatch) against the transposed encoder (the whole e on the owner): the transposed step is never
    # longer, and it is strictly shorter once the encoder is not negligible -- the warm-up bubble absorbs it
    for e_cost in (0.5, 2.0):
        enc_sharded = lambda e: (e_cost / P if e.region == 1 else 1.0) if e.kind == "Fwd" else (1.0 if e.kind == "Bwd" and e.region == 2 else 0.0)
        enc_transposed = lambda e: (e_cost if e.region == 1 else 1.0) if e.kind == "Fwd" else (1.0 if e.kind == "Bwd" and e.region == 2 else 0.0)
        T_pipe, _, _ = _makespan(["1f1b", "1f1b"], [4], 12, [False, True], P, M, None, enc_sharded)
        owner = [(P - 1) - (m % P) for m in range(M)]     # later ranks have the longer warm-up slots
        T_tr, bub_tr, ev = _makespan(["transpose", "1f1b"], [4], 12, [False, True], P, M, owner, enc_transposed)
        assert T_tr <= T_pipe + 1e-12
        # lower bounds that any order must respect: the busiest rank's work, and microbatch 1's own critical path
        work = [sum(enc_transposed(e) for e in ev if e.rank == r) for r in range(P)]
        assert T_tr >= max(work) - 1e-12 and T_tr >= e_cost + 2 * P - 1e-12
        assert all(abs(b - (T_tr - w_)) < 1e-9 for b, w_ in zip(bub_tr, work))


def test_trainable_encoder_adds_its_backward_to_the_cool_down():
    P, M = 4, 6
    cost = lambda e: {"Fwd": 1.0, "Bwd": 2.0}.get(e.kind, 0.0) if e.region == 2 else ({"Fwd": 0.25, "Bwd": 0.5}.get(e.kind, 0.0) if e.region == 1 else 0.0)
    T_frozen, _, ev_f = _makespan(["transpose", "1f1b"], [4], 12, [False, True], P, M, None, cost)
    T_trained, _, ev_t = _makespan(["transpose", "1f1b"], [4], 12, [True, True], P, M, None, cost)
    assert T_trained >= T_frozen
    assert sum(1 for e in ev_t if e.kind == "Bwd" and e.region == 1) == M and not any(e.kind == "Bwd" and e.region == 1 for e in ev_f)
    # the last encoder backward can only start after the backbone's last backward on rank 0
    assert T_trained >= T_frozen + 0.5 - 1e-12
