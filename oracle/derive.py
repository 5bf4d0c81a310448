"""CPU oracle for `derive` (Section 4.1, "Schedule Algebra") and the makespan of Section 4.3 -- TEST
INFRASTRUCTURE, not product code.  Plain Python over named tuples and sets; it shares nothing with the library.

    derive : cut x schedule x model -> placement x collectives x order

Rules, in the paper's words where it has them:
* layout(transpose) = Replicated, layout(1f1b) = layout(gpipe) = Sharded.  A schedule is valid when its cut tiles
  the model and no two adjacent regions are Replicated; normalising collapses such a run into one region.
* Table 2 gives each seam's forward and backward collective from the layout pair.
* Lemma 1: region j receives a gradient / runs a backward iff some region i <= j is trainable; it sends its input
  gradient upstream (the reverse collective on seam (j-1, j)) iff some i < j is trainable; it reduces weight
  gradients iff it is trainable itself (ReplicaGroup when Replicated, DataGroup when Sharded).
* A Sharded region emits one Fwd(region, r, m) per rank on its ByLayer slab, a Replicated one emits one at
  r = ByMicrobatch(m).  stage_index = rank + (region - 1) P.
* Edges: forward arcs are Activation (and so is the saved activation Fwd -> its own Bwd), Loss -> Bwd is the
  Turnaround, backward arcs into a reverse seam and along the backward chain are Gradient, Bwd -> DpReduce is
  Accumulate, DpReduce -> StepBarrier is Sequence.
Readings where the paper is silent (its figure is missing): the per-stage orders of the three skeletons, the
unit-cost list scheduling that produces nodes(r) with the warm-up / cool-down priority, slabs by even split with
the remainder to the first ranks, the creation order of events (it breaks ties) -- all stated in the C header.

Pins: ``tests/test_derive.py`` (the instantiation the paper prints, its frozen collapse, VPP-3, the validity
examples, Lemma 1's truth table, closed-form makespans of GPipe and 1F1B).
"""
from __future__ import annotations

from collections import namedtuple
from typing import Dict, List, Optional, Sequence

Event = namedtuple("Event", "kind region rank mb comm group")   # kind in Fwd Bwd Coll DpReduce Loss StepBarrier

SEAM_TABLE = {("Replicated", "Sharded"): ("Gather", "Scatter"),
              ("Sharded", "Sharded"): ("Send", "RecvGrad"),
              ("Sharded", "Replicated"): ("Scatter", "Gather")}


def layout(skeleton: str) -> str:
    assert skeleton in ("1f1b", "gpipe", "transpose")
    return "Replicated" if skeleton == "transpose" else "Sharded"


def tiles(cut: Sequence[int], k: int, n_layers: int) -> bool:
    bounds = [0] + list(cut) + [n_layers]
    return len(cut) == k - 1 and all(a < b for a, b in zip(bounds, bounds[1:]))


def is_valid(skeletons: Sequence[str], cut: Sequence[int], n_layers: int) -> bool:
    if not skeletons or not tiles(cut, len(skeletons), n_layers):
        return False
    lay = [layout(s) for s in skeletons]
    return not any(a == b == "Replicated" for a, b in zip(lay, lay[1:]))


def normalize(skeletons: Sequence[str], cut: Sequence[int], n_layers: int):
    """Collapse every run of adjacent Replicated regions into one (the boundary between them goes away)."""
    assert tiles(cut, len(skeletons), n_layers)
    sk, ct = [skeletons[0]], []
    for j in range(1, len(skeletons)):
        if layout(sk[-1]) == "Replicated" and layout(skeletons[j]) == "Replicated":
            continue
        sk.append(skeletons[j])
        ct.append(cut[j - 1])
    return sk, ct


def gates(trainable: Sequence[bool]):
    """Lemma 1 for regions 1..k -> (receives[j], sends[j], reduces[j]) as dicts keyed by the 1-based region."""
    k = len(trainable)
    receives = {j: any(trainable[:j]) for j in range(1, k + 1)}
    sends = {j: any(trainable[:j - 1]) for j in range(1, k + 1)}
    reduces = {j: bool(trainable[j - 1]) for j in range(1, k + 1)}
    return receives, sends, reduces


def slabs_by_layer(first: int, count: int, P: int):
    out, at = [], first
    for r in range(P):
        n = count // P + (1 if r < count % P else 0)
        out.append((at, n))
        at += n
    return out


def derive(skeletons: Sequence[str], cut: Sequence[int], n_layers: int, trainable: Sequence[bool], P: int, M: int,
           owner: Optional[Sequence[int]] = None) -> Dict:
    assert is_valid(skeletons, cut, n_layers)
    k = len(skeletons)
    lay = {j: layout(skeletons[j - 1]) for j in range(1, k + 1)}
    bounds = [0] + list(cut) + [n_layers]
    own = (lambda m: owner[m - 1]) if owner is not None else (lambda m: (m - 1) % P)
    receives, sends, reduces_gate = gates(trainable)

    placement = {}
    for j in range(1, k + 1):
        first, count = bounds[j - 1], bounds[j] - bounds[j - 1]
        if lay[j] == "Sharded":
            assert count >= P
            placement[j] = ("Sharded", "ByLayer", slabs_by_layer(first, count, P))
        else:
            placement[j] = ("Replicated", "ByMicrobatch", [(first, count)] * P)
    seams = []
    for j in range(1, k):
        fwd, bwd = SEAM_TABLE[(lay[j], lay[j + 1])]
        seams.append((j, fwd, bwd if sends[j + 1] else None))
    reduces = [(j, "ReplicaGroup" if lay[j] == "Replicated" else "DataGroup") for j in range(1, k + 1) if reduces_gate[j]]

    events: List[Event] = []
    edges = []            # (src index, dst index, type)

    def emit(*a):
        events.append(Event(*a))
        return len(events) - 1

    def ranks_of(j, m):
        return list(range(P)) if lay[j] == "Sharded" else [own(m)]

    fwd_of, bwd_of, loss_of = {}, {}, {}
    for m in range(1, M + 1):
        prev = None
        for j in range(1, k + 1):
            for r in ranks_of(j, m):
                e = emit("Fwd", j, r, m, None, None)
                fwd_of[(j, r, m)] = e
                if prev is not None:
                    edges.append((prev, e, "Activation"))
                prev = e
            if j < k:
                c = emit("Coll", j, ranks_of(j + 1, m)[0], m, seams[j - 1][1], None)
                edges.append((prev, c, "Activation"))
                prev = c
        loss_of[m] = emit("Loss", k, ranks_of(k, m)[-1], m, None, None)
        edges.append((prev, loss_of[m], "Activation"))
        prev, kind = loss_of[m], "Turnaround"
        for j in range(k, 0, -1):
            if not receives[j]:
                break
            for r in reversed(ranks_of(j, m)):
                e = emit("Bwd", j, r, m, None, None)
                bwd_of[(j, r, m)] = e
                edges.append((prev, e, kind))
                kind = "Gradient"
                edges.append((fwd_of[(j, r, m)], e, "Activation"))
                prev = e
            if sends[j]:
                c = emit("Coll", j - 1, ranks_of(j - 1, m)[-1], m, seams[j - 2][2], None)
                edges.append((prev, c, "Gradient"))
                prev = c
    reduce_of = {j: emit("DpReduce", j, -1, 0, None, g) for j, g in reduces}
    barrier = emit("StepBarrier", 0, -1, 0, None, None)
    for j, _ in reduces:
        for m in range(1, M + 1):
            for r in range(P):
                if (j, r, m) in bwd_of:
                    edges.append((bwd_of[(j, r, m)], reduce_of[j], "Accumulate"))
        edges.append((reduce_of[j], barrier, "Sequence"))
    if not reduces:
        for m in range(1, M + 1):
            edges.append((loss_of[m], barrier, "Sequence"))

    # the skeleton's order inside a stage
    for j in range(1, k + 1):
        for r in range(P):
            f = [fwd_of[(j, r, m)] for m in range(1, M + 1) if (j, r, m) in fwd_of]
            b = [bwd_of[(j, r, m)] for m in range(1, M + 1) if (j, r, m) in bwd_of]
            sk = skeletons[j - 1]
            if sk == "1f1b" and b:
                # forwards in flight before the first backward = the stages downstream of this one
                depth = (P - 1 - r) + sum(P if lay[i] == "Sharded" else 1 for i in range(j + 1, k + 1))
                warm = min(len(f), depth)
                seq = f[:warm]
                for i, fe in enumerate(f[warm:]):
                    seq += [fe, b[i]]
                seq += b[len(f) - warm:]
            elif sk == "gpipe":
                seq = f + b[::-1]
            else:
                seq = f + b
            edges += [(a, c, "Sequence") for a, c in zip(seq, seq[1:])]

    # nodes(r): unit-cost list scheduling with the warm-up / cool-down priority
    sharded = [j for j in range(1, k + 1) if lay[j] == "Sharded"]
    first_sharded = sharded[0] if sharded else k + 1

    def prio(e: Event):
        if e.kind in ("Fwd", "Bwd") and lay[e.region] == "Replicated":
            return 0 if (e.kind == "Fwd" and e.region < first_sharded) else 2
        return 1
    preds = {i: set() for i in range(len(events))}
    for a, c, _ in edges:
        preds[c].add(a)
    finished_at = {}
    nodes = [[] for _ in range(P)]
    step = 0
    while len(finished_at) < len(events):
        ready = [i for i in range(len(events)) if i not in finished_at
                 and all(p in finished_at and finished_at[p] < step for p in preds[i])]
        run = [i for i in ready if events[i].rank < 0]
        for r in range(P):
            mine = [i for i in ready if events[i].rank == r]
            if mine:
                best = min(mine, key=lambda i: (prio(events[i]), i))
                run.append(best)
                nodes[r].append(best)
        for i in run:
            finished_at[i] = step
        step += 1
        assert step <= 4 * len(events) + 4, "no progress: the graph would have a cycle"
    have = {(a, c) for a, c, _ in edges}
    for r in range(P):
        for a, c in zip(nodes[r], nodes[r][1:]):
            if (a, c) not in have:
                edges.append((a, c, "Sequence"))
    return {"placement": placement, "seams": seams, "reduces": reduces, "events": events, "edges": edges, "nodes": nodes}


def makespan(events: Sequence[Event], edges, cost: Sequence[float], P: int):
    """T = longest path (costs on events), earliest starts, bub(r) = T - sum of rank r's costs."""
    n = len(events)
    preds = {i: [] for i in range(n)}
    for a, c, _ in edges:
        preds[c].append(a)
    start: Dict[int, float] = {}

    def start_of(i):   # memoised recursion over predecessors (the graphs here are small)
        if i not in start:
            start[i] = max((start_of(p) + cost[p] for p in preds[i]), default=0.0)
        return start[i]
    import sys
    sys.setrecursionlimit(max(10000, 4 * n))
    T = max((start_of(i) + cost[i] for i in range(n)), default=0.0)
    bub = [T - sum(cost[i] for i in range(n) if events[i].rank == r) for r in range(P)]
    return T, [start_of(i) for i in range(n)], bub
