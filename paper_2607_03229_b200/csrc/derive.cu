// derive : cut x schedule x model -> placement x collectives x order   (Section 4.1, "Schedule Algebra")
//
// Host-only, integer logic: validity and normal form of a schedule, the placement of every region, the seam
// collectives of Table 2 gated by Lemma 1, and the order graph (six event kinds, five edge kinds) with each
// rank's projection nodes(r).  mpipe_order_makespan reads the step time and the per-rank bubbles off that graph
// (Section 4.3: T = longest path when each rank's events follow nodes(r); bub(r) = T - sum of its costs).
#include <stdint.h>

#include <algorithm>
#include <vector>

#include "common.h"

namespace mpipe {
namespace {

inline int layout_of(int skeleton) { return skeleton == MPIPE_SK_TRANSPOSE ? MPIPE_LAYOUT_REPLICATED : MPIPE_LAYOUT_SHARDED; }

bool cut_tiles(const int32_t* cut, int k, int n_layers) {
    int prev = 0;
    for (int j = 0; j + 1 < k; ++j) {
        if (cut[j] <= prev || cut[j] >= n_layers) return false;
        prev = cut[j];
    }
    return k >= 1 && n_layers >= k;
}

bool skeletons_ok(const int32_t* sk, int k) {
    for (int j = 0; j < k; ++j)
        if (sk[j] != MPIPE_SK_1F1B && sk[j] != MPIPE_SK_GPIPE && sk[j] != MPIPE_SK_TRANSPOSE) return false;
    return true;
}

struct Builder {
    std::vector<mpipe_event_t> ev;
    std::vector<mpipe_edge_t> ed;
    int add_event(int kind, int region, int rank, int mb, int comm, int group) {
        ev.push_back(mpipe_event_t{kind, region, rank, mb, comm, group});
        return int(ev.size()) - 1;
    }
    void add_edge(int src, int dst, int type) {
        if (src >= 0 && dst >= 0) ed.push_back(mpipe_edge_t{src, dst, type});
    }
};

}  // namespace
}  // namespace mpipe

extern "C" {

int32_t mpipe_stage_index(int32_t rank, int32_t region, int32_t n_ranks) { return rank + (region - 1) * n_ranks; }

int32_t mpipe_schedule_valid(const int32_t* skeletons, const int32_t* cut, int32_t k, int32_t n_layers) {
    using namespace mpipe;
    if (skeletons == nullptr || k < 1 || n_layers < 1 || (k > 1 && cut == nullptr)) return MPIPE_ERR_INVALID_ARG;
    if (!skeletons_ok(skeletons, k) || !cut_tiles(cut, k, n_layers)) return MPIPE_ERR_INVALID_ARG;
    for (int j = 0; j + 1 < k; ++j)   // normal form: no two adjacent Replicated regions
        if (layout_of(skeletons[j]) == MPIPE_LAYOUT_REPLICATED && layout_of(skeletons[j + 1]) == MPIPE_LAYOUT_REPLICATED)
            return MPIPE_ERR_INVALID_ARG;
    return MPIPE_OK;
}

int32_t mpipe_schedule_normalize(const int32_t* skeletons, const int32_t* cut, int32_t k, int32_t n_layers,
                                 int32_t* out_skeletons, int32_t* out_cut, int32_t* out_k) {
    using namespace mpipe;
    if (skeletons == nullptr || out_skeletons == nullptr || out_k == nullptr || k < 1 || (k > 1 && (cut == nullptr || out_cut == nullptr)))
        return MPIPE_ERR_INVALID_ARG;
    if (!skeletons_ok(skeletons, k) || !cut_tiles(cut, k, n_layers)) return MPIPE_ERR_INVALID_ARG;
    int n = 0;
    for (int j = 0; j < k; ++j) {
        // two adjacent Replicated regions share one owner: their seam is the identity and they are one region
        if (n > 0 && layout_of(out_skeletons[n - 1]) == MPIPE_LAYOUT_REPLICATED && layout_of(skeletons[j]) == MPIPE_LAYOUT_REPLICATED)
            continue;                       // the boundary before region j disappears
        if (n > 0) out_cut[n - 1] = cut[j - 1];
        out_skeletons[n++] = skeletons[j];
    }
    *out_k = n;
    return MPIPE_OK;
}

int32_t mpipe_derive(const int32_t* skeletons, const int32_t* cut, int32_t k, int32_t n_layers, const int32_t* trainable,
                     int32_t n_ranks, int32_t n_microbatches, const int32_t* owner, mpipe_region_t* regions, int32_t* slabs,
                     mpipe_seam_t* seams, mpipe_reduce_t* reduces, int32_t* n_reduces, mpipe_event_t* events, int32_t events_cap,
                     int32_t* n_events, mpipe_edge_t* edges, int32_t edges_cap, int32_t* n_edges, int32_t* node_order,
                     int32_t* node_offsets) {
    using namespace mpipe;
    const int P = n_ranks, M = n_microbatches;
    if (mpipe_schedule_valid(skeletons, cut, k, n_layers) != MPIPE_OK) return MPIPE_ERR_INVALID_ARG;
    if (trainable == nullptr || P < 1 || M < 0 || n_events == nullptr || n_edges == nullptr || n_reduces == nullptr)
        return MPIPE_ERR_INVALID_ARG;
    if (regions == nullptr || slabs == nullptr || (k > 1 && seams == nullptr) || reduces == nullptr || node_offsets == nullptr)
        return MPIPE_ERR_INVALID_ARG;
    if (owner != nullptr)
        for (int m = 0; m < M; ++m)
            if (owner[m] < 0 || owner[m] >= P) return MPIPE_ERR_INDEX;
    auto owner_of = [&](int m) { return owner != nullptr ? owner[m - 1] : (m - 1) % P; };   // mb is 1-based

    // ---- placement: layout, and the owner's table (ByLayer: contiguous slabs, the remainder to the first ranks;
    //      ByMicrobatch: the whole region on every rank, microbatch -> rank given by `owner`)
    std::vector<int> layout(k + 2, -1), first(k + 2), count(k + 2);
    for (int j = 1; j <= k; ++j) {
        first[j] = (j == 1) ? 0 : cut[j - 2];
        count[j] = ((j == k) ? n_layers : cut[j - 1]) - first[j];
        layout[j] = layout_of(skeletons[j - 1]);
        if (layout[j] == MPIPE_LAYOUT_SHARDED && count[j] < P) return MPIPE_ERR_INVALID_ARG;   // a rank without a slab
        regions[j - 1] = mpipe_region_t{layout[j], first[j], count[j], skeletons[j - 1]};
        int at = first[j];
        for (int r = 0; r < P; ++r) {
            int32_t* s = slabs + (size_t(j - 1) * P + r) * 2;
            if (layout[j] == MPIPE_LAYOUT_SHARDED) {
                const int len = count[j] / P + (r < count[j] % P ? 1 : 0);
                s[0] = at; s[1] = len; at += len;
            } else {
                s[0] = first[j]; s[1] = count[j];
            }
        }
    }
    // ---- Lemma 1: gate (ii) "region j runs a backward / receives a gradient" iff some i <= j is trainable;
    //      gate (i) "region j sends its input gradient upstream" iff some i < j is trainable; gate (iii) reduce iff trainable(j)
    std::vector<char> any_le(k + 2, 0);
    for (int j = 1; j <= k; ++j) any_le[j] = any_le[j - 1] || trainable[j - 1] != 0;
    auto has_bwd = [&](int j) { return any_le[j] != 0; };
    auto sends_up = [&](int j) { return j > 1 && any_le[j - 1] != 0; };
    // ---- collectives: Table 2 per adjacent layout pair; the backward comm is present iff sends_up(j + 1)
    for (int j = 1; j < k; ++j) {
        int fwd, bwd;
        if (layout[j] == MPIPE_LAYOUT_REPLICATED) { fwd = MPIPE_COMM_GATHER; bwd = MPIPE_COMM_SCATTER; }
        else if (layout[j + 1] == MPIPE_LAYOUT_REPLICATED) { fwd = MPIPE_COMM_SCATTER; bwd = MPIPE_COMM_GATHER; }
        else { fwd = MPIPE_COMM_SEND; bwd = MPIPE_COMM_RECVGRAD; }
        seams[j - 1] = mpipe_seam_t{j, fwd, sends_up(j + 1) ? bwd : MPIPE_COMM_NONE};
    }
    int nr = 0;
    for (int j = 1; j <= k; ++j)
        if (trainable[j - 1]) reduces[nr++] = mpipe_reduce_t{j, layout[j] == MPIPE_LAYOUT_REPLICATED ? MPIPE_GROUP_REPLICA : MPIPE_GROUP_DATA};
    *n_reduces = nr;

    // ---- order: events.  fwd_id / bwd_id [(j, r, m)] -> event index (-1 where the stage has no such event)
    Builder b;
    auto idx = [&](int j, int r, int m) { return (size_t(j - 1) * P + r) * size_t(M) + (m - 1); };
    std::vector<int> fwd_id(size_t(k) * P * std::max(M, 1), -1), bwd_id(fwd_id.size(), -1);
    std::vector<int> loss_id(M + 1, -1);
    auto first_rank = [&](int j, int m) { return layout[j] == MPIPE_LAYOUT_SHARDED ? 0 : owner_of(m); };
    auto last_rank = [&](int j, int m) { return layout[j] == MPIPE_LAYOUT_SHARDED ? P - 1 : owner_of(m); };
    for (int m = 1; m <= M; ++m) {
        int prev = -1;   // the event whose output feeds the next forward
        for (int j = 1; j <= k; ++j) {
            const int r0 = first_rank(j, m), r1 = last_rank(j, m);
            for (int r = r0; r <= r1; ++r) {
                const int e = b.add_event(MPIPE_EV_FWD, j, r, m, MPIPE_COMM_NONE, -1);
                fwd_id[idx(j, r, m)] = e;
                b.add_edge(prev, e, MPIPE_EDGE_ACTIVATION);
                prev = e;
            }
            if (j < k) {   // the seam's forward collective, received by the first rank of the next region
                const int c = b.add_event(MPIPE_EV_COLL, j, first_rank(j + 1, m), m, seams[j - 1].fwd_comm, -1);
                b.add_edge(prev, c, MPIPE_EDGE_ACTIVATION);
                prev = c;
            }
        }
        loss_id[m] = b.add_event(MPIPE_EV_LOSS, k, last_rank(k, m), m, MPIPE_COMM_NONE, -1);
        b.add_edge(prev, loss_id[m], MPIPE_EDGE_ACTIVATION);
        prev = loss_id[m];
        int type = MPIPE_EDGE_TURNAROUND;   // Loss -> first Bwd is the turnaround; everything after it is a gradient arc
        for (int j = k; j >= 1 && has_bwd(j); --j) {
            const int r0 = first_rank(j, m), r1 = last_rank(j, m);
            for (int r = r1; r >= r0; --r) {
                const int e = b.add_event(MPIPE_EV_BWD, j, r, m, MPIPE_COMM_NONE, -1);
                bwd_id[idx(j, r, m)] = e;
                b.add_edge(prev, e, type);
                type = MPIPE_EDGE_GRADIENT;
                b.add_edge(fwd_id[idx(j, r, m)], e, MPIPE_EDGE_ACTIVATION);   // the saved activation: live from Fwd to Bwd
                prev = e;
            }
            if (sends_up(j)) {   // reverse collective on the input seam (j-1, j), received by region j-1's last rank
                const int c = b.add_event(MPIPE_EV_COLL, j - 1, last_rank(j - 1, m), m, seams[j - 2].bwd_comm, -1);
                b.add_edge(prev, c, MPIPE_EDGE_GRADIENT);
                prev = c;
            }
        }
    }
    std::vector<int> reduce_id(k + 2, -1);
    for (int i = 0; i < nr; ++i)
        reduce_id[reduces[i].region] = b.add_event(MPIPE_EV_DPREDUCE, reduces[i].region, -1, 0, MPIPE_COMM_NONE, reduces[i].group);
    const int barrier = b.add_event(MPIPE_EV_STEPBARRIER, 0, -1, 0, MPIPE_COMM_NONE, -1);
    for (int j = 1; j <= k; ++j) {
        if (reduce_id[j] < 0) continue;
        for (int m = 1; m <= M; ++m)
            for (int r = 0; r < P; ++r) b.add_edge(bwd_id[idx(j, r, m)], reduce_id[j], MPIPE_EDGE_ACCUMULATE);
        b.add_edge(reduce_id[j], barrier, MPIPE_EDGE_SEQUENCE);
    }
    if (nr == 0)   // nothing trainable: the step ends after the last loss
        for (int m = 1; m <= M; ++m) b.add_edge(loss_id[m], barrier, MPIPE_EDGE_SEQUENCE);

    // ---- the skeleton's order inside each stage (region, rank): Sequence edges between consecutive events
    std::vector<std::vector<int>> stage_seq(size_t(k) * P);
    for (int j = 1; j <= k; ++j) {
        for (int r = 0; r < P; ++r) {
            std::vector<int>& seq = stage_seq[size_t(j - 1) * P + r];
            std::vector<int> f, bw;
            for (int m = 1; m <= M; ++m) {
                if (fwd_id[idx(j, r, m)] >= 0) f.push_back(fwd_id[idx(j, r, m)]);
                if (bwd_id[idx(j, r, m)] >= 0) bw.push_back(bwd_id[idx(j, r, m)]);
            }
            if (skeletons[j - 1] == MPIPE_SK_1F1B && !bw.empty()) {
                // forwards in flight before the first backward = the stages downstream of this one
                int depth = P - 1 - r;
                for (int i = j + 1; i <= k; ++i) depth += (layout[i] == MPIPE_LAYOUT_SHARDED) ? P : 1;
                const size_t warm = std::min<size_t>(f.size(), size_t(depth));
                size_t fi = 0, bi = 0;
                for (; fi < warm; ++fi) seq.push_back(f[fi]);
                while (fi < f.size()) { seq.push_back(f[fi++]); seq.push_back(bw[bi++]); }
                while (bi < bw.size()) seq.push_back(bw[bi++]);
            } else if (skeletons[j - 1] == MPIPE_SK_GPIPE) {
                seq = f;
                for (size_t i = bw.size(); i-- > 0;) seq.push_back(bw[i]);   // all forwards, then the backwards last-in first-out
            } else {   // transpose (or a 1f1b region with no backward): forwards, then backwards, by microbatch
                seq = f;
                seq.insert(seq.end(), bw.begin(), bw.end());
            }
            for (size_t i = 1; i < seq.size(); ++i) b.add_edge(seq[i - 1], seq[i], MPIPE_EDGE_SEQUENCE);
        }
    }
    // ---- nodes(r): list scheduling with unit costs over the graph so far.  Priority when several events of one rank
    //      are ready: (0) forwards of a Replicated region that no Sharded region precedes -- they fill the warm-up
    //      bubble and go first; (1) events of Sharded regions, collectives, losses; (2) the other events of Replicated
    //      regions (their backwards go to the cool-down).  Ties: lower event index.
    const int n = int(b.ev.size());
    int first_sharded = k + 1;
    for (int j = k; j >= 1; --j) if (layout[j] == MPIPE_LAYOUT_SHARDED) first_sharded = j;
    auto prio = [&](const mpipe_event_t& e) {
        if ((e.kind == MPIPE_EV_FWD || e.kind == MPIPE_EV_BWD) && layout[e.region] == MPIPE_LAYOUT_REPLICATED)
            return (e.kind == MPIPE_EV_FWD && e.region < first_sharded) ? 0 : 2;
        return 1;
    };
    std::vector<int> indeg(n, 0);
    std::vector<std::vector<int>> succ(n);
    for (const mpipe_edge_t& e : b.ed) { succ[e.src].push_back(e.dst); ++indeg[e.dst]; }
    std::vector<std::vector<int>> nodes(P);
    std::vector<int> ready_at(n, 0), done(n, 0);
    int remaining = n;
    std::vector<int> frontier;
    for (int e = 0; e < n; ++e) if (indeg[e] == 0) frontier.push_back(e);
    for (int step = 0; remaining > 0; ++step) {
        std::vector<int> run;   // one event per rank per step; rank-less events (reduces, barrier) run as soon as ready
        std::vector<int> pick(P, -1);
        for (int e : frontier) {
            if (done[e] || ready_at[e] > step) continue;
            const int r = b.ev[e].rank;
            if (r < 0) { run.push_back(e); continue; }
            if (pick[r] < 0 || prio(b.ev[e]) < prio(b.ev[pick[r]]) || (prio(b.ev[e]) == prio(b.ev[pick[r]]) && e < pick[r])) pick[r] = e;
        }
        for (int r = 0; r < P; ++r) if (pick[r] >= 0) { run.push_back(pick[r]); nodes[r].push_back(pick[r]); }
        if (run.empty()) {
            bool waiting = false;
            for (int e : frontier) waiting = waiting || (!done[e] && ready_at[e] > step);
            if (!waiting) return MPIPE_ERR_INVALID_ARG;   // cannot happen: the graph is acyclic by construction
            continue;
        }
        for (int e : run) {
            done[e] = 1; --remaining;
            for (int s : succ[e]) {
                ready_at[s] = std::max(ready_at[s], step + 1);
                if (--indeg[s] == 0) frontier.push_back(s);
            }
        }
        frontier.erase(std::remove_if(frontier.begin(), frontier.end(), [&](int e) { return done[e] != 0; }), frontier.end());
    }
    // each rank's events follow nodes(r): Sequence edges between neighbours that are not ordered already by one edge
    for (int r = 0; r < P; ++r)
        for (size_t i = 1; i < nodes[r].size(); ++i) {
            const int a = nodes[r][i - 1], c = nodes[r][i];
            bool have = false;
            for (int s : succ[a]) have = have || s == c;
            if (!have) b.add_edge(a, c, MPIPE_EDGE_SEQUENCE);
        }

    *n_events = n;
    *n_edges = int(b.ed.size());
    node_offsets[0] = 0;
    for (int r = 0; r < P; ++r) node_offsets[r + 1] = node_offsets[r] + int(nodes[r].size());
    if (n > events_cap || int(b.ed.size()) > edges_cap || events == nullptr || edges == nullptr || node_order == nullptr)
        return MPIPE_ERR_WORKSPACE;   // the counts say what is needed
    std::copy(b.ev.begin(), b.ev.end(), events);
    std::copy(b.ed.begin(), b.ed.end(), edges);
    for (int r = 0; r < P; ++r) std::copy(nodes[r].begin(), nodes[r].end(), node_order + node_offsets[r]);
    return MPIPE_OK;
}

int32_t mpipe_order_makespan(const mpipe_event_t* events, int32_t n_events, const mpipe_edge_t* edges, int32_t n_edges,
                             const double* cost, int32_t n_ranks, double* makespan, double* start, double* bubble) {
    if (events == nullptr || (n_edges > 0 && edges == nullptr) || cost == nullptr || makespan == nullptr || n_events < 0 || n_edges < 0)
        return MPIPE_ERR_INVALID_ARG;
    std::vector<int> indeg(n_events, 0);
    std::vector<std::vector<int>> succ(n_events);
    for (int i = 0; i < n_edges; ++i) {
        if (edges[i].src < 0 || edges[i].src >= n_events || edges[i].dst < 0 || edges[i].dst >= n_events) return MPIPE_ERR_INDEX;
        succ[edges[i].src].push_back(edges[i].dst);
        ++indeg[edges[i].dst];
    }
    std::vector<double> st(n_events, 0.0);
    std::vector<int> queue;
    for (int e = 0; e < n_events; ++e) {
        if (!(cost[e] >= 0.0)) return MPIPE_ERR_INVALID_ARG;
        if (indeg[e] == 0) queue.push_back(e);
    }
    double T = 0.0;
    size_t head = 0;
    while (head < queue.size()) {
        const int e = queue[head++];
        const double end = st[e] + cost[e];
        T = std::max(T, end);
        for (int s : succ[e]) {
            st[s] = std::max(st[s], end);
            if (--indeg[s] == 0) queue.push_back(s);
        }
    }
    if (int(queue.size()) != n_events) return MPIPE_ERR_INVALID_ARG;   // a cycle: not an order graph
    *makespan = T;
    if (start != nullptr) std::copy(st.begin(), st.end(), start);
    if (bubble != nullptr) {
        for (int r = 0; r < n_ranks; ++r) bubble[r] = T;
        for (int e = 0; e < n_events; ++e)
            if (events[e].rank >= 0 && events[e].rank < n_ranks) bubble[events[e].rank] -= cost[e];
    }
    return MPIPE_OK;
}

}  // extern "C"
