// Host-side cost model of the transpose schedule (Section 4.3): roofline cost of a compute event,
// alpha-beta cost of a collective, warm-up slack under 1F1B, and the ByMicrobatch owner map -- the greedy
// min-max assignment of encoder microbatches to pipeline ranks against their warm-up slack.  Plain
// double arithmetic on the host; nothing here touches the device.
#include <algorithm>
#include <numeric>
#include <vector>
#include "common.h"

extern "C" {

int32_t mpipe_event_cost(double flops, double bytes, double peak_flops, double peak_bw, double* cost) {
    if (cost == nullptr || !(flops >= 0) || !(bytes >= 0) || !(peak_flops > 0) || !(peak_bw > 0)) return MPIPE_ERR_INVALID_ARG;
    *cost = std::max(flops / peak_flops, bytes / peak_bw);
    return MPIPE_OK;
}

int32_t mpipe_coll_cost(double alpha, double beta, double payload_bytes, double* cost) {
    if (cost == nullptr || !(alpha >= 0) || !(beta >= 0) || !(payload_bytes >= 0)) return MPIPE_ERR_INVALID_ARG;
    *cost = alpha + beta * payload_bytes;
    return MPIPE_OK;
}

int32_t mpipe_encoder_attn_work(const int32_t* patch_counts, int32_t n_seg, int32_t n_heads, int32_t head_dim,
                                int32_t mode, double* fwd_flops, double* fwd_bytes, double* bwd_flops,
                                double* bwd_bytes) {
    if (n_seg < 0 || (n_seg > 0 && patch_counts == nullptr) || n_heads <= 0 || head_dim <= 0) return MPIPE_ERR_INVALID_ARG;
    if (mode != MPIPE_ENC_FROZEN && mode != MPIPE_ENC_TRAINED) return MPIPE_ERR_INVALID_ARG;
    if (fwd_flops == nullptr || fwd_bytes == nullptr || bwd_flops == nullptr || bwd_bytes == nullptr) return MPIPE_ERR_INVALID_ARG;
    double sum_n = 0, sum_n2 = 0;
    for (int32_t i = 0; i < n_seg; ++i) {
        if (patch_counts[i] < 0) return MPIPE_ERR_INVALID_ARG;
        sum_n += patch_counts[i];
        sum_n2 += double(patch_counts[i]) * patch_counts[i];
    }
    const double hd = double(n_heads) * head_dim;
    const bool trained = (mode == MPIPE_ENC_TRAINED);
    *fwd_flops = 4.0 * hd * sum_n2;                                                        // S = QK^T and O = PV
    *fwd_bytes = sum_n * n_heads * (8.0 * head_dim + (trained ? 4.0 : 0.0));               // Q, K, V, O (+ LSE)
    *bwd_flops = trained ? 10.0 * hd * sum_n2 : 0.0;                                       // five contractions
    *bwd_bytes = trained ? sum_n * n_heads * (16.0 * head_dim + 16.0) : 0.0;               // 5 reads, 3 writes, LSE, Delta
    return MPIPE_OK;
}

int32_t mpipe_warmup_slack_1f1b(int32_t n_ranks, double stage_fwd_cost, double seam_cost, double* slack) {
    if (n_ranks <= 0 || slack == nullptr || !(stage_fwd_cost >= 0) || !(seam_cost >= 0)) return MPIPE_ERR_INVALID_ARG;
    for (int32_t r = 0; r < n_ranks; ++r) slack[r] = r * (stage_fwd_cost + seam_cost);
    return MPIPE_OK;
}

int32_t mpipe_owner_map(const double* enc_cost, int32_t n_microbatches, const double* warmup_slack, int32_t n_ranks,
                        int32_t* owner, double* enc_work, double* spill, double* max_spill) {
    if (n_microbatches < 0 || n_ranks <= 0 || (n_microbatches > 0 && (enc_cost == nullptr || owner == nullptr)) ||
        warmup_slack == nullptr || enc_work == nullptr || spill == nullptr || max_spill == nullptr)
        return MPIPE_ERR_INVALID_ARG;
    for (int32_t m = 0; m < n_microbatches; ++m)
        if (!(enc_cost[m] >= 0)) return MPIPE_ERR_INVALID_ARG;
    for (int32_t r = 0; r < n_ranks; ++r) {
        if (!(warmup_slack[r] >= 0)) return MPIPE_ERR_INVALID_ARG;
        enc_work[r] = 0.0;
    }
    std::vector<int32_t> order(static_cast<size_t>(n_microbatches));
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return enc_cost[a] > enc_cost[b]; });
    for (int32_t m : order) {   // heaviest encode first, into the rank with the most warm-up slack left
        int32_t best = 0;
        double best_left = warmup_slack[0] - enc_work[0];
        for (int32_t r = 1; r < n_ranks; ++r) {
            const double left = warmup_slack[r] - enc_work[r];
            if (left > best_left) {
                best_left = left;
                best = r;
            }
        }
        owner[m] = best;
        enc_work[best] += enc_cost[m];
    }
    *max_spill = 0.0;
    for (int32_t r = 0; r < n_ranks; ++r) {
        spill[r] = std::max(0.0, enc_work[r] - warmup_slack[r]);
        *max_spill = std::max(*max_spill, spill[r]);
    }
    return MPIPE_OK;
}

}  // extern "C"
