// Host-side pieces of libmpipe_enc: the segment planner, the position validator, status strings.
#include <algorithm>
#include <numeric>
#include <vector>
#include "common.h"

namespace mpipe {

thread_local ProfileEvents g_profile[kProfileSlots];

int sm_count() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

// Tiles of every non-empty segment, longest segment first (ties: lower index first).
static int32_t emit_items(const int32_t* counts, const int32_t* cu, const std::vector<int32_t>& order,
                          int32_t tile_rows, mpipe_work_item_t* out) {
    int64_t n_items = 0;
    for (int32_t s : order) {
        const int32_t n = counts[s];
        if (n == 0) continue;
        const int32_t tiles = (n + tile_rows - 1) / tile_rows;
        if (out != nullptr) {
            for (int32_t t = 0; t < tiles; ++t) {
                mpipe_work_item_t& it = out[n_items + t];
                it.seg = s;
                it.tile = t;
                it.row_start = cu[s] + t * tile_rows;
                it.row_len = std::min(tile_rows, n - t * tile_rows);
                it.kv_start = cu[s];
                it.kv_len = n;
            }
        }
        n_items += tiles;
    }
    return static_cast<int32_t>(n_items);
}

}  // namespace mpipe

extern "C" {

int32_t mpipe_seg_plan(const int32_t* patch_counts, int32_t n_seg, int32_t fwd_tile_rows, int32_t bwd_tile_rows,
                       int32_t mode, int32_t* cu_seqlens, int32_t* total_tokens, int32_t* max_seqlen,
                       mpipe_work_item_t* fwd_items, int32_t* n_fwd_items, mpipe_work_item_t* bwd_items,
                       int32_t* n_bwd_items) {
    if (n_seg < 0 || (n_seg > 0 && patch_counts == nullptr) || cu_seqlens == nullptr || total_tokens == nullptr ||
        max_seqlen == nullptr || n_fwd_items == nullptr || n_bwd_items == nullptr)
        return MPIPE_ERR_INVALID_ARG;
    if (fwd_tile_rows <= 0 || bwd_tile_rows <= 0) return MPIPE_ERR_INVALID_ARG;
    if (mode != MPIPE_ENC_FROZEN && mode != MPIPE_ENC_TRAINED) return MPIPE_ERR_INVALID_ARG;
    int64_t acc = 0;
    int32_t mx = 0;
    for (int32_t i = 0; i < n_seg; ++i) {
        if (patch_counts[i] < 0) return MPIPE_ERR_INVALID_ARG;
        acc += patch_counts[i];
        if (acc >= (int64_t(1) << 31)) return MPIPE_ERR_INVALID_ARG;
        mx = std::max(mx, patch_counts[i]);
    }
    cu_seqlens[0] = 0;
    for (int32_t i = 0; i < n_seg; ++i) cu_seqlens[i + 1] = cu_seqlens[i] + patch_counts[i];
    *total_tokens = cu_seqlens[n_seg];
    *max_seqlen = mx;

    std::vector<int32_t> order(static_cast<size_t>(n_seg));
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(),
                     [&](int32_t a, int32_t b) { return patch_counts[a] > patch_counts[b]; });
    *n_fwd_items = mpipe::emit_items(patch_counts, cu_seqlens, order, fwd_tile_rows, fwd_items);
    *n_bwd_items = (mode == MPIPE_ENC_TRAINED)
                       ? mpipe::emit_items(patch_counts, cu_seqlens, order, bwd_tile_rows, bwd_items)
                       : 0;
    return MPIPE_OK;
}

int32_t mpipe_validate_positions(const int32_t* positions, int32_t n, int32_t n_llm_tokens) {
    if (n < 0 || n_llm_tokens < 0 || (n > 0 && positions == nullptr)) return MPIPE_ERR_INVALID_ARG;
    std::vector<uint8_t> seen(static_cast<size_t>(n_llm_tokens), 0);
    for (int32_t i = 0; i < n; ++i) {
        const int32_t p = positions[i];
        if (p < 0 || p >= n_llm_tokens) return MPIPE_ERR_INDEX;
        if (seen[p]) return MPIPE_ERR_INVALID_ARG;
        seen[p] = 1;
    }
    return MPIPE_OK;
}

const char* mpipe_status_str(int32_t status) {
    switch (status) {
        case MPIPE_OK: return "ok";
        case MPIPE_ERR_INVALID_ARG: return "invalid argument";
        case MPIPE_ERR_UNSUPPORTED: return "unsupported configuration";
        case MPIPE_ERR_WORKSPACE: return "workspace missing or too small";
        case MPIPE_ERR_CUDA: return "CUDA call failed";
        case MPIPE_ERR_TIMEOUT: return "device wait timed out";
        case MPIPE_ERR_INDEX: return "index out of range";
        default: return "unknown status";
    }
}

int32_t mpipe_version(void) { return 100; }

int32_t mpipe_set_profile_events(int32_t which, void* start_event, void* stop_event) {
    if (which < 0 || which >= mpipe::kProfileSlots) return MPIPE_ERR_INVALID_ARG;
    mpipe::g_profile[which].start = static_cast<cudaEvent_t>(start_event);
    mpipe::g_profile[which].stop = static_cast<cudaEvent_t>(stop_event);
    return MPIPE_OK;
}

}  // extern "C"
