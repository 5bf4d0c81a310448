// mpipe_varlen_attn_bwd (placeholder until the tcgen05 backward lands).
#include "common.h"

extern "C" {

int32_t mpipe_bwd_tile_rows(void) { return 128; }

size_t mpipe_attn_workspace_bytes(int32_t total_tokens, int32_t n_heads, int32_t head_dim, int32_t mode) {
    if (mode != MPIPE_ENC_TRAINED || total_tokens <= 0 || n_heads <= 0 || head_dim <= 0) return 0;
    const size_t dq = (size_t(total_tokens) * n_heads * head_dim * 4 + 255) & ~size_t(255);
    const size_t delta = (size_t(total_tokens) * n_heads * 4 + 255) & ~size_t(255);
    return dq + delta;
}

int32_t mpipe_varlen_attn_bwd(const void*, const void*, const void*, const void*, const void*, const float*, void*,
                              void*, void*, int64_t, int64_t, int64_t, int64_t, int64_t, int64_t, const int32_t*,
                              int32_t, int32_t, int32_t, const mpipe_work_item_t*, int32_t, int32_t, int32_t, float,
                              int32_t mode, void*, size_t, int32_t*, void*) {
    if (mode == MPIPE_ENC_FROZEN) return MPIPE_OK;
    return MPIPE_ERR_UNSUPPORTED;
}

}  // extern "C"
