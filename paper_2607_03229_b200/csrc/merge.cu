// mpipe_merge_tokens / mpipe_merge_tokens_bwd: the local half of the Replicated->Sharded seam of
// Table 2.  Forward ("Gather"): encoder row i overwrites row positions[i] of the LLM input-embedding
// buffer.  Backward ("Scatter", only when the encoder is trainable, Lemma 1 gate (i)): gradient row
// positions[i] is read back into encoder row i.  Both are pure row copies: HBM-bound, bit-exact.
//
// One kernel serves both directions.  Work is the flat list of 16-byte chunks of all rows; every
// thread moves kUnroll chunks per step with all its loads issued before the first store, so that
// each SM keeps tens of kilobytes in flight.  Source rows are read once (streaming loads); the
// indexed side goes through the position table, which stays in L1/L2.
#include "common.h"

namespace mpipe {

constexpr int kMergeThreads = 256;
constexpr int kMergeUnroll = 4;

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.cs.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// kScatter = true : dst[pos[i]] = src[i]   (forward merge)
// kScatter = false: dst[i] = src[pos[i]]   (backward merge)
template <bool kScatter>
__global__ void __launch_bounds__(kMergeThreads)
merge_rows_kernel(const uint4* __restrict__ src, int64_t src_row_stride16, uint4* __restrict__ dst,
                  int64_t dst_row_stride16, const int32_t* __restrict__ positions, int32_t n_rows,
                  int32_t n_indexed_rows, int32_t chunks_per_row, int32_t* status_buf) {
    const int64_t total = int64_t(n_rows) * chunks_per_row;
    const int64_t step = int64_t(gridDim.x) * kMergeThreads * kMergeUnroll;
    for (int64_t base = int64_t(blockIdx.x) * kMergeThreads * kMergeUnroll + threadIdx.x; base < total; base += step) {
        uint4 val[kMergeUnroll];
        int64_t dst_off[kMergeUnroll];
#pragma unroll
        for (int u = 0; u < kMergeUnroll; ++u) {
            const int64_t c = base + int64_t(u) * kMergeThreads;
            dst_off[u] = -1;
            if (c < total) {
                const int32_t row = int32_t(c / chunks_per_row);
                const int32_t col = int32_t(c - int64_t(row) * chunks_per_row);
                const int32_t p = __ldg(positions + row);
                if (p < 0 || p >= n_indexed_rows) {
                    if (col == 0) report_status(status_buf, MPIPE_ERR_INDEX, row);
                } else {
                    const int64_t s = kScatter ? int64_t(row) : int64_t(p);
                    const int64_t d = kScatter ? int64_t(p) : int64_t(row);
                    val[u] = ld_stream(src + s * src_row_stride16 + col);
                    dst_off[u] = d * dst_row_stride16 + col;
                }
            }
        }
#pragma unroll
        for (int u = 0; u < kMergeUnroll; ++u)
            if (dst_off[u] >= 0) dst[dst_off[u]] = val[u];
    }
}

static int32_t merge_launch(bool scatter, const void* src, int64_t src_stride, void* dst, int64_t dst_stride,
                            const int32_t* positions_dev, int32_t n_enc_tokens, int32_t n_llm_tokens, int32_t hidden,
                            int32_t* status_buf, void* stream) {
    if (n_enc_tokens < 0 || n_llm_tokens < 0 || hidden <= 0) return MPIPE_ERR_INVALID_ARG;
    if (n_enc_tokens == 0) return MPIPE_OK;
    if (src == nullptr || dst == nullptr || positions_dev == nullptr) return MPIPE_ERR_INVALID_ARG;
    if ((hidden & 7) != 0 || (src_stride & 7) != 0 || (dst_stride & 7) != 0) return MPIPE_ERR_INVALID_ARG;
    if (src_stride < hidden || dst_stride < hidden) return MPIPE_ERR_INVALID_ARG;
    if (!aligned16(src) || !aligned16(dst)) return MPIPE_ERR_INVALID_ARG;
    const int32_t chunks = hidden / 8;
    const int64_t total = int64_t(n_enc_tokens) * chunks;
    const int64_t per_block = int64_t(kMergeThreads) * kMergeUnroll;
    const int64_t want = (total + per_block - 1) / per_block;
    const int64_t cap = int64_t(sm_count()) * 8 * 4;  // a few waves of 8 resident blocks per SM
    const int grid = int(want < cap ? want : cap);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    profile_start(kProfileMerge, st);
    if (scatter)
        merge_rows_kernel<true><<<grid, kMergeThreads, 0, st>>>(
            static_cast<const uint4*>(src), src_stride / 8, static_cast<uint4*>(dst), dst_stride / 8, positions_dev,
            n_enc_tokens, n_llm_tokens, chunks, status_buf);
    else
        merge_rows_kernel<false><<<grid, kMergeThreads, 0, st>>>(
            static_cast<const uint4*>(src), src_stride / 8, static_cast<uint4*>(dst), dst_stride / 8, positions_dev,
            n_enc_tokens, n_llm_tokens, chunks, status_buf);
    profile_stop(kProfileMerge, st);
    return cudaGetLastError() == cudaSuccess ? MPIPE_OK : MPIPE_ERR_CUDA;
}

}  // namespace mpipe

extern "C" {

int32_t mpipe_merge_tokens(const void* enc_tokens, int64_t enc_row_stride, void* llm_embeds, int64_t emb_row_stride,
                           const int32_t* positions_dev, int32_t n_enc_tokens, int32_t n_llm_tokens, int32_t hidden,
                           int32_t mode, int32_t* status_buf, void* stream) {
    if (mode != MPIPE_ENC_FROZEN && mode != MPIPE_ENC_TRAINED) return MPIPE_ERR_INVALID_ARG;
    return mpipe::merge_launch(true, enc_tokens, enc_row_stride, llm_embeds, emb_row_stride, positions_dev,
                               n_enc_tokens, n_llm_tokens, hidden, status_buf, stream);
}

int32_t mpipe_merge_tokens_bwd(const void* d_llm_embeds, int64_t emb_row_stride, void* d_enc, int64_t enc_row_stride,
                               const int32_t* positions_dev, int32_t n_enc_tokens, int32_t n_llm_tokens,
                               int32_t hidden, int32_t mode, int32_t* status_buf, void* stream) {
    if (mode != MPIPE_ENC_FROZEN && mode != MPIPE_ENC_TRAINED) return MPIPE_ERR_INVALID_ARG;
    if (mode == MPIPE_ENC_FROZEN) return MPIPE_OK;  // no trainable region upstream: the reverse seam does not exist
    return mpipe::merge_launch(false, d_llm_embeds, emb_row_stride, d_enc, enc_row_stride, positions_dev,
                               n_enc_tokens, n_llm_tokens, hidden, status_buf, stream);
}

}  // extern "C"
