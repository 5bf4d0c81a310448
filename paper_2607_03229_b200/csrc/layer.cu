// The rest of the packed encoder layer around the attention kernels: LayerNorm (HBM-bound, one warp per
// token row) and the host-side call sequence of the whole pre-norm block
//     x1 = x + (attn(LN1(x) Wqkv^T + bqkv)) Wo^T + bo ;  y = x1 + GELU(LN2(x1) W1^T + b1) W2^T + b2
// which is what one Fwd(enc, r, m) event of the transpose schedule executes (Section 4.2).  The projections
// are mpipe_linear_fwd (tcgen05), attention is mpipe_varlen_attn_fwd on strided views of the packed QKV matrix.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "common.h"

namespace mpipe {

constexpr int kLnMaxChunks = 8;   // 16-byte chunks per lane: hidden <= 8 * 32 * 8 = 2048

// y[t, :] = (x[t, :] - mean) * rsqrt(var + eps) * gamma + beta, biased variance, fp32 statistics (two passes over
// registers, so no cancellation).  One warp per row; lane l owns chunks l, l + 32, ...
template <int kChunks>
__global__ void __launch_bounds__(256) layernorm_kernel(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ gamma,
                                                        const __nv_bfloat16* __restrict__ beta, __nv_bfloat16* __restrict__ y,
                                                        int32_t T, int32_t hidden, int64_t ldx, int64_t ldy, float eps) {
    const int row = blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= T) return;
    const int n_chunks = hidden >> 3;
    const uint4* xr = reinterpret_cast<const uint4*>(x + int64_t(row) * ldx);
    float v[kChunks][8];
    float sum = 0.f;
#pragma unroll
    for (int i = 0; i < kChunks; ++i) {
        const int c = lane + 32 * i;
        if (c < n_chunks) {
            const uint4 q = xr[c];
            const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                v[i][2 * j] = __uint_as_float(w[j] << 16);
                v[i][2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
                sum += v[i][2 * j] + v[i][2 * j + 1];
            }
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    const float mean = sum / float(hidden);
    float sq = 0.f;
#pragma unroll
    for (int i = 0; i < kChunks; ++i) {
        if (lane + 32 * i < n_chunks) {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const float d = v[i][j] - mean;
                sq = fmaf(d, d, sq);
            }
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
    const float rstd = rsqrtf(sq / float(hidden) + eps);
    uint4* yr = reinterpret_cast<uint4*>(y + int64_t(row) * ldy);
    const uint4* g4 = reinterpret_cast<const uint4*>(gamma);
    const uint4* b4 = reinterpret_cast<const uint4*>(beta);
#pragma unroll
    for (int i = 0; i < kChunks; ++i) {
        const int c = lane + 32 * i;
        if (c < n_chunks) {
            const uint4 g = __ldg(g4 + c), b = __ldg(b4 + c);
            const uint32_t gw[4] = {g.x, g.y, g.z, g.w}, bw[4] = {b.x, b.y, b.z, b.w};
            uint32_t o[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float lo = (v[i][2 * j] - mean) * rstd * __uint_as_float(gw[j] << 16) + __uint_as_float(bw[j] << 16);
                const float hi = (v[i][2 * j + 1] - mean) * rstd * __uint_as_float(gw[j] & 0xffff0000u) +
                                 __uint_as_float(bw[j] & 0xffff0000u);
                const __nv_bfloat162 pk = __floats2bfloat162_rn(lo, hi);
                o[j] = *reinterpret_cast<const uint32_t*>(&pk);
            }
            yr[c] = make_uint4(o[0], o[1], o[2], o[3]);
        }
    }
}

// Rotary position encoding in the rotate-half form, in place on q and k inside the packed projection:
// (x1, x2) -> (x1 cos - x2 sin, x2 cos + x1 sin) for x1 = x[0 .. D/2), x2 = x[D/2 .. D), angles per token and pair.
// One thread per (token, q|k, head, 8-pair chunk): 2 x 16 bytes in, 2 x 16 bytes out, 2 x 32 bytes of table.
__global__ void __launch_bounds__(256) rope_kernel(__nv_bfloat16* __restrict__ qk, int64_t tok_stride, int64_t k_offset,
                                                   const float* __restrict__ cos_t, const float* __restrict__ sin_t, int32_t T,
                                                   int32_t n_heads, int32_t head_dim) {
    const int half = head_dim >> 1, chunks = half >> 3;
    const int64_t idx = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    const int64_t total = int64_t(T) * 2 * n_heads * chunks;
    if (idx >= total) return;
    const int c = int(idx % chunks);
    const int h = int((idx / chunks) % n_heads);
    const int which = int((idx / (int64_t(chunks) * n_heads)) & 1);
    const int64_t t = idx / (int64_t(chunks) * n_heads * 2);
    __nv_bfloat16* x = qk + t * tok_stride + which * k_offset + int64_t(h) * head_dim + c * 8;
    const uint4 a = *reinterpret_cast<const uint4*>(x), b = *reinterpret_cast<const uint4*>(x + half);
    const float4* cp = reinterpret_cast<const float4*>(cos_t + t * half + c * 8);
    const float4* sp = reinterpret_cast<const float4*>(sin_t + t * half + c * 8);
    const float4 c0 = __ldg(cp), c1 = __ldg(cp + 1), s0 = __ldg(sp), s1 = __ldg(sp + 1);
    const float cs[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
    const float sn[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
    const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
    uint32_t oa[4], ob[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const float x1l = __uint_as_float(aw[j] << 16), x1h = __uint_as_float(aw[j] & 0xffff0000u);
        const float x2l = __uint_as_float(bw[j] << 16), x2h = __uint_as_float(bw[j] & 0xffff0000u);
        const __nv_bfloat162 o1 = __floats2bfloat162_rn(x1l * cs[2 * j] - x2l * sn[2 * j], x1h * cs[2 * j + 1] - x2h * sn[2 * j + 1]);
        const __nv_bfloat162 o2 = __floats2bfloat162_rn(x2l * cs[2 * j] + x1l * sn[2 * j], x2h * cs[2 * j + 1] + x1h * sn[2 * j + 1]);
        oa[j] = *reinterpret_cast<const uint32_t*>(&o1);
        ob[j] = *reinterpret_cast<const uint32_t*>(&o2);
    }
    *reinterpret_cast<uint4*>(x) = make_uint4(oa[0], oa[1], oa[2], oa[3]);
    *reinterpret_cast<uint4*>(x + half) = make_uint4(ob[0], ob[1], ob[2], ob[3]);
}

static size_t align256(size_t v) { return (v + 255) & ~size_t(255); }

}  // namespace mpipe

extern "C" {

int32_t mpipe_layernorm_fwd(const void* x, const void* gamma, const void* beta, void* y, int32_t n_tokens, int32_t hidden,
                            int64_t ldx, int64_t ldy, float eps, void* stream) {
    using namespace mpipe;
    if (n_tokens < 0 || hidden <= 0 || !(eps >= 0.f)) return MPIPE_ERR_INVALID_ARG;
    if (n_tokens == 0) return MPIPE_OK;
    if (x == nullptr || gamma == nullptr || beta == nullptr || y == nullptr || ldx < hidden || ldy < hidden) return MPIPE_ERR_INVALID_ARG;
    if ((hidden % 8) != 0 || hidden > kLnMaxChunks * 256 || (ldx % 8) != 0 || (ldy % 8) != 0) return MPIPE_ERR_UNSUPPORTED;
    if (!aligned16(x) || !aligned16(y) || !aligned16(gamma) || !aligned16(beta)) return MPIPE_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int grid = cdiv(n_tokens, 8);
    const auto* xp = static_cast<const __nv_bfloat16*>(x);
    const auto* gp = static_cast<const __nv_bfloat16*>(gamma);
    const auto* bp = static_cast<const __nv_bfloat16*>(beta);
    auto* yp = static_cast<__nv_bfloat16*>(y);
    profile_start(kProfileLayerNorm, st);
    const int chunks = cdiv(hidden, 256);   // 16-byte chunks per lane: instantiate what the row length needs, not the maximum
#define MPIPE_LN_LAUNCH(C) layernorm_kernel<C><<<grid, 256, 0, st>>>(xp, gp, bp, yp, n_tokens, hidden, ldx, ldy, eps)
    if (chunks <= 1) MPIPE_LN_LAUNCH(1);
    else if (chunks <= 2) MPIPE_LN_LAUNCH(2);
    else if (chunks <= 3) MPIPE_LN_LAUNCH(3);
    else if (chunks <= 4) MPIPE_LN_LAUNCH(4);
    else if (chunks <= 5) MPIPE_LN_LAUNCH(5);
    else if (chunks <= 6) MPIPE_LN_LAUNCH(6);
    else MPIPE_LN_LAUNCH(kLnMaxChunks);
#undef MPIPE_LN_LAUNCH
    profile_stop(kProfileLayerNorm, st);
    return cudaGetLastError() == cudaSuccess ? MPIPE_OK : MPIPE_ERR_CUDA;
}

int32_t mpipe_rope_apply(void* qk, int64_t tok_stride, int64_t k_offset, const float* cos_table, const float* sin_table,
                         int32_t n_tokens, int32_t n_heads, int32_t head_dim, void* stream) {
    using namespace mpipe;
    if (n_tokens < 0 || n_heads <= 0 || head_dim <= 0) return MPIPE_ERR_INVALID_ARG;
    if (n_tokens == 0) return MPIPE_OK;
    if (qk == nullptr || cos_table == nullptr || sin_table == nullptr) return MPIPE_ERR_INVALID_ARG;
    if ((head_dim % 16) != 0 || (tok_stride % 8) != 0 || (k_offset % 8) != 0) return MPIPE_ERR_UNSUPPORTED;
    if (!aligned16(qk) || !aligned16(cos_table) || !aligned16(sin_table)) return MPIPE_ERR_UNSUPPORTED;
    const int64_t total = int64_t(n_tokens) * 2 * n_heads * (head_dim / 16);
    const int64_t blocks = (total + 255) / 256;
    if (blocks > 0x7fffffffLL) return MPIPE_ERR_UNSUPPORTED;
    rope_kernel<<<int(blocks), 256, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<__nv_bfloat16*>(qk), tok_stride, k_offset, cos_table,
                                                                           sin_table, n_tokens, n_heads, head_dim);
    return cudaGetLastError() == cudaSuccess ? MPIPE_OK : MPIPE_ERR_CUDA;
}

size_t mpipe_encoder_layer_workspace_bytes(int32_t n_tokens, int32_t hidden, int32_t ffn) {
    using namespace mpipe;
    if (n_tokens <= 0 || hidden <= 0 || ffn <= 0) return 0;
    const size_t t = size_t(n_tokens);
    // normalised rows (reused by both norms), packed QKV, attention output, x1, MLP hidden
    return align256(t * hidden * 2) + align256(t * 3 * hidden * 2) + align256(t * hidden * 2) + align256(t * hidden * 2) +
           align256(t * ffn * 2);
}

int32_t mpipe_encoder_layer_fwd(const void* x, void* y, const mpipe_layer_weights_t* w, int32_t n_tokens, int32_t hidden,
                                int32_t n_heads, int32_t ffn, const int32_t* cu_seqlens_dev, int32_t n_seg, int32_t max_seqlen,
                                const mpipe_work_item_t* fwd_items_dev, int32_t n_fwd_items, float softmax_scale, float ln_eps,
                                const float* rope_cos, const float* rope_sin, int32_t mode, float* lse, void* workspace,
                                size_t workspace_bytes, int32_t* status_buf, void* stream) {
    using namespace mpipe;
    if (n_tokens < 0 || hidden <= 0 || n_heads <= 0 || ffn <= 0 || w == nullptr) return MPIPE_ERR_INVALID_ARG;
    if (mode != MPIPE_ENC_FROZEN && mode != MPIPE_ENC_TRAINED) return MPIPE_ERR_INVALID_ARG;
    if (n_tokens == 0) return MPIPE_OK;
    if (x == nullptr || y == nullptr || (hidden % n_heads) != 0) return MPIPE_ERR_INVALID_ARG;
    const int32_t head_dim = hidden / n_heads;
    if (workspace == nullptr || workspace_bytes < mpipe_encoder_layer_workspace_bytes(n_tokens, hidden, ffn)) return MPIPE_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return MPIPE_ERR_UNSUPPORTED;
    const size_t t = size_t(n_tokens);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    uint8_t* norm = ws;               ws += align256(t * hidden * 2);
    uint8_t* qkv = ws;                ws += align256(t * 3 * hidden * 2);
    uint8_t* attn = ws;               ws += align256(t * hidden * 2);
    uint8_t* x1 = ws;                 ws += align256(t * hidden * 2);
    uint8_t* fc1 = ws;
    int32_t rc;
    if ((rc = mpipe_layernorm_fwd(x, w->ln1_gamma, w->ln1_beta, norm, n_tokens, hidden, hidden, hidden, ln_eps, stream)) != MPIPE_OK) return rc;
    if ((rc = mpipe_linear_fwd(norm, w->w_qkv, w->b_qkv, nullptr, qkv, n_tokens, 3 * hidden, hidden, hidden, hidden, 0,
                               3 * int64_t(hidden), 0, status_buf, stream)) != MPIPE_OK) return rc;
    if ((rope_cos == nullptr) != (rope_sin == nullptr)) return MPIPE_ERR_INVALID_ARG;
    if (rope_cos != nullptr &&
        (rc = mpipe_rope_apply(qkv, 3 * int64_t(hidden), hidden, rope_cos, rope_sin, n_tokens, n_heads, head_dim, stream)) != MPIPE_OK)
        return rc;
    const uint8_t* q = qkv;
    const uint8_t* k = qkv + size_t(hidden) * 2;
    const uint8_t* v = qkv + size_t(hidden) * 4;
    if ((rc = mpipe_varlen_attn_fwd(q, k, v, attn, lse, 3 * int64_t(hidden), head_dim, hidden, head_dim, cu_seqlens_dev, n_seg,
                                    n_tokens, max_seqlen, fwd_items_dev, n_fwd_items, n_heads, head_dim, softmax_scale, mode,
                                    status_buf, stream)) != MPIPE_OK) return rc;
    if ((rc = mpipe_linear_fwd(attn, w->w_o, w->b_o, x, x1, n_tokens, hidden, hidden, hidden, hidden, hidden, hidden, 0,
                               status_buf, stream)) != MPIPE_OK) return rc;
    if ((rc = mpipe_layernorm_fwd(x1, w->ln2_gamma, w->ln2_beta, norm, n_tokens, hidden, hidden, hidden, ln_eps, stream)) != MPIPE_OK) return rc;
    if ((rc = mpipe_linear_fwd(norm, w->w_fc1, w->b_fc1, nullptr, fc1, n_tokens, ffn, hidden, hidden, hidden, 0, ffn,
                               MPIPE_LINEAR_GELU, status_buf, stream)) != MPIPE_OK) return rc;
    return mpipe_linear_fwd(fc1, w->w_fc2, w->b_fc2, x1, y, n_tokens, hidden, ffn, ffn, ffn, hidden, hidden, 0, status_buf, stream);
}

}  // extern "C"
