// The rest of the packed encoder layer around the attention kernels: LayerNorm (HBM-bound, one warp per
// token row) and the host-side call sequence of the whole pre-norm block
//     x1 = x + (attn(LN1(x) Wqkv^T + bqkv)) Wo^T + bo ;  y = x1 + GELU(LN2(x1) W1^T + b1) W2^T + b2
// which is what one Fwd(enc, r, m) event of the transpose schedule executes (Section 4.2).  The projections
// are mpipe_linear_fwd (tcgen05), attention is mpipe_varlen_attn_fwd on strided views of the packed QKV matrix.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <algorithm>

#include "common.h"
#include "gelu.cuh"

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
                                                   int32_t n_heads, int32_t head_dim, float sin_sign) {
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
    // sin_sign = -1 turns by the opposite angle: the transpose of the rotation, i.e. its backward
    const float sn[8] = {sin_sign * s0.x, sin_sign * s0.y, sin_sign * s0.z, sin_sign * s0.w,
                         sin_sign * s1.x, sin_sign * s1.y, sin_sign * s1.z, sin_sign * s1.w};
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

// LayerNorm backward.  With xhat = (x - mean) rstd and g = dy gamma:  dx = rstd (g - mean(g) - xhat mean(g xhat)) + dres,
// dgamma += sum_t dy xhat, dbeta += sum_t dy.  One warp per row as in the forward; a block of four warps walks rows
// blockIdx.x * 4 + warp, + gridDim.x * 4, ...  Each warp keeps its own column sums in shared memory (plain
// read-modify-write: a lane owns its columns, a warp handles one row at a time), so registers hold one row only and
// several blocks fit an SM; at the end the four copies are added and each column costs one global atomic per block
// (same-address atomics serialise in L2, so the grid is kept to a few blocks per SM).
template <int kChunks>
__global__ void __launch_bounds__(128) layernorm_bwd_kernel(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ dy,
                                                            const __nv_bfloat16* __restrict__ gamma, const __nv_bfloat16* __restrict__ dres,
                                                            __nv_bfloat16* __restrict__ dx, float* __restrict__ dgamma,
                                                            float* __restrict__ dbeta, int32_t T, int32_t hidden, int64_t ldx,
                                                            int64_t lddy, int64_t ldr, int64_t lddx, float eps) {
    extern __shared__ float red[];   // [4 warps][2][kChunks * 256]
    constexpr int kCols = kChunks * 256;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_chunks = hidden >> 3;
    float* my_g = red + warp * 2 * kCols;
    float* my_b = my_g + kCols;
    for (int i = threadIdx.x; i < 4 * 2 * kCols; i += 128) red[i] = 0.f;
    __syncthreads();
    const uint4* g4 = reinterpret_cast<const uint4*>(gamma);
    for (int row = blockIdx.x * 4 + warp; row < T; row += gridDim.x * 4) {
        const uint4* xr = reinterpret_cast<const uint4*>(x + int64_t(row) * ldx);
        const uint4* dr = reinterpret_cast<const uint4*>(dy + int64_t(row) * lddy);
        const uint4* rr = dres != nullptr ? reinterpret_cast<const uint4*>(dres + int64_t(row) * ldr) : nullptr;
        uint4 xq[kChunks], dq[kChunks], rq[kChunks];
#pragma unroll
        for (int i = 0; i < kChunks; ++i) {   // every load of the row is issued before the first use
            const int c = lane + 32 * i;
            const bool in = c < n_chunks;
            xq[i] = in ? xr[c] : make_uint4(0u, 0u, 0u, 0u);
            dq[i] = in ? dr[c] : make_uint4(0u, 0u, 0u, 0u);
            rq[i] = (in && rr != nullptr) ? rr[c] : make_uint4(0u, 0u, 0u, 0u);
        }
        float xv[kChunks][8];
        float sum = 0.f;
#pragma unroll
        for (int i = 0; i < kChunks; ++i) {
            const uint32_t w[4] = {xq[i].x, xq[i].y, xq[i].z, xq[i].w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                xv[i][2 * j] = __uint_as_float(w[j] << 16);
                xv[i][2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
                sum += xv[i][2 * j] + xv[i][2 * j + 1];   // chunks past the row hold zeros
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        const float mean = sum / float(hidden);
        float sq = 0.f;
#pragma unroll
        for (int i = 0; i < kChunks; ++i)
            if (lane + 32 * i < n_chunks)
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float d = xv[i][j] - mean;
                    sq = fmaf(d, d, sq);
                }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
        const float rstd = rsqrtf(sq / float(hidden) + eps);
        float gv[kChunks][8];
        float s1 = 0.f, s2 = 0.f;   // sum g, sum g xhat
#pragma unroll
        for (int i = 0; i < kChunks; ++i) {
            const int c = lane + 32 * i;
            if (c < n_chunks) {
                const uint4 gq = __ldg(g4 + c);
                const uint32_t w[4] = {dq[i].x, dq[i].y, dq[i].z, dq[i].w}, gw[4] = {gq.x, gq.y, gq.z, gq.w};
                float4* pg = reinterpret_cast<float4*>(my_g + c * 8);
                float4* pb = reinterpret_cast<float4*>(my_b + c * 8);
                float4 ag[2] = {pg[0], pg[1]}, ab[2] = {pb[0], pb[1]};
                float* fg = reinterpret_cast<float*>(ag);
                float* fb = reinterpret_cast<float*>(ab);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float d = (j & 1) ? __uint_as_float(w[j >> 1] & 0xffff0000u) : __uint_as_float(w[j >> 1] << 16);
                    const float gm = (j & 1) ? __uint_as_float(gw[j >> 1] & 0xffff0000u) : __uint_as_float(gw[j >> 1] << 16);
                    const float xh = (xv[i][j] - mean) * rstd;
                    xv[i][j] = xh;
                    gv[i][j] = d * gm;
                    s1 += gv[i][j];
                    s2 = fmaf(gv[i][j], xh, s2);
                    fg[j] = fmaf(d, xh, fg[j]);
                    fb[j] += d;
                }
                pg[0] = ag[0]; pg[1] = ag[1];
                pb[0] = ab[0]; pb[1] = ab[1];
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            s1 += __shfl_xor_sync(0xffffffffu, s1, o);
            s2 += __shfl_xor_sync(0xffffffffu, s2, o);
        }
        const float m1 = s1 / float(hidden), m2 = s2 / float(hidden);
        uint4* outr = reinterpret_cast<uint4*>(dx + int64_t(row) * lddx);
#pragma unroll
        for (int i = 0; i < kChunks; ++i) {
            const int c = lane + 32 * i;
            if (c < n_chunks) {
                const uint32_t rw[4] = {rq[i].x, rq[i].y, rq[i].z, rq[i].w};
                uint32_t o[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float lo = rstd * (gv[i][2 * j] - m1 - xv[i][2 * j] * m2) + __uint_as_float(rw[j] << 16);
                    const float hi = rstd * (gv[i][2 * j + 1] - m1 - xv[i][2 * j + 1] * m2) + __uint_as_float(rw[j] & 0xffff0000u);
                    const __nv_bfloat162 pk = __floats2bfloat162_rn(lo, hi);
                    o[j] = *reinterpret_cast<const uint32_t*>(&pk);
                }
                outr[c] = make_uint4(o[0], o[1], o[2], o[3]);
            }
        }
    }
    __syncthreads();
    for (int col = threadIdx.x; col < hidden; col += 128) {
        float sg = 0.f, sb = 0.f;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            sg += red[w * 2 * kCols + col];
            sb += red[w * 2 * kCols + kCols + col];
        }
        atomicAdd(dgamma + col, sg);
        atomicAdd(dbeta + col, sb);
    }
}

// out[n] += sum_t a[t, n] (fp32): the bias gradient of a projection.  A block is 32 chunk lanes (8 columns each) x 8 row
// lanes over one group of 256 columns and one slice of the rows, four rows in flight per thread; the row lanes are added
// in shared memory, so a column costs one global atomic per block (same-address atomics serialise in L2).
__global__ void __launch_bounds__(256) colsum_kernel(const __nv_bfloat16* __restrict__ a, float* __restrict__ out, int32_t T, int32_t N,
                                                     int64_t lda, int32_t n_groups, int32_t n_slices) {
    __shared__ float red[8][256];
    const int cl = threadIdx.x & 31, rl = threadIdx.x >> 5;
    const int group = blockIdx.x % n_groups, slice = blockIdx.x / n_groups;
    const int chunk = group * 32 + cl;
    const bool in = chunk * 8 < N;
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    const __nv_bfloat16* base = a + chunk * 8;
    const int stride = n_slices * 8;
    for (int row = slice * 8 + rl; row < T && in; row += 4 * stride) {
        uint4 q[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int r = row + u * stride;
            q[u] = r < T ? *reinterpret_cast<const uint4*>(base + int64_t(r) * lda) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const uint32_t w[4] = {q[u].x, q[u].y, q[u].z, q[u].w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                acc[2 * j] += __uint_as_float(w[j] << 16);
                acc[2 * j + 1] += __uint_as_float(w[j] & 0xffff0000u);
            }
        }
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) red[rl][cl * 8 + j] = acc[j];
    __syncthreads();
    const int col = group * 256 + threadIdx.x;
    if (col < N) {
        float sacc = 0.f;
#pragma unroll
        for (int r = 0; r < 8; ++r) sacc += red[r][threadIdx.x];
        atomicAdd(out + col, sacc);
    }
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
                                                                           sin_table, n_tokens, n_heads, head_dim, 1.0f);
    return cudaGetLastError() == cudaSuccess ? MPIPE_OK : MPIPE_ERR_CUDA;
}

int32_t mpipe_rope_apply_bwd(void* dqk, int64_t tok_stride, int64_t k_offset, const float* cos_table, const float* sin_table,
                             int32_t n_tokens, int32_t n_heads, int32_t head_dim, void* stream) {
    using namespace mpipe;
    if (n_tokens < 0 || n_heads <= 0 || head_dim <= 0) return MPIPE_ERR_INVALID_ARG;
    if (n_tokens == 0) return MPIPE_OK;
    if (dqk == nullptr || cos_table == nullptr || sin_table == nullptr) return MPIPE_ERR_INVALID_ARG;
    if ((head_dim % 16) != 0 || (tok_stride % 8) != 0 || (k_offset % 8) != 0) return MPIPE_ERR_UNSUPPORTED;
    if (!aligned16(dqk) || !aligned16(cos_table) || !aligned16(sin_table)) return MPIPE_ERR_UNSUPPORTED;
    const int64_t total = int64_t(n_tokens) * 2 * n_heads * (head_dim / 16);
    const int64_t blocks = (total + 255) / 256;
    if (blocks > 0x7fffffffLL) return MPIPE_ERR_UNSUPPORTED;
    rope_kernel<<<int(blocks), 256, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<__nv_bfloat16*>(dqk), tok_stride, k_offset, cos_table,
                                                                           sin_table, n_tokens, n_heads, head_dim, -1.0f);
    return cudaGetLastError() == cudaSuccess ? MPIPE_OK : MPIPE_ERR_CUDA;
}

int32_t mpipe_layernorm_bwd(const void* x, const void* dy, const void* gamma, const void* dres, void* dx, float* dgamma, float* dbeta,
                            int32_t n_tokens, int32_t hidden, int64_t ldx, int64_t lddy, int64_t ldr, int64_t lddx, float eps,
                            void* stream) {
    using namespace mpipe;
    if (n_tokens < 0 || hidden <= 0 || !(eps >= 0.f)) return MPIPE_ERR_INVALID_ARG;
    if (n_tokens == 0) return MPIPE_OK;
    if (x == nullptr || dy == nullptr || gamma == nullptr || dx == nullptr || dgamma == nullptr || dbeta == nullptr) return MPIPE_ERR_INVALID_ARG;
    if (ldx < hidden || lddy < hidden || lddx < hidden || (dres != nullptr && ldr < hidden)) return MPIPE_ERR_INVALID_ARG;
    if ((hidden % 8) != 0 || hidden > kLnMaxChunks * 256 || (ldx % 8) != 0 || (lddy % 8) != 0 || (lddx % 8) != 0 ||
        (dres != nullptr && (ldr % 8) != 0))
        return MPIPE_ERR_UNSUPPORTED;
    if (!aligned16(x) || !aligned16(dy) || !aligned16(gamma) || !aligned16(dres) || !aligned16(dx)) return MPIPE_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int grid = std::min(cdiv(n_tokens, 4), sm_count() * 6);
    const int chunks = cdiv(hidden, 256);
#define MPIPE_LNB_LAUNCH(C)                                                                                                    \
    do {                                                                                                                       \
        cudaFuncSetAttribute(layernorm_bwd_kernel<C>, cudaFuncAttributeMaxDynamicSharedMemorySize, 4 * 2 * (C) * 256 * 4);      \
        layernorm_bwd_kernel<C><<<grid, 128, 4 * 2 * (C) * 256 * 4, st>>>(                                                      \
            static_cast<const __nv_bfloat16*>(x), static_cast<const __nv_bfloat16*>(dy), static_cast<const __nv_bfloat16*>(gamma), \
            static_cast<const __nv_bfloat16*>(dres), static_cast<__nv_bfloat16*>(dx), dgamma, dbeta, n_tokens, hidden, ldx, lddy, \
            ldr, lddx, eps);                                                                                                   \
    } while (0)
    if (chunks <= 1) MPIPE_LNB_LAUNCH(1);
    else if (chunks <= 2) MPIPE_LNB_LAUNCH(2);
    else if (chunks <= 4) MPIPE_LNB_LAUNCH(4);
    else if (chunks <= 5) MPIPE_LNB_LAUNCH(5);
    else MPIPE_LNB_LAUNCH(kLnMaxChunks);
#undef MPIPE_LNB_LAUNCH
    return cudaGetLastError() == cudaSuccess ? MPIPE_OK : MPIPE_ERR_CUDA;
}

int32_t mpipe_colsum_accumulate(const void* a, float* out, int32_t n_tokens, int32_t n_cols, int64_t lda, void* stream) {
    using namespace mpipe;
    if (n_tokens < 0 || n_cols <= 0) return MPIPE_ERR_INVALID_ARG;
    if (n_tokens == 0) return MPIPE_OK;
    if (a == nullptr || out == nullptr || lda < n_cols) return MPIPE_ERR_INVALID_ARG;
    if ((n_cols % 8) != 0 || (lda % 8) != 0 || !aligned16(a)) return MPIPE_ERR_UNSUPPORTED;
    const int n_groups = cdiv(n_cols, 256);
    const int n_slices = std::max(1, std::min(cdiv(n_tokens, 8), (sm_count() * 6) / n_groups));
    colsum_kernel<<<n_groups * n_slices, 256, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<const __nv_bfloat16*>(a), out, n_tokens,
                                                                                      n_cols, lda, n_groups, n_slices);
    return cudaGetLastError() == cudaSuccess ? MPIPE_OK : MPIPE_ERR_CUDA;
}

size_t mpipe_encoder_layer_workspace_bytes(int32_t n_tokens, int32_t hidden, int32_t ffn) {
    using namespace mpipe;
    if (n_tokens <= 0 || hidden <= 0 || ffn <= 0) return 0;
    const size_t t = size_t(n_tokens);
    // normalised rows (reused by both norms), packed QKV, attention output, x1, MLP hidden GELU(u), and u itself (kept by a
    // trained forward for the backward; one size serves both modes)
    return align256(t * hidden * 2) + align256(t * 3 * hidden * 2) + align256(t * hidden * 2) + align256(t * hidden * 2) +
           2 * align256(t * ffn * 2);
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
    uint8_t* fc1 = ws;                ws += align256(t * ffn * 2);
    uint8_t* ubuf = ws;
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
    if (mode == MPIPE_ENC_TRAINED) {   // the backward needs the pre-activation: the same launch stores it beside GELU(u)
        if ((rc = linear_fwd_gelu_keep_preact(norm, w->w_fc1, w->b_fc1, fc1, ubuf, n_tokens, ffn, hidden, hidden, hidden, ffn, ffn,
                                              status_buf, stream)) != MPIPE_OK) return rc;
    } else if ((rc = mpipe_linear_fwd(norm, w->w_fc1, w->b_fc1, nullptr, fc1, n_tokens, ffn, hidden, hidden, hidden, 0, ffn,
                                      MPIPE_LINEAR_GELU, status_buf, stream)) != MPIPE_OK) {
        return rc;
    }
    return mpipe_linear_fwd(fc1, w->w_fc2, w->b_fc2, x1, y, n_tokens, hidden, ffn, ffn, ffn, hidden, hidden, 0, status_buf, stream);
}

size_t mpipe_encoder_layer_bwd_workspace_bytes(int32_t n_tokens, int32_t hidden, int32_t n_heads, int32_t ffn) {
    using namespace mpipe;
    if (n_tokens <= 0 || hidden <= 0 || n_heads <= 0 || ffn <= 0 || (hidden % n_heads) != 0) return 0;
    const size_t t = size_t(n_tokens);
    // dL/du, dL/dqkv, dL/dx1, one [T, hidden] temporary, the attention backward's own workspace
    return align256(t * ffn * 2) + align256(t * 3 * hidden * 2) + 2 * align256(t * hidden * 2) +
           align256(mpipe_attn_workspace_bytes(n_tokens, n_heads, hidden / n_heads, MPIPE_ENC_TRAINED));
}

int32_t mpipe_encoder_layer_bwd(const void* dy, const void* x, void* dx, const mpipe_layer_weights_t* w, const mpipe_layer_grads_t* g,
                                int32_t n_tokens, int32_t hidden, int32_t n_heads, int32_t ffn, const int32_t* cu_seqlens_dev,
                                int32_t n_seg, int32_t max_seqlen, const mpipe_work_item_t* bwd_items_dev, int32_t n_bwd_items,
                                float softmax_scale, float ln_eps, const float* rope_cos, const float* rope_sin, int32_t mode,
                                const float* lse, void* fwd_workspace, void* workspace, size_t workspace_bytes, int32_t* status_buf,
                                void* stream) {
    using namespace mpipe;
    if (mode != MPIPE_ENC_FROZEN && mode != MPIPE_ENC_TRAINED) return MPIPE_ERR_INVALID_ARG;
    if (mode == MPIPE_ENC_FROZEN) return MPIPE_OK;   // Lemma 1: a frozen encoder has no backward events
    if (n_tokens < 0 || hidden <= 0 || n_heads <= 0 || ffn <= 0 || w == nullptr || g == nullptr) return MPIPE_ERR_INVALID_ARG;
    if (n_tokens == 0) return MPIPE_OK;
    if (dy == nullptr || x == nullptr || dx == nullptr || lse == nullptr || fwd_workspace == nullptr || (hidden % n_heads) != 0)
        return MPIPE_ERR_INVALID_ARG;
    if ((rope_cos == nullptr) != (rope_sin == nullptr)) return MPIPE_ERR_INVALID_ARG;
    if (workspace == nullptr || workspace_bytes < mpipe_encoder_layer_bwd_workspace_bytes(n_tokens, hidden, n_heads, ffn))
        return MPIPE_ERR_WORKSPACE;
    if (((reinterpret_cast<uintptr_t>(workspace) | reinterpret_cast<uintptr_t>(fwd_workspace)) & 255u) != 0) return MPIPE_ERR_UNSUPPORTED;
    const int32_t head_dim = hidden / n_heads;
    const size_t t = size_t(n_tokens);
    const int64_t h = hidden, h3 = 3 * int64_t(hidden), f = ffn;
    // what the forward left in its workspace: LN output (stale), packed q|k|v (q, k rotated), attention output, x1, GELU(u), u
    uint8_t* fw = static_cast<uint8_t*>(fwd_workspace);
    uint8_t* norm = fw;               fw += align256(t * hidden * 2);
    uint8_t* qkv = fw;                fw += align256(t * 3 * hidden * 2);
    uint8_t* attn = fw;               fw += align256(t * hidden * 2);
    uint8_t* x1 = fw;                 fw += align256(t * hidden * 2);
    uint8_t* act = fw;                fw += align256(t * ffn * 2);
    uint8_t* ubuf = fw;
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    uint8_t* dubuf = ws;              ws += align256(t * ffn * 2);
    uint8_t* dqkv = ws;               ws += align256(t * 3 * hidden * 2);
    uint8_t* dx1 = ws;                ws += align256(t * hidden * 2);
    uint8_t* tmp = ws;                ws += align256(t * hidden * 2);
    uint8_t* attn_ws = ws;
    const size_t attn_ws_bytes = mpipe_attn_workspace_bytes(n_tokens, n_heads, head_dim, MPIPE_ENC_TRAINED);
    int32_t rc;
#define MPIPE_TRY(call) do { if ((rc = (call)) != MPIPE_OK) return rc; } while (0)
    // ---- MLP branch: y = x1 + GELU(m W1^T + b1) W2^T + b2, m = LN2(x1)
    MPIPE_TRY(mpipe_layernorm_fwd(x1, w->ln2_gamma, w->ln2_beta, norm, n_tokens, hidden, h, h, ln_eps, stream));                 // m
    MPIPE_TRY(mpipe_linear_wgrad(dy, act, g->w_fc2, n_tokens, hidden, ffn, h, f, f, status_buf, stream));                          // dW2 += dy^T GELU(u)
    MPIPE_TRY(mpipe_colsum_accumulate(dy, g->b_fc2, n_tokens, hidden, h, stream));
    MPIPE_TRY(mpipe_linear_dgrad(dy, w->w_fc2, ubuf, nullptr, dubuf, n_tokens, hidden, ffn, h, f, f, 0, f, status_buf, stream));    // du = (dy W2) o GELU'(u)
    MPIPE_TRY(mpipe_linear_wgrad(dubuf, norm, g->w_fc1, n_tokens, ffn, hidden, f, h, h, status_buf, stream));                     // dW1 += du^T m
    MPIPE_TRY(mpipe_colsum_accumulate(dubuf, g->b_fc1, n_tokens, ffn, f, stream));
    MPIPE_TRY(mpipe_linear_dgrad(dubuf, w->w_fc1, nullptr, nullptr, tmp, n_tokens, ffn, hidden, f, h, 0, 0, h, status_buf, stream)); // dm = du W1
    MPIPE_TRY(mpipe_layernorm_bwd(x1, tmp, w->ln2_gamma, dy, dx1, g->ln2_gamma, g->ln2_beta, n_tokens, hidden, h, h, h, h, ln_eps, stream)); // dx1 = dy + LN2'(dm)
    // ---- attention branch: x1 = x + o Wo^T + bo, o = attention(rope(a Wqkv^T + bqkv)), a = LN1(x)
    MPIPE_TRY(mpipe_linear_wgrad(dx1, attn, g->w_o, n_tokens, hidden, hidden, h, h, h, status_buf, stream));                       // dWo += dx1^T o
    MPIPE_TRY(mpipe_colsum_accumulate(dx1, g->b_o, n_tokens, hidden, h, stream));
    MPIPE_TRY(mpipe_linear_dgrad(dx1, w->w_o, nullptr, nullptr, tmp, n_tokens, hidden, hidden, h, h, 0, 0, h, status_buf, stream)); // do = dx1 Wo
    MPIPE_TRY(mpipe_varlen_attn_bwd(tmp, qkv, qkv + size_t(hidden) * 2, qkv + size_t(hidden) * 4, attn, lse, dqkv, dqkv + size_t(hidden) * 2,
                                    dqkv + size_t(hidden) * 4, h3, head_dim, h, head_dim, h3, head_dim, cu_seqlens_dev, n_seg, n_tokens,
                                    max_seqlen, bwd_items_dev, n_bwd_items, n_heads, head_dim, softmax_scale, MPIPE_ENC_TRAINED, attn_ws,
                                    attn_ws_bytes, status_buf, stream));
    if (rope_cos != nullptr)
        MPIPE_TRY(mpipe_rope_apply_bwd(dqkv, h3, hidden, rope_cos, rope_sin, n_tokens, n_heads, head_dim, stream));
    MPIPE_TRY(mpipe_layernorm_fwd(x, w->ln1_gamma, w->ln1_beta, norm, n_tokens, hidden, h, h, ln_eps, stream));                    // a (recomputed)
    MPIPE_TRY(mpipe_linear_wgrad(dqkv, norm, g->w_qkv, n_tokens, 3 * hidden, hidden, h3, h, h, status_buf, stream));               // dWqkv += dqkv^T a
    MPIPE_TRY(mpipe_colsum_accumulate(dqkv, g->b_qkv, n_tokens, 3 * hidden, h3, stream));
    MPIPE_TRY(mpipe_linear_dgrad(dqkv, w->w_qkv, nullptr, nullptr, tmp, n_tokens, 3 * hidden, hidden, h3, h, 0, 0, h, status_buf, stream)); // da = dqkv Wqkv
    MPIPE_TRY(mpipe_layernorm_bwd(x, tmp, w->ln1_gamma, dx1, dx, g->ln1_gamma, g->ln1_beta, n_tokens, hidden, h, h, h, h, ln_eps, stream)); // dx = dx1 + LN1'(da)
#undef MPIPE_TRY
    return MPIPE_OK;
}

// ---- the whole encoder: n_layers identical blocks, one after the other (what Fwd(enc, r, m) / Bwd(enc, r, m) run)
size_t mpipe_encoder_workspace_bytes(int32_t n_layers, int32_t n_tokens, int32_t hidden, int32_t ffn, int32_t mode) {
    using namespace mpipe;
    if (n_layers <= 0 || n_tokens <= 0 || hidden <= 0 || ffn <= 0) return 0;
    const size_t per_layer = mpipe_encoder_layer_workspace_bytes(n_tokens, hidden, ffn);
    const size_t act = align256(size_t(n_tokens) * hidden * 2);
    // FROZEN: one layer workspace reused + two ping-pong activations.  TRAINED: every layer's workspace and input are kept.
    return mode == MPIPE_ENC_TRAINED ? size_t(n_layers) * (per_layer + act) : per_layer + 2 * act;
}

int32_t mpipe_encoder_fwd(const void* x, void* y, const mpipe_layer_weights_t* layers, int32_t n_layers, int32_t n_tokens,
                          int32_t hidden, int32_t n_heads, int32_t ffn, const int32_t* cu_seqlens_dev, int32_t n_seg,
                          int32_t max_seqlen, const mpipe_work_item_t* fwd_items_dev, int32_t n_fwd_items, float softmax_scale,
                          float ln_eps, const float* rope_cos, const float* rope_sin, int32_t mode, float* lse, void* workspace,
                          size_t workspace_bytes, int32_t* status_buf, void* stream) {
    using namespace mpipe;
    if (n_layers <= 0 || layers == nullptr || n_tokens < 0) return MPIPE_ERR_INVALID_ARG;
    if (mode != MPIPE_ENC_FROZEN && mode != MPIPE_ENC_TRAINED) return MPIPE_ERR_INVALID_ARG;
    if (n_tokens == 0) return MPIPE_OK;
    if (x == nullptr || y == nullptr || (mode == MPIPE_ENC_TRAINED && lse == nullptr)) return MPIPE_ERR_INVALID_ARG;
    if (workspace == nullptr || workspace_bytes < mpipe_encoder_workspace_bytes(n_layers, n_tokens, hidden, ffn, mode)) return MPIPE_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return MPIPE_ERR_UNSUPPORTED;
    const size_t per_layer = mpipe_encoder_layer_workspace_bytes(n_tokens, hidden, ffn);
    const size_t act = align256(size_t(n_tokens) * hidden * 2);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    const void* in = x;
    for (int l = 0; l < n_layers; ++l) {
        // TRAINED: layer l's workspace at l * (per_layer + act), its OUTPUT (= layer l+1's input) right behind it
        uint8_t* lws = mode == MPIPE_ENC_TRAINED ? ws + size_t(l) * (per_layer + act) : ws;
        void* out = (l == n_layers - 1) ? y
                    : (mode == MPIPE_ENC_TRAINED ? static_cast<void*>(lws + per_layer) : static_cast<void*>(ws + per_layer + size_t(l & 1) * act));
        float* lse_l = mode == MPIPE_ENC_TRAINED ? lse + size_t(l) * n_heads * size_t(n_tokens) : nullptr;
        const int32_t rc = mpipe_encoder_layer_fwd(in, out, layers + l, n_tokens, hidden, n_heads, ffn, cu_seqlens_dev, n_seg, max_seqlen,
                                                   fwd_items_dev, n_fwd_items, softmax_scale, ln_eps, rope_cos, rope_sin, mode, lse_l, lws,
                                                   per_layer, status_buf, stream);
        if (rc != MPIPE_OK) return rc;
        in = out;
    }
    return MPIPE_OK;
}

int32_t mpipe_encoder_bwd(const void* dy, const void* x, void* dx, const mpipe_layer_weights_t* layers, const mpipe_layer_grads_t* grads,
                          int32_t n_layers, int32_t n_tokens, int32_t hidden, int32_t n_heads, int32_t ffn,
                          const int32_t* cu_seqlens_dev, int32_t n_seg, int32_t max_seqlen, const mpipe_work_item_t* bwd_items_dev,
                          int32_t n_bwd_items, float softmax_scale, float ln_eps, const float* rope_cos, const float* rope_sin,
                          int32_t mode, const float* lse, void* fwd_workspace, void* workspace, size_t workspace_bytes,
                          int32_t* status_buf, void* stream) {
    using namespace mpipe;
    if (mode != MPIPE_ENC_FROZEN && mode != MPIPE_ENC_TRAINED) return MPIPE_ERR_INVALID_ARG;
    if (mode == MPIPE_ENC_FROZEN) return MPIPE_OK;
    if (n_layers <= 0 || layers == nullptr || grads == nullptr || n_tokens < 0) return MPIPE_ERR_INVALID_ARG;
    if (n_tokens == 0) return MPIPE_OK;
    if (dy == nullptr || x == nullptr || dx == nullptr || lse == nullptr || fwd_workspace == nullptr) return MPIPE_ERR_INVALID_ARG;
    const size_t per_bwd = mpipe_encoder_layer_bwd_workspace_bytes(n_tokens, hidden, n_heads, ffn);
    const size_t act = align256(size_t(n_tokens) * hidden * 2);
    if (workspace == nullptr || workspace_bytes < per_bwd + 2 * act) return MPIPE_ERR_WORKSPACE;
    if (((reinterpret_cast<uintptr_t>(workspace) | reinterpret_cast<uintptr_t>(fwd_workspace)) & 255u) != 0) return MPIPE_ERR_UNSUPPORTED;
    const size_t per_layer = mpipe_encoder_layer_workspace_bytes(n_tokens, hidden, ffn);
    uint8_t* fws = static_cast<uint8_t*>(fwd_workspace);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    const void* grad_in = dy;
    for (int l = n_layers - 1; l >= 0; --l) {
        uint8_t* lws = fws + size_t(l) * (per_layer + act);
        const void* in = (l == 0) ? x : static_cast<const void*>(fws + size_t(l - 1) * (per_layer + act) + per_layer);   // layer l's input
        void* grad_out = (l == 0) ? dx : static_cast<void*>(ws + per_bwd + size_t(l & 1) * act);
        const int32_t rc = mpipe_encoder_layer_bwd(grad_in, in, grad_out, layers + l, grads + l, n_tokens, hidden, n_heads, ffn, cu_seqlens_dev,
                                                   n_seg, max_seqlen, bwd_items_dev, n_bwd_items, softmax_scale, ln_eps, rope_cos, rope_sin,
                                                   mode, lse + size_t(l) * n_heads * size_t(n_tokens), lws, ws, per_bwd, status_buf, stream);
        if (rc != MPIPE_OK) return rc;
        grad_in = grad_out;
    }
    return MPIPE_OK;
}

size_t mpipe_encoder_bwd_workspace_bytes(int32_t n_tokens, int32_t hidden, int32_t n_heads, int32_t ffn) {
    using namespace mpipe;
    const size_t per_bwd = mpipe_encoder_layer_bwd_workspace_bytes(n_tokens, hidden, n_heads, ffn);
    return per_bwd == 0 ? 0 : per_bwd + 2 * align256(size_t(n_tokens) * hidden * 2);
}

}  // extern "C"
