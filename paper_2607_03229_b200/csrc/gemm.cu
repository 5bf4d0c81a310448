// mpipe_linear_fwd: C[M, N] = epilogue(A[M, K] * W[N, K]^T), the dense projections of the packed encoder layer
// (QKV, attention output, MLP) on the token matrix [T, hidden].  bf16 operands, fp32 accumulation in TMEM.
// mpipe_linear_dgrad: dX[M, K] = epilogue(dY[M, N] * W[N, K]) -- the same kernel with the second operand read as
// [contraction][output] (an MN-major B: four 64-column atoms per stage, loaded as four TMA boxes).
// mpipe_linear_wgrad: dW[N, K] += dY[M, N]^T * X[M, K] in fp32 -- both operands MN-major (the token index is the
// contraction), the token range split over CTAs, partial tiles added with TMA reduce-add.
//
// Persistent kernel, one CTA per SM, static round-robin over 128 x 256 output tiles (n fastest, so that the
// CTAs of a wave share the few weight tiles in L2 and walk down the token rows together).
//   warp 0      TMA producer: A box [128 rows][64 k], W box [256 rows][64 k] per stage, 128-byte swizzle, 4 stages
//   warp 1      tcgen05 issuer: 4 x (M 128, N 256, K 16) smem x smem MMAs per stage into one of TWO 256-column
//               TMEM accumulators, so the epilogue of tile i overlaps the main loop of tile i + 1
//   warp 2      TMEM allocation
//   warps 4-11  epilogue: thread = output row = TMEM lane; warpgroup 0 takes columns 0..127, warpgroup 1
//               columns 128..255; 32 columns per TMEM round trip; + bias, GELU, + residual in fp32, bf16 into a
//               64-byte-swizzled [128 rows][32 columns] staging box (two per warpgroup), one TMA store per box --
//               row-per-thread global stores cost 32 L1 wavefronts per instruction and bound the K = 1024 cases
// Every mbarrier wait is bounded (status MPIPE_ERR_TIMEOUT), as in the attention kernels.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "common.h"
#include "gelu.cuh"
#include "sm100_ptx.cuh"
#include "tensormap.h"

namespace mpipe {

constexpr int kGemmBM = 128, kGemmBN = 256, kGemmBK = 64, kGemmStages = 4;
constexpr int kGemmThreads = 384;
constexpr int kGemmABytes = kGemmBM * kGemmBK * 2;   // 16 KB
constexpr int kGemmBBytes = kGemmBN * kGemmBK * 2;   // 32 KB
constexpr int kGemmStageBytes = kGemmABytes + kGemmBBytes;
constexpr int kGemmOutBox = kGemmBM * 64;            // [128 rows][32 bf16] staging box
constexpr int kGemmSmemOut = kGemmStages * kGemmStageBytes;   // 2 warpgroups x 2 boxes
constexpr int kGemmSmem = kGemmSmemOut + 4 * kGemmOutBox + 1024;
static_assert(kGemmSmem <= 227 * 1024, "shared memory budget");

struct GemmParams {
    int32_t M, N, K;
    int32_t tiles_m, tiles_n;
    const __nv_bfloat16* bias;       // [N] or null
    const __nv_bfloat16* residual;   // [M, ldr] or null
    const __nv_bfloat16* aux;        // [M, ldx] or null: pre-activation u; the result is multiplied by GELU'(u)
    int64_t ldx;
    __nv_bfloat16* C;                // [M, ldc]
    int64_t ldr, ldc;
    int32_t gelu;
    int32_t store_pre;               // with gelu: also store the pre-activation (bf16) through map_u
    int32_t splits;                  // weight gradient: parts the contraction (token) range is cut into
    int32_t* status_buf;
};

struct GemmBarriers {
    uint64_t full[kGemmStages], empty[kGemmStages], acc_full[2], acc_empty[2];
};

// kBMode 0: W tile [256 output rows][64 k], K-major (forward).  kBMode 1: W tile [64 contraction rows][256 output
// columns], MN-major: four [64][64] atoms 8 KB apart (input gradient).  kBMode 2 (weight gradient): as 1, and the first
// operand too is [64 contraction rows][128 output columns], MN-major, two atoms; work items are (tile, split) pairs and
// the fp32 result is added to the output with TMA reductions instead of being stored as bf16.
template <int kBMode>
__global__ void __launch_bounds__(kGemmThreads, 1)
linear_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_w,
                  const __grid_constant__ CUtensorMap map_c, const __grid_constant__ CUtensorMap map_u, const GemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ GemmBarriers bars;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        abort_flag = 0;
        for (int s = 0; s < kGemmStages; ++s) {
            mbar_init(&bars.full[s], 1);
            mbar_init(&bars.empty[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&bars.acc_full[a], 1);
            mbar_init(&bars.acc_empty[a], 8);
        }
        fence_mbar_init();
    }
    if (warp == 2) {
        tmem_alloc(&tmem_base_slot, 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_slot;
    const int nk = (p.K + kGemmBK - 1) / kGemmBK;
    const int n_tiles = p.tiles_m * p.tiles_n * (kBMode == 2 ? p.splits : 1);   // work items
    // work item -> output tile and range of contraction blocks
    // (weight gradient: the split index is the slow one, so that the CTAs of a wave work on the same token range and
    //  share its dY and X rows through L2)
    const int n_out_tiles = p.tiles_m * p.tiles_n;
    auto tile_of = [&](int t) { return kBMode == 2 ? t % n_out_tiles : t; };
    auto kb_lo_of = [&](int t) { return kBMode == 2 ? int((long long)(t / n_out_tiles) * nk / p.splits) : 0; };
    auto kb_hi_of = [&](int t) { return kBMode == 2 ? int((long long)(t / n_out_tiles + 1) * nk / p.splits) : nk; };

    if (warp == 0) {
        if (lane == 0) {
            prefetch_tmap(&map_a);
            prefetch_tmap(&map_w);
            uint32_t it = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x) {
                const int m0 = (tile_of(t) / p.tiles_n) * kGemmBM, n0 = (tile_of(t) % p.tiles_n) * kGemmBN;
                for (int kb = kb_lo_of(t); kb < kb_hi_of(t); ++kb, ++it) {
                    const int s = it % kGemmStages;
                    ok = mbar_wait<100>(&bars.empty[s], ((it / kGemmStages) & 1) ^ 1, &abort_flag);
                    if (!ok) break;
                    uint8_t* st = smem + s * kGemmStageBytes;
                    mbar_expect_tx(&bars.full[s], kGemmStageBytes);   // out-of-range rows / columns are zero-filled, still counted
                    if (kBMode == 2) {
#pragma unroll
                        for (int i = 0; i < kGemmBM / 64; ++i)
                            tma_load_3d(st + i * (kGemmBK * 128), &map_a, &bars.full[s], m0 + 64 * i, 0, kb * kGemmBK);
                    } else {
                        tma_load_3d(st, &map_a, &bars.full[s], kb * kGemmBK, 0, m0);
                    }
                    if (kBMode == 0) {
                        tma_load_3d(st + kGemmABytes, &map_w, &bars.full[s], kb * kGemmBK, 0, n0);
                    } else {
#pragma unroll
                        for (int i = 0; i < kGemmBN / 64; ++i)
                            tma_load_3d(st + kGemmABytes + i * (kGemmBK * 128), &map_w, &bars.full[s], n0 + 64 * i, 0, kb * kGemmBK);
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        const bool leader = elect_one();
        const uint32_t sbase = smem_u32(smem);
        constexpr uint32_t hi128 = umma_desc_hi(1024, kSwizzle128);
        constexpr uint32_t idesc = umma_idesc_bf16(kGemmBM, kGemmBN, kBMode == 2 ? 1 : 0, kBMode != 0 ? 1 : 0);
        uint32_t it = 0, tile_it = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++tile_it) {
            if (kb_lo_of(t) >= kb_hi_of(t)) { --tile_it; continue; }   // an empty split: no role touches it
            const uint32_t acc = tile_it & 1;
            ok = mbar_wait(&bars.acc_empty[acc], ((tile_it >> 1) & 1) ^ 1, &abort_flag);
            if (!ok) break;
            tc_fence_after();
            for (int kb = kb_lo_of(t); kb < kb_hi_of(t); ++kb, ++it) {
                const int s = it % kGemmStages;
                ok = mbar_wait(&bars.full[s], (it / kGemmStages) & 1, &abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a_lo = umma_desc_lo(sbase + s * kGemmStageBytes, kBMode == 2 ? kGemmBK * 128 : 0);
                constexpr uint32_t a_step = kBMode == 2 ? 128 : 2;
                const uint32_t b_lo = umma_desc_lo(sbase + s * kGemmStageBytes + kGemmABytes, kBMode == 0 ? 0 : kGemmBK * 128);
                constexpr uint32_t b_step = kBMode == 0 ? 2 : 128;   // one K-step: 32 bytes along a row, or 16 rows of 128 bytes
                if (leader) {
#pragma unroll
                    for (int ks = 0; ks < kGemmBK / 16; ++ks)
                        umma_ss(tmem + acc * kGemmBN, umma_desc(a_lo + ks * a_step, hi128), umma_desc(b_lo + ks * b_step, hi128), idesc,
                                (kb > kb_lo_of(t) || ks > 0) ? 1u : 0u);
                    umma_commit(&bars.empty[s]);
                }
            }
            if (!ok) break;
            if (leader) umma_commit(&bars.acc_full[acc]);
        }
        __syncwarp();
    } else if (warp >= 4) {
        const int wg = (warp - 4) >> 2;                 // column half of the tile
        const int r = ((warp & 3) << 5) | lane;         // output row inside the tile = TMEM lane
        const uint32_t lane_base = uint32_t((warp & 3) * 32) << 16;
        const int wt = tid - (4 + 4 * wg) * 32;         // thread index inside the warpgroup
        uint8_t* boxes = smem + kGemmSmemOut + wg * 2 * kGemmOutBox;
        uint32_t tile_it = 0, box_it = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < n_tiles; t += gridDim.x, ++tile_it) {
            // no early exit: the warpgroup meets at named barriers, so after a time-out it keeps walking empty tiles
            if (kb_lo_of(t) >= kb_hi_of(t)) { --tile_it; continue; }
            const uint32_t acc = tile_it & 1;
            const int m0 = (tile_of(t) / p.tiles_n) * kGemmBM;
            const int m = m0 + r;
            const int n_base = (tile_of(t) % p.tiles_n) * kGemmBN + wg * (kGemmBN / 2);
            const bool row_ok = m < p.M;
            const __nv_bfloat16* rrow = (p.residual != nullptr && row_ok) ? p.residual + int64_t(m) * p.ldr : nullptr;
            // the residual row is fetched one 32-column chunk ahead (each thread reads its own row: latency, not bandwidth)
            uint4 res[4];
            auto load_res = [&](int c0) {
#pragma unroll
                for (int g8 = 0; g8 < 4; ++g8) {
                    const int n = n_base + c0 + 8 * g8;
                    res[g8] = (rrow != nullptr && n < p.N) ? __ldg(reinterpret_cast<const uint4*>(rrow + n)) : make_uint4(0u, 0u, 0u, 0u);
                }
            };
            const __nv_bfloat16* xrow = (p.aux != nullptr && row_ok) ? p.aux + int64_t(m) * p.ldx : nullptr;
            uint4 aux[4];
            auto load_aux = [&](int c0) {
#pragma unroll
                for (int g8 = 0; g8 < 4; ++g8) {
                    const int n = n_base + c0 + 8 * g8;
                    aux[g8] = (xrow != nullptr && n < p.N) ? __ldg(reinterpret_cast<const uint4*>(xrow + n)) : make_uint4(0u, 0u, 0u, 0u);
                }
            };
            if (p.residual != nullptr) load_res(0);
            if (p.aux != nullptr) load_aux(0);
            if (ok) ok = mbar_wait(&bars.acc_full[acc], (tile_it >> 1) & 1, &abort_flag);
            tc_fence_after();
#pragma unroll 1
            for (int c0 = 0; c0 < kGemmBN / 2; c0 += 32, ++box_it) {
                uint32_t v[32];
                uint32_t out[16];
                uint32_t pre[16];   // pre-activation of the same 32 columns (only with store_pre)
                uint4 rcur[4];
                uint4 xcur[4];
                if (p.residual != nullptr) {
#pragma unroll
                    for (int g8 = 0; g8 < 4; ++g8) rcur[g8] = res[g8];
                    if (c0 + 32 < kGemmBN / 2) load_res(c0 + 32);
                }
                if (p.aux != nullptr) {
#pragma unroll
                    for (int g8 = 0; g8 < 4; ++g8) xcur[g8] = aux[g8];
                    if (c0 + 32 < kGemmBN / 2) load_aux(c0 + 32);
                }
                if (ok) {
                    tmem_ld32(tmem + lane_base + acc * kGemmBN + wg * (kGemmBN / 2) + c0, v);
                    tmem_wait_ld();
                    if (c0 + 32 == kGemmBN / 2) {   // this thread's part of the accumulator is in registers
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&bars.acc_empty[acc]);
                    }
#pragma unroll
                    for (int g8 = 0; g8 < 4; ++g8) {   // 8 columns = 16 bytes of output
                        const int n = n_base + c0 + 8 * g8;
                        const bool col_ok = n < p.N;     // N is a multiple of 8; the store clips what lies outside
                        float f[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) f[i] = __uint_as_float(v[8 * g8 + i]);
                        if (p.bias != nullptr && col_ok) {
                            const uint4 b4 = __ldg(reinterpret_cast<const uint4*>(p.bias + n));
                            const uint32_t bw[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                f[2 * i] += __uint_as_float(bw[i] << 16);
                                f[2 * i + 1] += __uint_as_float(bw[i] & 0xffff0000u);
                            }
                        }
                        if (p.gelu) {
                            if (p.store_pre) {
#pragma unroll
                                for (int i = 0; i < 4; ++i) pre[4 * g8 + i] = pack_bf16(f[2 * i], f[2 * i + 1]);
                            }
#pragma unroll
                            for (int i = 0; i < 8; ++i) f[i] = gelu_erf(f[i]);   // of the fp32 value, in both modes
                        }
                        if (p.aux != nullptr) {
                            const uint32_t xw[4] = {xcur[g8].x, xcur[g8].y, xcur[g8].z, xcur[g8].w};
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                f[2 * i] *= gelu_erf_grad(__uint_as_float(xw[i] << 16));
                                f[2 * i + 1] *= gelu_erf_grad(__uint_as_float(xw[i] & 0xffff0000u));
                            }
                        }
                        if (p.residual != nullptr) {
                            const uint32_t rw[4] = {rcur[g8].x, rcur[g8].y, rcur[g8].z, rcur[g8].w};
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                f[2 * i] += __uint_as_float(rw[i] << 16);
                                f[2 * i + 1] += __uint_as_float(rw[i] & 0xffff0000u);
                            }
                        }
#pragma unroll
                        for (int i = 0; i < 4; ++i) out[4 * g8 + i] = pack_bf16(f[2 * i], f[2 * i + 1]);
                    }
                }
                if (kBMode == 2) {   // fp32 partial tile: one [128 rows][32 fp32] box (128-byte swizzle), added to the output
                    if (wt == 0) bulk_wait_group_read<0>();
                    named_barrier_sync(1 + wg, 128);
                    if (ok) {
#pragma unroll
                        for (int ch = 0; ch < 8; ++ch)
                            *reinterpret_cast<uint4*>(boxes + r * 128 + ((ch ^ (r & 7)) << 4)) =
                                make_uint4(v[4 * ch], v[4 * ch + 1], v[4 * ch + 2], v[4 * ch + 3]);
                    }
                    fence_async_smem();
                    named_barrier_sync(1 + wg, 128);
                    if (ok && wt == 0) {
                        tma_reduce_add_3d(&map_c, boxes, n_base + c0, 0, m0);
                        bulk_commit_group();
                    }
                    continue;
                }
                // one [128 rows][32 bf16] box per output: the result, and before it the pre-activation if asked for
                auto emit = [&](const CUtensorMap* map, const uint32_t (&w)[16]) {
                    uint8_t* box = boxes + (box_it & 1) * kGemmOutBox;
                    if (wt == 0) bulk_wait_group_read<1>();   // the store issued two boxes ago has read this box
                    named_barrier_sync(1 + wg, 128);
                    if (ok) {
#pragma unroll
                        for (int g8 = 0; g8 < 4; ++g8)
                            *reinterpret_cast<uint4*>(box + r * 64 + ((g8 ^ ((r >> 1) & 3)) << 4)) =
                                make_uint4(w[4 * g8], w[4 * g8 + 1], w[4 * g8 + 2], w[4 * g8 + 3]);
                    }
                    fence_async_smem();
                    named_barrier_sync(1 + wg, 128);
                    if (ok && wt == 0) {
                        tma_store_3d(map, box, n_base + c0, 0, m0);
                        bulk_commit_group();
                    }
                };
                if (p.gelu && p.store_pre) {
                    emit(&map_u, pre);
                    ++box_it;
                }
                emit(&map_c, out);
            }
        }
        if (wt == 0) bulk_wait_group<0>();   // shared memory must outlive the copy engine's reads
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 2) tmem_dealloc(tmem, 512);
    if (tid == 0 && abort_flag) report_status(p.status_buf, MPIPE_ERR_TIMEOUT, int32_t(blockIdx.x));
}

}  // namespace mpipe

namespace mpipe {

// Shared host side of the two entry points.  n_out / n_contract are the output columns and the contraction length.
// `pre` (optional, forward with GELU only): bf16 [M, ldp] that receives the pre-activation a W^T + bias as well.
static int32_t launch_linear(int b_mode, const void* a, const void* w, const void* bias, const void* residual, const void* aux,
                             void* c, int32_t M, int32_t n_out, int32_t n_contract, int64_t lda, int64_t ldw, int64_t ldr,
                             int64_t ldx, int64_t ldc, int32_t gelu, int32_t* status_buf, void* stream,
                             void* pre = nullptr, int64_t ldp = 0) {
    if (M < 0 || n_out <= 0 || n_contract <= 0) return MPIPE_ERR_INVALID_ARG;
    if (M == 0) return MPIPE_OK;
    if (a == nullptr || w == nullptr || c == nullptr) return MPIPE_ERR_INVALID_ARG;
    if ((n_out % 8) != 0 || (n_contract % 8) != 0) return MPIPE_ERR_UNSUPPORTED;
    const int64_t w_cols = b_mode == 0 ? n_contract : n_out;
    if (lda < n_contract || ldw < w_cols || ldc < n_out || (residual != nullptr && ldr < n_out) || (aux != nullptr && ldx < n_out))
        return MPIPE_ERR_INVALID_ARG;
    if ((lda % 8) != 0 || (ldw % 8) != 0 || (ldc % 8) != 0 || (residual != nullptr && (ldr % 8) != 0) || (aux != nullptr && (ldx % 8) != 0))
        return MPIPE_ERR_UNSUPPORTED;
    if (!aligned16(a) || !aligned16(w) || !aligned16(c) || !aligned16(bias) || !aligned16(residual) || !aligned16(aux))
        return MPIPE_ERR_UNSUPPORTED;
    if (pre != nullptr && (b_mode != 0 || !gelu || ldp < n_out || (ldp % 8) != 0 || !aligned16(pre))) return MPIPE_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    CUtensorMap map_a, map_w, map_c, map_u;
    bool ok = make_tensor_map_thd(&map_a, a, M, 1, n_contract, lda, lda, kGemmBK, kGemmBM, 128) &&
              make_tensor_map_thd(&map_c, c, M, 1, n_out, ldc, ldc, 32, kGemmBM, 64);
    map_u = map_c;
    if (pre != nullptr) ok = ok && make_tensor_map_thd(&map_u, pre, M, 1, n_out, ldp, ldp, 32, kGemmBM, 64);
    if (b_mode == 0)   // W[n_out rows, n_contract columns]: boxes of 256 rows x 64 k
        ok = ok && make_tensor_map_thd(&map_w, w, n_out, 1, n_contract, ldw, ldw, kGemmBK, kGemmBN, 128);
    else               // W[n_contract rows, n_out columns]: boxes of 64 contraction rows x 64 output columns
        ok = ok && make_tensor_map_thd(&map_w, w, n_contract, 1, n_out, ldw, ldw, 64, kGemmBK, 128);
    if (!ok) return MPIPE_ERR_CUDA;
    GemmParams p;
    p.M = M; p.N = n_out; p.K = n_contract;
    p.tiles_m = cdiv(M, kGemmBM);
    p.tiles_n = cdiv(n_out, kGemmBN);
    p.bias = static_cast<const __nv_bfloat16*>(bias);
    p.residual = static_cast<const __nv_bfloat16*>(residual);
    p.aux = static_cast<const __nv_bfloat16*>(aux);
    p.C = static_cast<__nv_bfloat16*>(c);
    p.ldr = ldr; p.ldx = ldx; p.ldc = ldc;
    p.gelu = gelu;
    p.store_pre = pre != nullptr ? 1 : 0;
    p.splits = 1;
    p.status_buf = status_buf;
    const long long tiles = (long long)p.tiles_m * p.tiles_n;
    const int grid = int(tiles < sm_count() ? tiles : sm_count());
    profile_start(kProfileLinear, st);
    if (b_mode == 0) {
        if (!ensure_dynamic_smem<linear_kernel<0>>(kGemmSmem)) return MPIPE_ERR_CUDA;
        linear_kernel<0><<<grid, kGemmThreads, kGemmSmem, st>>>(map_a, map_w, map_c, map_u, p);
    } else {
        if (!ensure_dynamic_smem<linear_kernel<1>>(kGemmSmem)) return MPIPE_ERR_CUDA;
        linear_kernel<1><<<grid, kGemmThreads, kGemmSmem, st>>>(map_a, map_w, map_c, map_u, p);
    }
    profile_stop(kProfileLinear, st);
    return cudaGetLastError() == cudaSuccess ? MPIPE_OK : MPIPE_ERR_CUDA;
}

// dW[n_rows, n_cols] (fp32) += dY[tokens, n_rows]^T X[tokens, n_cols]
static int32_t launch_wgrad(const void* dy, const void* x, float* dw, int32_t tokens, int32_t n_rows, int32_t n_cols, int64_t lddy,
                            int64_t ldx, int64_t lddw, int32_t* status_buf, void* stream) {
    if (tokens < 0 || n_rows <= 0 || n_cols <= 0) return MPIPE_ERR_INVALID_ARG;
    if (tokens == 0) return MPIPE_OK;
    if (dy == nullptr || x == nullptr || dw == nullptr || lddy < n_rows || ldx < n_cols || lddw < n_cols) return MPIPE_ERR_INVALID_ARG;
    if ((n_rows % 8) != 0 || (n_cols % 8) != 0 || (lddy % 8) != 0 || (ldx % 8) != 0 || (lddw % 4) != 0) return MPIPE_ERR_UNSUPPORTED;
    if (!aligned16(dy) || !aligned16(x) || !aligned16(dw)) return MPIPE_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    CUtensorMap map_a, map_w, map_c;
    if (!make_tensor_map_thd(&map_a, dy, tokens, 1, n_rows, lddy, lddy, 64, kGemmBK, 128) ||
        !make_tensor_map_thd(&map_w, x, tokens, 1, n_cols, ldx, ldx, 64, kGemmBK, 128) ||
        !make_tensor_map_thd(&map_c, dw, n_rows, 1, n_cols, lddw, lddw, 32, kGemmBM, 128, 4))
        return MPIPE_ERR_CUDA;
    GemmParams p;
    p.M = n_rows; p.N = n_cols; p.K = tokens;
    p.tiles_m = cdiv(n_rows, kGemmBM);
    p.tiles_n = cdiv(n_cols, kGemmBN);
    p.bias = nullptr; p.residual = nullptr; p.aux = nullptr; p.C = nullptr;
    p.ldr = p.ldx = p.ldc = 0;
    p.gelu = 0;
    p.store_pre = 0;
    p.status_buf = status_buf;
    // split the token range so that (tiles x splits) fills whole waves of the SMs; more splits mean more reduction traffic
    const int sms = sm_count(), tiles = p.tiles_m * p.tiles_n, nk = cdiv(tokens, kGemmBK);
    int best = 1;
    double best_score = -1.0;
    for (int sp = 1; sp <= 32 && sp <= nk; ++sp) {
        const long long items = (long long)tiles * sp;
        const double eff = double(items) / double(((items + sms - 1) / sms) * sms);
        const double score = eff - 0.004 * sp;
        if (score > best_score) { best_score = score; best = sp; }
    }
    p.splits = best;
    const long long items = (long long)tiles * p.splits;
    const int grid = int(items < sms ? items : sms);
    if (!ensure_dynamic_smem<linear_kernel<2>>(kGemmSmem)) return MPIPE_ERR_CUDA;
    profile_start(kProfileLinear, st);
    linear_kernel<2><<<grid, kGemmThreads, kGemmSmem, st>>>(map_a, map_w, map_c, map_c, p);
    profile_stop(kProfileLinear, st);
    return cudaGetLastError() == cudaSuccess ? MPIPE_OK : MPIPE_ERR_CUDA;
}

// fc1 of a TRAINED layer forward: act = GELU(a W^T + bias) and pre = a W^T + bias from ONE accumulator, so that the
// activation is computed from the same fp32 value as in the FROZEN forward (freezing changes no forward bit).
int32_t linear_fwd_gelu_keep_preact(const void* a, const void* w, const void* bias, void* act, void* pre, int32_t M, int32_t N,
                                    int32_t K, int64_t lda, int64_t ldw, int64_t ldact, int64_t ldpre, int32_t* status_buf,
                                    void* stream) {
    return launch_linear(0, a, w, bias, nullptr, nullptr, act, M, N, K, lda, ldw, 0, 0, ldact, 1, status_buf, stream, pre, ldpre);
}

}  // namespace mpipe

extern "C" {

int32_t mpipe_linear_wgrad(const void* dy, const void* x, float* dw, int32_t n_tokens, int32_t N, int32_t K, int64_t lddy,
                           int64_t ldx, int64_t lddw, int32_t* status_buf, void* stream) {
    return mpipe::launch_wgrad(dy, x, dw, n_tokens, N, K, lddy, ldx, lddw, status_buf, stream);
}

int32_t mpipe_linear_fwd(const void* a, const void* w, const void* bias, const void* residual, void* c, int32_t M,
                         int32_t N, int32_t K, int64_t lda, int64_t ldw, int64_t ldr, int64_t ldc, int32_t flags,
                         int32_t* status_buf, void* stream) {
    if ((flags & ~(MPIPE_LINEAR_GELU)) != 0) return MPIPE_ERR_INVALID_ARG;
    return mpipe::launch_linear(0, a, w, bias, residual, nullptr, c, M, N, K, lda, ldw, ldr, 0, ldc,
                                (flags & MPIPE_LINEAR_GELU) ? 1 : 0, status_buf, stream);
}

int32_t mpipe_linear_dgrad(const void* dy, const void* w, const void* gelu_input, const void* residual, void* dx, int32_t M,
                           int32_t N, int32_t K, int64_t lddy, int64_t ldw, int64_t ldu, int64_t ldr, int64_t lddx,
                           int32_t* status_buf, void* stream) {
    return mpipe::launch_linear(1, dy, w, nullptr, residual, gelu_input, dx, M, K, N, lddy, ldw, ldr, ldu, lddx, 0, status_buf,
                                stream);
}

}  // extern "C"
