// mpipe_varlen_attn_fwd: block-diagonal (per-image) softmax attention over a packed token sequence,
// the attention of the relocated Fwd(enc, r, m) event (Section 4.2).
//
// One persistent CTA per SM walks the (work item x head) list.  A work item is up to 256 query rows of
// one segment = two 128-row query tiles that share every K/V tile.  Warp roles:
//   warp 0      TMA producer: Q tiles once per unit, K and V tiles through a kStages-deep ring
//   warp 1      tcgen05 issuer: S_w = Q_w K^T into TMEM, O_w += P_w V with P_w read from TMEM
//   warp 2      TMEM allocation
//   warps 4-7   softmax of query tile 0 (thread = query row = TMEM lane)
//   warps 8-11  softmax of query tile 1
// The issuer interleaves the two query tiles (PV_0(j), S_0(j+1), PV_1(j), S_1(j+1)) so that the tensor
// pipe works on one tile while the other tile's softmax runs.  Softmax is online with a lazily updated
// reference maximum: the accumulator in TMEM is rescaled only when a row maximum grows by more than
// 2^8, so P stays <= 256 and almost no tile needs the rescale.  P is written back over S in TMEM as
// packed bf16 and consumed from there as the A operand of the second MMA.
//
// Every mbarrier wait is bounded; on expiry the CTA sets an abort flag, all roles drain, TMEM is freed
// and MPIPE_ERR_TIMEOUT is reported through status_buf.
#include <cuda.h>
#include <math_constants.h>
#include "common.h"
#include "sm100_ptx.cuh"
#include "tensormap.h"

namespace mpipe {

constexpr int kFwdThreads = 384;
constexpr int kTileM = 128;        // query rows per tile (= TMEM lanes)
constexpr int kTileN = 128;        // keys per K/V tile
constexpr float kRescaleThreshold = 8.0f;  // in log2 units
// setmaxnreg: the 4 light warps release what the 8 softmax warps take (an increase blocks until the CTA's
// own pool has the registers).
constexpr int kFwdRegsLaunch = 168, kFwdRegsLight = 56, kFwdRegsSoftmax = 224;
static_assert(4 * (kFwdRegsLaunch - kFwdRegsLight) >= 8 * (kFwdRegsSoftmax - kFwdRegsLaunch), "setmaxnreg pool arithmetic");

template <int D>
struct FwdCfg {
    static constexpr int kStages = (D == 64) ? 4 : 3;
    static constexpr int kTail = D - 64;                              // 0 or 16 head-dim columns beyond the first 64
    static constexpr int kQBytesMain = kTileM * 128;                  // 64 bf16 per row, 128-byte swizzle
    static constexpr int kQBytesTail = kTail ? kTileM * 32 : 0;       // 16 bf16 per row, 32-byte swizzle
    static constexpr int kQBytes = kQBytesMain + kQBytesTail;         // Q and K tiles (K-major operands)
    static constexpr int kVBytes = kTail ? 2 * kTileN * 128 : kTileN * 128;  // V (MN-major): two 64-wide atoms if D=80
    static constexpr int kSmemQ = 0;
    static constexpr int kSmemK = 2 * kQBytes;
    static constexpr int kSmemV = kSmemK + kStages * kQBytes;
    static constexpr int kSmemTotal = kSmemV + kStages * kVBytes;
    static constexpr int kSmemAlloc = kSmemTotal + 1024;              // slack for manual 1024-byte alignment
    // TMEM: S_w at 128 w, O_w at 256 + 128 w.  head_dim 64 leaves 64 columns behind each O_w: P_w (128 keys as bf16) goes
    // there instead of overlaying S_w, so that S_w(j+1) can be issued as soon as the softmax warps have READ S_w(j)
    // and runs under their exponentials, instead of waiting behind P_w(j) V(j).
    static constexpr bool kPSep = (D + kTileN / 2 <= 128);
    // bit i: column pair i (mod 8) of a row forms its exponential with the polynomial on the FMA pipes instead of the
    // special-function unit.  3 of 8 balances the two when the query tiles' softmax passes alternate (head_dim 80);
    // with separate P columns the two passes run side by side and 2 of 8 measured best (all-MUFU 752, 1 of 8 781,
    // 2 of 8 800, 3 of 8 770 TFLOP/s on the ViT-L workload).
    static constexpr unsigned kPolyMask = kPSep ? 0x12u : 0x52u;
    static constexpr int kColP0 = kPSep ? 256 + 64 : 0, kColPStride = 128;
};

struct FwdParams {
    const mpipe_work_item_t* items;
    int32_t n_items, n_heads;
    __nv_bfloat16* o;
    float* lse;  // nullptr when the encoder is frozen
    int64_t tok_stride_o, head_stride_o;
    int32_t total_tokens;
    float scale_log2;  // softmax_scale * log2(e)
    int32_t* status_buf;
};

struct FwdBarriers {
    uint64_t q_full, q_empty;
    uint64_t k_full[4], k_empty[4], v_full[4], v_empty[4];
    uint64_t s_full[2], p_full[2], o_full[2], s_read[2], pv_done[2];
};

template <int D>
__global__ void __maxnreg__(kFwdRegsLaunch)
attn_fwd_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_q_tail,
                const __grid_constant__ CUtensorMap map_k_tail, const FwdParams p) {
    using Cfg = FwdCfg<D>;
    constexpr int NS = Cfg::kStages;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ FwdBarriers bars;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;

    if (tid == 0) {
        abort_flag = 0;
        mbar_init(&bars.q_full, 1);
        mbar_init(&bars.q_empty, 1);
        for (int s = 0; s < 4; ++s) {
            mbar_init(&bars.k_full[s], 1);
            mbar_init(&bars.k_empty[s], 1);
            mbar_init(&bars.v_full[s], 1);
            mbar_init(&bars.v_empty[s], 1);
        }
        for (int w = 0; w < 2; ++w) {
            mbar_init(&bars.s_full[w], 1);
            mbar_init(&bars.p_full[w], 4);  // one arrival per softmax warp
            mbar_init(&bars.o_full[w], 1);
            mbar_init(&bars.s_read[w], 4);   // (separate P only) S_w is in the softmax warps' registers
            mbar_init(&bars.pv_done[w], 1);  // (separate P only) P_w V has consumed P_w and updated O_w
        }
        fence_mbar_init();
    }
    if (warp == 2) {
        tmem_alloc(&tmem_base_slot, 512);
        tmem_relinquish();
    }
    if (warp == 0 && lane == 0) {
        prefetch_tmap(&map_q);
        prefetch_tmap(&map_k);
        prefetch_tmap(&map_v);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_slot;
    // TMEM columns: S_0 [0,128), S_1 [128,256), O_0 [256,256+D), O_1 [384,384+D); P_w overlays S_w.
    // The plan comes from device memory: it is checked as a whole before any role starts (see plan_ok_cta); a
    // rejected plan leaves every role with nothing to do.
    __shared__ int plan_flag;
    const int n_units = plan_ok_cta(p.items, p.n_items, 2 * kTileM, p.total_tokens, p.status_buf, &plan_flag) ? p.n_items * p.n_heads : 0;
    // Units are sorted by decreasing cost; CTAs walk them in boustrophedon order (0..G-1, then G-1..0, ...) so
    // that the CTA that got the most expensive unit of one round gets the cheapest of the next.
    auto unit_of = [&](int round) {
        const int g = int(gridDim.x), i = int(blockIdx.x);
        return round * g + ((round & 1) ? g - 1 - i : i);
    };
    auto item_at = [&](int u) {
        mpipe_work_item_t z = {0, 0, 0, 0, 0, 0};
        return (u < n_units) ? p.items[u / p.n_heads] : z;
    };

    if (warp == 0) {
        setmaxnreg_dec<kFwdRegsLight>();
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t kv_it = 0, unit_it = 0;
            bool ok = true;
            mpipe_work_item_t it_next = item_at(unit_of(0));   // one unit ahead: the global load is off the unit's critical path
            for (int ur = 0, u = unit_of(0); u < n_units && ok; ++ur, u = unit_of(ur), ++unit_it) {
                const mpipe_work_item_t it = it_next;
                it_next = item_at(unit_of(ur + 1));
                const int head = u % p.n_heads;
                const bool two = it.row_len > kTileM;
                const int nkv = (it.kv_len + kTileN - 1) / kTileN;
                ok = mbar_wait(&bars.q_empty, (unit_it & 1) ^ 1, &abort_flag);
                if (!ok) break;
                mbar_expect_tx(&bars.q_full, (two ? 2 : 1) * Cfg::kQBytes);
                for (int w = 0; w < (two ? 2 : 1); ++w) {
                    uint8_t* dst = smem + Cfg::kSmemQ + w * Cfg::kQBytes;
                    tma_load_3d(dst, &map_q, &bars.q_full, 0, head, it.row_start + w * kTileM);
                    if (Cfg::kTail) tma_load_3d(dst + Cfg::kQBytesMain, &map_q_tail, &bars.q_full, 64, head, it.row_start + w * kTileM);
                }
                for (int j = 0; j < nkv; ++j, ++kv_it) {
                    const int s = kv_it % NS;
                    const uint32_t ph = (kv_it / NS) & 1;
                    const int row = it.kv_start + j * kTileN;
                    ok = mbar_wait(&bars.k_empty[s], ph ^ 1, &abort_flag);
                    if (!ok) break;
                    mbar_expect_tx(&bars.k_full[s], Cfg::kQBytes);
                    uint8_t* kdst = smem + Cfg::kSmemK + s * Cfg::kQBytes;
                    tma_load_3d(kdst, &map_k, &bars.k_full[s], 0, head, row);
                    if (Cfg::kTail) tma_load_3d(kdst + Cfg::kQBytesMain, &map_k_tail, &bars.k_full[s], 64, head, row);
                    ok = mbar_wait(&bars.v_empty[s], ph ^ 1, &abort_flag);
                    if (!ok) break;
                    mbar_expect_tx(&bars.v_full[s], Cfg::kVBytes);
                    uint8_t* vdst = smem + Cfg::kSmemV + s * Cfg::kVBytes;
                    tma_load_3d(vdst, &map_v, &bars.v_full[s], 0, head, row);
                    if (Cfg::kTail) tma_load_3d(vdst + kTileN * 128, &map_v, &bars.v_full[s], 64, head, row);
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ tcgen05 issuer
        // The whole warp walks the loop (uniform control flow, uniform descriptors); one elected lane
        // issues the MMAs and commits.  Descriptors are precomputed: a K-step only bumps the low word.
        setmaxnreg_dec<kFwdRegsLight>();
        {
            const bool leader = elect_one();
            const uint32_t sbase = smem_u32(smem);
            constexpr uint32_t hi128 = umma_desc_hi(1024, kSwizzle128);
            constexpr uint32_t hi32 = umma_desc_hi(256, kSwizzle32);
            uint32_t kv_it = 0, unit_it = 0, cnt[2] = {0, 0};
            bool ok = true;
            // S_w = Q_w K^T for the KV tile in stage s; n_cols = keys to cover (multiple of 16)
            auto issue_s = [&](int w, int s, int n_cols) {
                const uint32_t qa = sbase + Cfg::kSmemQ + w * Cfg::kQBytes;
                const uint32_t ka = sbase + Cfg::kSmemK + s * Cfg::kQBytes;
                const uint32_t qlo = umma_desc_lo(qa, 0), klo = umma_desc_lo(ka, 0);
                const uint32_t idesc = umma_idesc_bf16(kTileM, n_cols, 0, 0);
                const uint32_t d = tmem + w * 128;
                if (leader) {
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        umma_ss(d, umma_desc(qlo + ks * 2, hi128), umma_desc(klo + ks * 2, hi128), idesc, ks > 0);
                    if (Cfg::kTail)
                        umma_ss(d, umma_desc(umma_desc_lo(qa + Cfg::kQBytesMain, 0), hi32),
                                umma_desc(umma_desc_lo(ka + Cfg::kQBytesMain, 0), hi32), idesc, 1);
                }
            };
            // O_w (+)= P_w V for the KV tile in stage s; n_keys = keys to cover (multiple of 16)
            auto issue_pv = [&](int w, int s, int n_keys, bool accumulate) {
                const uint32_t vlo = umma_desc_lo(sbase + Cfg::kSmemV + s * Cfg::kVBytes, kTileN * 128);
                constexpr uint32_t idesc = umma_idesc_bf16(kTileM, D, 0, 1);
                const uint32_t d = tmem + 256 + w * 128;
                const uint32_t pa = tmem + Cfg::kColP0 + w * Cfg::kColPStride;
                if (leader) {
                    if (n_keys == kTileN) {
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks)
                            umma_ts(d, pa + ks * 8, umma_desc(vlo + ks * 128, hi128), idesc, (accumulate || ks > 0) ? 1u : 0u);
                    } else {
                        for (int ks = 0; ks < n_keys / 16; ++ks)
                            umma_ts(d, pa + ks * 8, umma_desc(vlo + ks * 128, hi128), idesc, (accumulate || ks > 0) ? 1u : 0u);
                    }
                }
            };
            mpipe_work_item_t it_next = item_at(unit_of(0));   // one unit ahead: the global load is off the unit's critical path
            for (int ur = 0, u = unit_of(0); u < n_units && ok; ++ur, u = unit_of(ur), ++unit_it) {
                const mpipe_work_item_t it = it_next;
                it_next = item_at(unit_of(ur + 1));
                const bool two = it.row_len > kTileM;
                const int nkv = (it.kv_len + kTileN - 1) / kTileN;
                auto cols_of = [&](int j) {
                    const int rem = it.kv_len - j * kTileN;
                    return rem >= kTileN ? kTileN : ((rem + 15) & ~15);
                };
                ok = mbar_wait(&bars.q_full, unit_it & 1, &abort_flag);
                if (!ok) break;
                {
                    const int s = kv_it % NS;
                    ok = mbar_wait(&bars.k_full[s], (kv_it / NS) & 1, &abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    issue_s(0, s, cols_of(0));
                    if (leader) umma_commit(&bars.s_full[0]);
                    if (two) {
                        issue_s(1, s, cols_of(0));
                        if (leader) umma_commit(&bars.s_full[1]);
                    }
                    if (leader) umma_commit(&bars.k_empty[s]);
                    if (nkv == 1) if (leader) umma_commit(&bars.q_empty);
                }
                if (Cfg::kPSep) {
                    // Order per KV tile j:  S_0(j+1) | PV_1(j-1) | S_1(j+1) | PV_0(j): each S goes out as soon as its
                    // predecessor has been read, each PV as soon as its P is complete, and the two query tiles stay half
                    // a pass apart.
                    for (int j = 0; j < nkv; ++j) {
                        const uint32_t itv = kv_it + j;
                        const int sv = itv % NS;
                        const bool more = (j + 1 < nkv);
                        const int sk = (itv + 1) % NS;
                        if (more) {
                            ok = mbar_wait(&bars.k_full[sk], ((itv + 1) / NS) & 1, &abort_flag);
                            if (ok) ok = mbar_wait(&bars.s_read[0], (cnt[0] + j) & 1, &abort_flag);
                            if (!ok) break;
                            tc_fence_after();
                            issue_s(0, sk, cols_of(j + 1));
                            if (leader) umma_commit(&bars.s_full[0]);
                        }
                        if (two && j > 0) {
                            ok = mbar_wait(&bars.p_full[1], (cnt[1] + j - 1) & 1, &abort_flag);
                            if (!ok) break;
                            tc_fence_after();
                            issue_pv(1, (itv - 1) % NS, cols_of(j - 1), j - 1 > 0);
                            if (leader) umma_commit(&bars.pv_done[1]);
                            if (leader) umma_commit(&bars.v_empty[(itv - 1) % NS]);
                        }
                        if (more) {
                            if (two) {
                                ok = mbar_wait(&bars.s_read[1], (cnt[1] + j) & 1, &abort_flag);
                                if (!ok) break;
                                tc_fence_after();
                                issue_s(1, sk, cols_of(j + 1));
                                if (leader) umma_commit(&bars.s_full[1]);
                            }
                            if (leader) umma_commit(&bars.k_empty[sk]);
                            if (j + 2 == nkv) if (leader) umma_commit(&bars.q_empty);
                        }
                        ok = mbar_wait(&bars.v_full[sv], (itv / NS) & 1, &abort_flag);
                        if (ok) ok = mbar_wait(&bars.p_full[0], (cnt[0] + j) & 1, &abort_flag);
                        if (!ok) break;
                        tc_fence_after();
                        issue_pv(0, sv, cols_of(j), j > 0);
                        if (leader) umma_commit(&bars.pv_done[0]);
                        if (!more) if (leader) umma_commit(&bars.o_full[0]);
                        if (!two) if (leader) umma_commit(&bars.v_empty[sv]);
                    }
                    if (ok && two) {   // PV_1 of the unit's last KV tile
                        const uint32_t itv = kv_it + nkv - 1;
                        ok = mbar_wait(&bars.p_full[1], (cnt[1] + nkv - 1) & 1, &abort_flag);
                        if (!ok) break;
                        tc_fence_after();
                        issue_pv(1, itv % NS, cols_of(nkv - 1), nkv - 1 > 0);
                        if (leader) umma_commit(&bars.pv_done[1]);
                        if (leader) umma_commit(&bars.o_full[1]);
                        if (leader) umma_commit(&bars.v_empty[itv % NS]);
                    }
                    if (!ok) break;
                } else
                for (int j = 0; j < nkv; ++j) {
                    const uint32_t itv = kv_it + j;
                    const int sv = itv % NS;
                    const bool more = (j + 1 < nkv);
                    const int sk = (itv + 1) % NS;
                    ok = mbar_wait(&bars.v_full[sv], (itv / NS) & 1, &abort_flag);
                    if (!ok) break;
                    ok = mbar_wait(&bars.p_full[0], (cnt[0] + j) & 1, &abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    issue_pv(0, sv, cols_of(j), j > 0);
                    if (more) {
                        ok = mbar_wait(&bars.k_full[sk], ((itv + 1) / NS) & 1, &abort_flag);
                        if (!ok) break;
                        tc_fence_after();
                        issue_s(0, sk, cols_of(j + 1));
                        if (leader) umma_commit(&bars.s_full[0]);
                    } else {
                        if (leader) umma_commit(&bars.o_full[0]);
                    }
                    if (two) {
                        ok = mbar_wait(&bars.p_full[1], (cnt[1] + j) & 1, &abort_flag);
                        if (!ok) break;
                        tc_fence_after();
                        issue_pv(1, sv, cols_of(j), j > 0);
                        if (more) {
                            issue_s(1, sk, cols_of(j + 1));
                            if (leader) umma_commit(&bars.s_full[1]);
                        } else {
                            if (leader) umma_commit(&bars.o_full[1]);
                        }
                    }
                    if (leader) umma_commit(&bars.v_empty[sv]);
                    if (more) {
                        if (leader) umma_commit(&bars.k_empty[sk]);
                        if (j + 2 == nkv) if (leader) umma_commit(&bars.q_empty);
                    }
                }
                kv_it += nkv;
                cnt[0] += nkv;
                if (two) cnt[1] += nkv;
            }
        }
        __syncwarp();
    } else if (warp < 4) {
        setmaxnreg_dec<kFwdRegsLight>();
    } else {
        // ------------------------------------------------------------------ softmax + epilogue
        setmaxnreg_inc<kFwdRegsSoftmax>();
        const int w = (warp - 4) >> 2;              // query tile handled by this warpgroup
        const int r = ((warp & 3) << 5) | lane;     // row inside the tile = TMEM lane
        const uint32_t lane_base = uint32_t((warp & 3) * 32) << 16;
        const uint32_t t_s = tmem + lane_base + w * 128;
        const uint32_t t_o = tmem + lane_base + 256 + w * 128;
        const uint32_t t_p = tmem + lane_base + Cfg::kColP0 + w * Cfg::kColPStride;   // = t_s when P overlays S
        uint32_t cnt = 0, ocnt = 0;
        bool ok = true;
        mpipe_work_item_t it_next = item_at(unit_of(0));   // one unit ahead: the global load is off the unit's critical path
        for (int ur = 0, u = unit_of(0); u < n_units && ok; ++ur, u = unit_of(ur)) {
            const mpipe_work_item_t it = it_next;
            it_next = item_at(unit_of(ur + 1));
            const int head = u % p.n_heads;
            const int rows_here = it.row_len - w * kTileM;  // valid rows of this tile
            if (rows_here <= 0) continue;
            const int nkv = (it.kv_len + kTileN - 1) / kTileN;
            float m_ref = -CUDART_INF_F;  // reference maximum, scaled log2 domain
            float l = 0.f;
            for (int j = 0; j < nkv; ++j) {
                ok = mbar_wait(&bars.s_full[w], (cnt + j) & 1, &abort_flag);
                if (!ok) break;
                tc_fence_after();
                uint32_t sr[128];
                tmem_ld32(t_s + 0, *reinterpret_cast<uint32_t(*)[32]>(&sr[0]));
                tmem_ld32(t_s + 32, *reinterpret_cast<uint32_t(*)[32]>(&sr[32]));
                tmem_ld32(t_s + 64, *reinterpret_cast<uint32_t(*)[32]>(&sr[64]));
                tmem_ld32(t_s + 96, *reinterpret_cast<uint32_t(*)[32]>(&sr[96]));
                tmem_wait_ld();
                if (Cfg::kPSep) {   // the scores are in registers: S_w of the next KV tile may be written
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars.s_read[w]);
                }
                const int n_valid = it.kv_len - j * kTileN;
                if (n_valid < kTileN) {
#pragma unroll
                    for (int c = 0; c < 128; ++c)
                        if (c >= n_valid) sr[c] = 0xFF800000u;  // -inf
                }
                // eight independent running maxima, three inputs per instruction (a single chain of 127
                // dependent max ops would cost ~4 cycles each with only two softmax warps per scheduler)
                float mx8[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) mx8[e] = fmaxf(__uint_as_float(sr[e]), __uint_as_float(sr[8 + e]));
#pragma unroll
                for (int c = 16; c < 128; c += 16) {
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        mx8[e] = fmax3(mx8[e], __uint_as_float(sr[c + e]), __uint_as_float(sr[c + 8 + e]));
                }
                const float mx = fmax3(fmax3(mx8[0], mx8[1], mx8[2]), fmax3(mx8[3], mx8[4], mx8[5]), fmaxf(mx8[6], mx8[7]));
                const float m_tile = mx * p.scale_log2;
                const bool grow = m_tile > m_ref + kRescaleThreshold;  // always true on the first tile
                const float m_new = grow ? m_tile : m_ref;
                const float alpha = ex2_approx(m_ref - m_new);         // 0 on the first tile, 1 if unchanged
                m_ref = m_new;
                if (Cfg::kPSep && j > 0) {   // P_w V of the previous KV tile has read P_w and updated O_w (long since, as a rule)
                    ok = mbar_wait(&bars.pv_done[w], (cnt + j - 1) & 1, &abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                }
                if (j > 0 && __any_sync(0xffffffffu, grow)) {
                    // rescale this warp's rows of the accumulator; PV(j-1) has completed (overlaid P: it was issued
                    // before S(j), whose completion we just observed; separate P: waited for above)
#pragma unroll
                    for (int c0 = 0; c0 < D; c0 += 16) {
                        uint32_t orr[16];
                        tmem_ld16(t_o + c0, orr);
                        tmem_wait_ld();
#pragma unroll
                        for (int c = 0; c < 16; ++c) orr[c] = __float_as_uint(__uint_as_float(orr[c]) * alpha);
                        tmem_st16(t_o + c0, orr);
                    }
                }
                // p = exp2(s * scale*log2e - m_ref): packed fp32 pairs for the multiply-add and the row sum,
                // four independent partial sums
                const float2 sc2 = make_float2(p.scale_log2, p.scale_log2);
                const float2 nm2 = make_float2(-m_ref, -m_ref);
                float2 acc[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
                for (int c0 = 0; c0 < 128; c0 += 32) {
                    uint32_t pk[16];
#pragma unroll
                    for (int c = 0; c < 32; c += 2) {
                        const float2 x = fma2(make_float2(__uint_as_float(sr[c0 + c]), __uint_as_float(sr[c0 + c + 1])), sc2, nm2);
                        // kPolyMask picks, out of every 8 column pairs, those whose exponential runs on the FMA
                        // pipes; the rest use the special-function unit.  The split balances the two.
                        const float2 e = ((Cfg::kPolyMask >> ((c >> 1) & 7)) & 1) ? exp2_poly2(x)
                                                                           : make_float2(ex2_approx(x.x), ex2_approx(x.y));
                        acc[(c >> 1) & 3] = add2(acc[(c >> 1) & 3], e);
                        pk[c >> 1] = pack_bf16(e.x, e.y);
                    }
                    tmem_st16(t_p + (c0 >> 1), pk);
                }
                const float2 s01 = add2(add2(acc[0], acc[1]), add2(acc[2], acc[3]));
                l = l * alpha + (s01.x + s01.y);
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars.p_full[w]);
            }
            if (!ok) break;
            cnt += nkv;
            // epilogue: O / l -> bf16, LSE = ln2 * m_ref + ln l
            ok = mbar_wait(&bars.o_full[w], ocnt & 1, &abort_flag);
            if (!ok) break;
            ++ocnt;
            tc_fence_after();
            const float inv_l = 1.0f / l;
            const bool store = r < rows_here;
            const int64_t tok = int64_t(it.row_start) + w * kTileM + r;
            __nv_bfloat16* orow = p.o + tok * p.tok_stride_o + int64_t(head) * p.head_stride_o;
#pragma unroll
            for (int c0 = 0; c0 < D; c0 += 16) {
                uint32_t orr[16];
                tmem_ld16(t_o + c0, orr);
                tmem_wait_ld();
                uint4 v0, v1;
                v0.x = pack_bf16(__uint_as_float(orr[0]) * inv_l, __uint_as_float(orr[1]) * inv_l);
                v0.y = pack_bf16(__uint_as_float(orr[2]) * inv_l, __uint_as_float(orr[3]) * inv_l);
                v0.z = pack_bf16(__uint_as_float(orr[4]) * inv_l, __uint_as_float(orr[5]) * inv_l);
                v0.w = pack_bf16(__uint_as_float(orr[6]) * inv_l, __uint_as_float(orr[7]) * inv_l);
                v1.x = pack_bf16(__uint_as_float(orr[8]) * inv_l, __uint_as_float(orr[9]) * inv_l);
                v1.y = pack_bf16(__uint_as_float(orr[10]) * inv_l, __uint_as_float(orr[11]) * inv_l);
                v1.z = pack_bf16(__uint_as_float(orr[12]) * inv_l, __uint_as_float(orr[13]) * inv_l);
                v1.w = pack_bf16(__uint_as_float(orr[14]) * inv_l, __uint_as_float(orr[15]) * inv_l);
                if (store) {
                    *reinterpret_cast<uint4*>(orow + c0) = v0;
                    *reinterpret_cast<uint4*>(orow + c0 + 8) = v1;
                }
            }
            if (store && p.lse != nullptr)
                p.lse[int64_t(head) * p.total_tokens + tok] = m_ref * 0.6931471805599453f + logf(l);
            tc_fence_before();
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 2) tmem_dealloc(tmem, 512);
    if (tid == 0 && abort_flag) report_status(p.status_buf, MPIPE_ERR_TIMEOUT, int32_t(blockIdx.x));
}

template <int D>
static int32_t launch_fwd(const void* q, const void* k, const void* v, int64_t tok_stride, int64_t head_stride,
                          int32_t total_tokens, int32_t n_heads, const FwdParams& prm, cudaStream_t stream) {
    using Cfg = FwdCfg<D>;
    CUtensorMap mq, mk, mv, mqt, mkt;
    const uint32_t main_box = 64;
    if (!make_tensor_map_thd(&mq, q, total_tokens, n_heads, D, tok_stride, head_stride, main_box, kTileM, 128) ||
        !make_tensor_map_thd(&mk, k, total_tokens, n_heads, D, tok_stride, head_stride, main_box, kTileN, 128) ||
        !make_tensor_map_thd(&mv, v, total_tokens, n_heads, D, tok_stride, head_stride, main_box, kTileN, 128))
        return MPIPE_ERR_CUDA;
    mqt = mq;
    mkt = mk;
    if (Cfg::kTail) {
        if (!make_tensor_map_thd(&mqt, q, total_tokens, n_heads, D, tok_stride, head_stride, 16, kTileM, 32) ||
            !make_tensor_map_thd(&mkt, k, total_tokens, n_heads, D, tok_stride, head_stride, 16, kTileN, 32))
            return MPIPE_ERR_CUDA;
    }
    if (!ensure_dynamic_smem<attn_fwd_kernel<D>>(Cfg::kSmemAlloc)) return MPIPE_ERR_CUDA;
    const int n_units = prm.n_items * prm.n_heads;
    const int grid = n_units < sm_count() ? n_units : sm_count();
    profile_start(kProfileFwd, stream);
    attn_fwd_kernel<D><<<grid, kFwdThreads, Cfg::kSmemAlloc, stream>>>(mq, mk, mv, mqt, mkt, prm);
    profile_stop(kProfileFwd, stream);
    return cudaGetLastError() == cudaSuccess ? MPIPE_OK : MPIPE_ERR_CUDA;
}

}  // namespace mpipe

extern "C" {

int32_t mpipe_fwd_tile_rows(void) { return 2 * mpipe::kTileM; }

int32_t mpipe_varlen_attn_fwd(const void* q, const void* k, const void* v, void* o, float* lse,
                              int64_t tok_stride_qkv, int64_t head_stride_qkv, int64_t tok_stride_o,
                              int64_t head_stride_o, const int32_t* cu_seqlens_dev, int32_t n_seg,
                              int32_t total_tokens, int32_t max_seqlen, const mpipe_work_item_t* fwd_items_dev,
                              int32_t n_fwd_items, int32_t n_heads, int32_t head_dim, float softmax_scale,
                              int32_t mode, int32_t* status_buf, void* stream) {
    using namespace mpipe;
    if (mode != MPIPE_ENC_FROZEN && mode != MPIPE_ENC_TRAINED) return MPIPE_ERR_INVALID_ARG;
    if (n_seg < 0 || total_tokens < 0 || max_seqlen < 0 || n_fwd_items < 0 || n_heads <= 0) return MPIPE_ERR_INVALID_ARG;
    if (head_dim != 64 && head_dim != 80) return MPIPE_ERR_UNSUPPORTED;
    if (total_tokens == 0 || n_fwd_items == 0) return MPIPE_OK;
    if (q == nullptr || k == nullptr || v == nullptr || o == nullptr || fwd_items_dev == nullptr ||
        cu_seqlens_dev == nullptr)
        return MPIPE_ERR_INVALID_ARG;
    if (mode == MPIPE_ENC_TRAINED && lse == nullptr) return MPIPE_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return MPIPE_ERR_INVALID_ARG;
    if ((tok_stride_qkv & 7) || (head_stride_qkv & 7) || (tok_stride_o & 7) || (head_stride_o & 7))
        return MPIPE_ERR_INVALID_ARG;
    if (head_stride_qkv < head_dim || head_stride_o < head_dim || tok_stride_qkv < head_dim || tok_stride_o < head_dim)
        return MPIPE_ERR_INVALID_ARG;
    if (!(softmax_scale > 0.f) || !(softmax_scale < 1e30f)) return MPIPE_ERR_INVALID_ARG;
    if (int64_t(n_fwd_items) * n_heads >= (int64_t(1) << 31)) return MPIPE_ERR_INVALID_ARG;

    FwdParams prm;
    prm.items = fwd_items_dev;
    prm.n_items = n_fwd_items;
    prm.n_heads = n_heads;
    prm.o = static_cast<__nv_bfloat16*>(o);
    prm.lse = (mode == MPIPE_ENC_TRAINED) ? lse : nullptr;
    prm.tok_stride_o = tok_stride_o;
    prm.head_stride_o = head_stride_o;
    prm.total_tokens = total_tokens;
    prm.scale_log2 = softmax_scale * 1.4426950408889634f;
    prm.status_buf = status_buf;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (head_dim == 64)
        return launch_fwd<64>(q, k, v, tok_stride_qkv, head_stride_qkv, total_tokens, n_heads, prm, st);
    return launch_fwd<80>(q, k, v, tok_stride_qkv, head_stride_qkv, total_tokens, n_heads, prm, st);
}

}  // extern "C"
