// mpipe_varlen_attn_bwd: gradient of the per-image softmax attention, the attention part of the
// optional Bwd(enc, r, m) event (it exists only when trainable(enc), Lemma 1).
//
// Three launches on the caller's stream:
//   1. prepass   Delta[h,t] = sum_d dO[t,h,d] O[t,h,d]  and the fp32 dQ accumulator is cleared
//   2. main      one persistent CTA per SM walks (key tile x head) units; a unit keeps one 128-key
//                K/V tile resident and loops over the 128-row query tiles of the same segment
//   3. convert   dQ = softmax_scale * accumulator -> bf16
//
// Main kernel, per query tile i (everything transposed so that the key index is the TMEM lane):
//   S^T  = K Q^T            tcgen05, operands in shared memory               -> TMEM
//   dP^T = V dO^T           tcgen05                                           -> TMEM
//   P^T  = exp2(S^T * scale*log2e - LSE*log2e)       softmax warps, written over S^T as bf16
//   dS^T = P^T o (dP^T - Delta)                      softmax warps, over dP^T as bf16 + to shared memory
//   dV  += P^T dO           tcgen05, A operand read from TMEM, dO as MN-major B
//   dK  += dS^T Q           tcgen05, A operand read from TMEM, Q as MN-major B
//   dQ_i = dS K             tcgen05, dS^T in shared memory read as an MN-major A, K as MN-major B
// dQ_i is read back from TMEM by a reducer warpgroup, staged in shared memory and added to the global fp32
// accumulator by the copy engine (cp.reduce.async.bulk.tensor, fp32 add): the order of those additions is not
// fixed, so the low bits of dQ can differ from run to run.  dK (x softmax_scale) and dV leave TMEM once per unit.
//
// Warp roles (512 threads): 0 TMA producer, 1 / 3 tcgen05 issuers of TMEM stage 0 / 1, 2 TMEM allocation and
// LSE/Delta staging, 4-7 / 8-11 softmax of stage 0 / 1, 12-15 dQ reducer and epilogue.
// Every wait is bounded (see sm100_ptx.cuh); expiry sets status_buf and drains the CTA.
#include <cuda.h>
#include <math_constants.h>
#include "common.h"
#include "sm100_ptx.cuh"
#include "tensormap.h"

namespace mpipe {

constexpr int kSleepAux = 100;   // ns between polls of the roles with slack (producer, staging, reducer)
constexpr int kBwdThreads = 512;
// Register re-balancing (setmaxnreg): an increase can only draw on registers that other warps of the
// same CTA have released, so what the 4 service and 4 reducer warps give back must cover what the 8
// softmax warps take -- otherwise the increase blocks forever.
constexpr int kRegsLaunch = 128, kRegsService = 72, kRegsReducer = 96, kRegsSoftmax = 168;
static_assert(4 * (kRegsLaunch - kRegsService) + 4 * (kRegsLaunch - kRegsReducer) >= 8 * (kRegsSoftmax - kRegsLaunch),
              "setmaxnreg pool arithmetic");
constexpr int kBT = 128;  // keys per unit = TMEM lanes
constexpr int kQS = 64;   // query rows per sub-tile (one pipeline stage of S^T / dP^T)

template <int D>
struct BwdCfg {
    static constexpr int kTail = D - 64;
    static constexpr int kTileMain = kBT * 128;                 // K, V: [128 rows][64 bf16], 128-byte swizzle
    static constexpr int kTileTail = kTail ? kBT * 32 : 0;      //       [128 rows][16 bf16], 32-byte swizzle
    static constexpr int kTile = kTileMain + kTileTail;
    static constexpr int kSubMain = kQS * 128;                  // Q, dO sub-tiles: [64 rows][64 bf16]
    static constexpr int kSubTail = kTail ? kQS * 32 : 0;
    static constexpr int kSub = kSubMain + kSubTail;
    static constexpr int kRing = 4;                             // Q/dO sub-tile stages
    // Issuing warps: two (one per TMEM stage) decouple the warpgroups and gain ~10 % at D = 80; at D = 64 a single
    // in-order issuer measured ~3 % faster (and keeps dK/dV bit-reproducible), so that is what D = 64 uses.
    static constexpr int kIssuers = (D == 64) ? 1 : 2;
    static constexpr int kKVBufs = (D == 64) ? 2 : 1;           // D = 64: the next unit's K/V tiles load during the current unit
    // LSE / Delta stages.  One issuing warp: they travel with the Q / dO stages (same ring, same full / empty barriers:
    // the issuer has no waits to spare).  Two issuing warps: a ring of 8 with barriers of its own, staged far ahead.
    static constexpr bool kStatFolded = (kIssuers == 1);
    static constexpr int kStatRing = kStatFolded ? kRing : 8;
    // dQ staging for the TMA reduction: one [128 q][32 fp32] box (used twice per pair) + the 16-column tail box
    static constexpr int kStageMain = kBT * 128;
    static constexpr int kStageBytes = kStageMain + (kTail ? kBT * 64 : 0);
    static constexpr int kSmemK = 0;                            // buffer i at kSmemK + i * 2 * kTile (K then V)
    static constexpr int kSmemV = kTile;
    static constexpr int kSmemQ = kKVBufs * 2 * kTile;
    static constexpr int kSmemDO = kSmemQ + kRing * kSub;
    static constexpr int kDSBytes = 2 * kBT * 128;              // dS^T of a pair as [key][q]: two 64-query atoms of 16 KB
    static constexpr int kSmemDS = kSmemDO + kRing * kSub;      // two of them: pair j writes buffer j & 1 while dQ(j-1) reads the other
    static constexpr int kSmemStage = kSmemDS + 2 * kDSBytes;
    static constexpr int kSmemStat = kSmemStage + kStageBytes;  // kStatRing x (LSE[64], Delta[64]) fp32
    static constexpr int kSmemTotal = kSmemStat + kStatRing * 2 * kQS * 4;
    static constexpr int kSmemAlloc = kSmemTotal + 1024;
    // TMEM columns: S^T stage b at 64*b, dP^T stage b at 128 + 64*b (P^T / dS^T overlay their first 32 columns)
    static constexpr int kColS = 0, kColDP = 128, kColDV = 256, kColDK = 256 + D, kColDQ = 256 + 2 * D;
    static_assert(kSmemAlloc <= 227 * 1024, "shared memory budget");
    static_assert(kColDQ + D <= 512, "TMEM budget");
};

struct BwdParams {
    const mpipe_work_item_t* items;
    int32_t n_items, n_heads, total_tokens;
    const float* lse;    // [H, T]
    const float* delta;  // [H, T]
    __nv_bfloat16 *dk, *dv;
    int64_t tok_stride_g, head_stride_g;
    float scale, scale_log2;
    int32_t* status_buf;
};

struct BwdBarriers {
    uint64_t kv_full[2], kv_empty[2], dkv_full, dkv_empty, acc_v, acc_k;
    uint64_t qdo_full[4], qdo_empty[4], stat_full[8], stat_empty[8];
    uint64_t s_full[2], p_full[2], dp_full[2], ds_full[2], dq_full[2], dq_empty, ds0_seen;
};

struct BwdMaps {
    CUtensorMap q, k, v, dout, q_tail, k_tail, v_tail, dout_tail, dq_acc, dq_acc_tail;
};

template <int D>
__global__ void __maxnreg__(kRegsLaunch)
attn_bwd_kernel(const __grid_constant__ BwdMaps maps, const BwdParams p) {
    using Cfg = BwdCfg<D>;
    constexpr int NR = Cfg::kRing;
    constexpr int NS = Cfg::kStatRing;
    constexpr int kIssuers = Cfg::kIssuers;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ BwdBarriers bars;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;

    if (tid == 0) {
        abort_flag = 0;
        for (int i = 0; i < 2; ++i) {
            mbar_init(&bars.kv_full[i], 1);
            mbar_init(&bars.kv_empty[i], kIssuers);   // one commit from each issuing warp
        }
        mbar_init(&bars.acc_v, 1);
        mbar_init(&bars.acc_k, 1);
        mbar_init(&bars.dkv_full, kIssuers);
        mbar_init(&bars.dkv_empty, 4);
        for (int s = 0; s < 4; ++s) {
            mbar_init(&bars.qdo_full[s], Cfg::kStatFolded ? 2 : 1);   // the producer's expect_tx arrival (+ the staging warp)
            mbar_init(&bars.qdo_empty[s], 1);
        }
        for (int s = 0; s < 8; ++s) {
            mbar_init(&bars.stat_full[s], 1);
            mbar_init(&bars.stat_empty[s], 1);   // released by the issuing warp once the sub-tile's dS^T has arrived
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&bars.s_full[b], 1);
            mbar_init(&bars.p_full[b], 4);
            mbar_init(&bars.dp_full[b], 1);
            mbar_init(&bars.ds_full[b], 4);
        }
        mbar_init(&bars.ds0_seen, 1);
        mbar_init(&bars.dq_full[0], 1);
        mbar_init(&bars.dq_full[1], 1);
        mbar_init(&bars.dq_empty, 4);
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
    const int n_units = p.n_items * p.n_heads;
    // Units are sorted by decreasing cost; CTAs walk them in boustrophedon order (0..G-1, then G-1..0, ...) so
    // that the CTA that got the most expensive unit of one round gets the cheapest of the next.
    auto unit_of = [&](int round) {
        const int g = int(gridDim.x), i = int(blockIdx.x);
        return round * g + ((round & 1) ? g - 1 - i : i);
    };
    // Items are clamped to the tensors before use (see sanitize_item): a corrupt plan cannot make a store, a
    // reduction or an LSE / Delta read leave them.
    auto item_at = [&](int u) {
        mpipe_work_item_t z = {0, 0, 0, 0, 0, 0};
        if (u >= n_units) return z;
        z = p.items[u / p.n_heads];
        if (sanitize_item(z, kBT, p.total_tokens) && tid == 12 * 32) report_status(p.status_buf, MPIPE_ERR_INDEX, u);
        return z;
    };
    // Every unit runs an even number of 64-query sub-tiles (a 128-query tile is two of them); a padding
    // sub-tile past the segment end contributes nothing because its probabilities are forced to zero.
    auto subtiles_of = [](const mpipe_work_item_t& it) { return 2 * ((it.kv_len + kBT - 1) / kBT); };

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        setmaxnreg_dec<kRegsService>();
        if (lane == 0) {
            uint32_t unit_it = 0, sc = 0;
            bool ok = true;
            mpipe_work_item_t it_next = item_at(unit_of(0));   // one unit ahead: the global load is off the unit's critical path
            for (int ur = 0, u = unit_of(0); u < n_units && ok; ++ur, u = unit_of(ur), ++unit_it) {
                const mpipe_work_item_t it = it_next;
                it_next = item_at(unit_of(ur + 1));
                const int head = u % p.n_heads;
                const int n2 = subtiles_of(it);
                const int kb = unit_it % Cfg::kKVBufs;            // K/V buffer of this unit
                uint8_t* kv = smem + kb * (2 * Cfg::kTile);
                ok = mbar_wait<kSleepAux>(&bars.kv_empty[kb], ((unit_it / Cfg::kKVBufs) & 1) ^ 1, &abort_flag);
                if (!ok) break;
                mbar_expect_tx(&bars.kv_full[kb], 2 * Cfg::kTile);
                tma_load_3d(kv + Cfg::kSmemK, &maps.k, &bars.kv_full[kb], 0, head, it.row_start);
                tma_load_3d(kv + Cfg::kSmemV, &maps.v, &bars.kv_full[kb], 0, head, it.row_start);
                if (Cfg::kTail) {
                    tma_load_3d(kv + Cfg::kSmemK + Cfg::kTileMain, &maps.k_tail, &bars.kv_full[kb], 64, head, it.row_start);
                    tma_load_3d(kv + Cfg::kSmemV + Cfg::kTileMain, &maps.v_tail, &bars.kv_full[kb], 64, head, it.row_start);
                }
                for (int s = 0; s < n2; ++s, ++sc) {
                    const int rs = sc % NR;
                    const int row = it.kv_start + s * kQS;
                    ok = mbar_wait<kSleepAux>(&bars.qdo_empty[rs], ((sc / NR) & 1) ^ 1, &abort_flag);
                    if (!ok) break;
                    mbar_expect_tx(&bars.qdo_full[rs], 2 * Cfg::kSub);
                    uint8_t* qd = smem + Cfg::kSmemQ + rs * Cfg::kSub;
                    uint8_t* dd = smem + Cfg::kSmemDO + rs * Cfg::kSub;
                    tma_load_3d(qd, &maps.q, &bars.qdo_full[rs], 0, head, row);
                    tma_load_3d(dd, &maps.dout, &bars.qdo_full[rs], 0, head, row);
                    if (Cfg::kTail) {
                        tma_load_3d(qd + Cfg::kSubMain, &maps.q_tail, &bars.qdo_full[rs], 64, head, row);
                        tma_load_3d(dd + Cfg::kSubMain, &maps.dout_tail, &bars.qdo_full[rs], 64, head, row);
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1 || (warp == 3 && kIssuers == 2)) {
        // ------------------------------------------------------------------ tcgen05 issuers
        // One issuing warp per TMEM stage (warp 1: even sub-tiles, warp 3: odd sub-tiles), so that neither
        // warpgroup's MMAs wait behind the other's slowest step; a barrier hop costs ~200 cycles (~340 when it
        // starts from a tcgen05.commit), and a single in-order issuer made every one of them serial.
        // The whole warp walks the loop (uniform control flow); one elected lane issues and commits.
        // Descriptors are precomputed halves: a K-step only adds a constant to the low word.
        // Cross-warp ordering on the tensor pipe is needed in two places only: the first (overwriting) dV / dK
        // MMA of a unit comes from stage 0 and must precede stage 1's first accumulation (acc_v / acc_k), and
        // the pair's dQ MMA (issued by stage 1) needs both stages' dS^T in shared memory (ds_full[0]).
        setmaxnreg_dec<kRegsService>();
        {
            const int b0 = (kIssuers == 2) ? (warp >> 1) : 0;   // first TMEM stage served by this warp
            constexpr int kStep = (kIssuers == 2) ? 2 : 1;      // two issuers: every other sub-tile; one: all, in order
            const bool leader = elect_one();
            const uint32_t sbase = smem_u32(smem);
            constexpr uint32_t hi128 = umma_desc_hi(1024, kSwizzle128);
            constexpr uint32_t hi32 = umma_desc_hi(256, kSwizzle32);
            const uint32_t ds_lo = umma_desc_lo(sbase + Cfg::kSmemDS, kBT * 128);   // two 64-query atoms 16 KB apart
            // LSE / Delta of a sub-tile must be staged before its S^T is issued: the softmax warps then need no barrier
            // of their own for them (S^T complete implies staged).  Folded: qdo_full completes only when the staging
            // warp has arrived too, so there is nothing more to wait for here.
            auto wait_stat = [&](uint32_t c) {
                return Cfg::kStatFolded ? true : mbar_wait(&bars.stat_full[c % NS], (c / NS) & 1, &abort_flag);
            };
            constexpr uint32_t idesc_s = umma_idesc_bf16(kBT, kQS, 0, 0);      // K-major x K-major, N = 64 queries
            constexpr uint32_t idesc_ts = umma_idesc_bf16(kBT, 64, 0, 1);      // A in TMEM, MN-major B, N = 64
            constexpr uint32_t idesc_ts_t = umma_idesc_bf16(kBT, 16, 0, 1);    // same, 16-wide head-dim tail
            constexpr uint32_t idesc_dq = umma_idesc_bf16(kBT, 64, 1, 1);      // MN-major A and B
            constexpr uint32_t idesc_dq_t = umma_idesc_bf16(kBT, 16, 1, 1);
            constexpr uint32_t kSubTailOff = Cfg::kSubMain >> 4;
            // descriptor low words of the ring's Q / dO stages: base + stage * (stage bytes / 16); no carry out of the 14
            // address bits as long as the stage lies in shared memory
            const uint32_t q_lo0 = umma_desc_lo(sbase + Cfg::kSmemQ, 0), do_lo0 = umma_desc_lo(sbase + Cfg::kSmemDO, 0);
            auto q_lo_of = [&](uint32_t c) { return q_lo0 + (c % NR) * uint32_t(Cfg::kSub >> 4); };
            auto do_lo_of = [&](uint32_t c) { return do_lo0 + (c % NR) * uint32_t(Cfg::kSub >> 4); };
            // dst[128 keys x 64 q] = A[128 x D] * B[64 x D]^T, both K-major (main 64 columns + optional 16 tail)
            auto issue_kk = [&](uint32_t dcol, uint32_t a, uint32_t at, uint32_t bq) {
                if (leader) {
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        umma_ss(tmem + dcol, umma_desc(a + ks * 2, hi128), umma_desc(bq + ks * 2, hi128), idesc_s, ks > 0);
                    if (Cfg::kTail) umma_ss(tmem + dcol, umma_desc(at, hi32), umma_desc(bq + kSubTailOff, hi32), idesc_s, 1);
                }
            };
            // dst[128 keys x D] (+)= A^T-in-TMEM[128 keys x 64 q] * B[64 q x D] (B rows = q, MN-major)
            auto issue_ts = [&](uint32_t dcol, uint32_t acol, uint32_t bq, bool acc) {
                if (leader) {
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) {
                        umma_ts(tmem + dcol, tmem + acol + ks * 8, umma_desc(bq + ks * 128, hi128), idesc_ts,
                                (acc || ks > 0) ? 1u : 0u);
                        if (Cfg::kTail)
                            umma_ts(tmem + dcol + 64, tmem + acol + ks * 8, umma_desc(bq + kSubTailOff + ks * 32, hi32),
                                    idesc_ts_t, (acc || ks > 0) ? 1u : 0u);
                    }
                }
            };
            uint32_t unit_it = 0, sc = 0;   // sc: global sub-tile counter at the start of the unit (even)
            bool ok = true;
            mpipe_work_item_t it_next = item_at(unit_of(0));   // one unit ahead: the global load is off the unit's critical path
            for (int ur = 0, u = unit_of(0); u < n_units && ok; ++ur, u = unit_of(ur), ++unit_it) {
                const mpipe_work_item_t it = it_next;
                it_next = item_at(unit_of(ur + 1));
                const int n2 = subtiles_of(it);
                const int kb = unit_it % Cfg::kKVBufs;
                const uint32_t kvb = sbase + kb * (2 * Cfg::kTile);
                const uint32_t k_lo = umma_desc_lo(kvb + Cfg::kSmemK, 0), v_lo = umma_desc_lo(kvb + Cfg::kSmemV, 0);
                const uint32_t kt_lo = umma_desc_lo(kvb + Cfg::kSmemK + Cfg::kTileMain, 0);
                const uint32_t vt_lo = umma_desc_lo(kvb + Cfg::kSmemV + Cfg::kTileMain, 0);
                // With two K/V buffers the stream of sub-tiles runs on across the unit boundary: the S^T / dP^T MMAs
                // of the next unit's first two sub-tiles are issued inside this unit's last two iterations, from
                // the other (prefetched) buffer, so the softmax warps never see the pipeline drain between units.
                constexpr bool kStream = (Cfg::kKVBufs == 2);
                const bool has_next = kStream && unit_of(ur + 1) < n_units;
                const uint32_t kvb_n = sbase + (kb ^ 1) * (2 * Cfg::kTile);
                const uint32_t k_lo_n = umma_desc_lo(kvb_n + Cfg::kSmemK, 0), v_lo_n = umma_desc_lo(kvb_n + Cfg::kSmemV, 0);
                ok = mbar_wait(&bars.kv_full[kb], (unit_it / Cfg::kKVBufs) & 1, &abort_flag);
                if (!ok) break;
                if (!kStream || unit_it == 0) {
                    for (int s = b0; s < 2; s += kStep) {   // prologue: S^T and dP^T of the first sub-tile of each stage served
                        const uint32_t c = sc + s;
                        ok = mbar_wait(&bars.qdo_full[c % NR], (c / NR) & 1, &abort_flag);
                        if (!ok) break;
                        ok = wait_stat(c);
                        if (!ok) break;
                        tc_fence_after();
                        issue_kk(Cfg::kColS + 64 * s, k_lo, kt_lo, q_lo_of(c));
                        if (leader) umma_commit(&bars.s_full[s]);
                        issue_kk(Cfg::kColDP + 64 * s, v_lo, vt_lo, do_lo_of(c));
                        if (leader) umma_commit(&bars.dp_full[s]);
                    }
                    if (!ok) break;
                }
                // One sub-tile of the issue order.  The TMEM stage b is a compile-time constant (the loop below is unrolled
                // over the two stages), so stage offsets and barrier addresses fold into immediates.
                auto sub_tile = [&](const int s, auto stage) -> bool {
                    constexpr int b = decltype(stage)::value;
                    const uint32_t c = sc + s;
                    const uint32_t ph = (c >> 1) & 1;   // phase of the per-stage barriers
                    const bool cross = (s + 2 >= n2) && has_next;   // sub-tile s+2 is the next unit's
                    const bool more = (s + 2 < n2) || cross;
                    const bool first = (s < 2);         // the stage's first sub-tile of the unit
                    ok = mbar_wait(&bars.p_full[b], ph, &abort_flag);
                    if (!ok) return false;
                    if (first && b == 0) {          // the accumulators are free: the previous unit's epilogue has read them
                        ok = mbar_wait(&bars.dkv_empty, (unit_it & 1) ^ 1, &abort_flag);
                        if (!ok) return false;
                    } else if (first && kIssuers == 2) {   // ... and stage 0's overwriting dV MMA has been issued
                        ok = mbar_wait(&bars.acc_v, unit_it & 1, &abort_flag);
                        if (!ok) return false;
                    }
                    tc_fence_after();
                    issue_ts(Cfg::kColDV, Cfg::kColS + 64 * b, do_lo_of(c), !(first && b == 0));         // dV += P^T dO
                    if (first && b == 0 && kIssuers == 2) {
                        tc_fence_before();
                        if (leader) mbar_arrive(&bars.acc_v);
                    }
                    if (more) {
                        if (cross && b == 0) {   // the next unit's K/V tiles (loaded while this unit ran)
                            ok = mbar_wait(&bars.kv_full[kb ^ 1], ((unit_it + 1) / Cfg::kKVBufs) & 1, &abort_flag);
                            if (!ok) return false;
                        }
                        ok = mbar_wait(&bars.qdo_full[(c + 2) % NR], ((c + 2) / NR) & 1, &abort_flag);
                        if (!ok) return false;
                        ok = wait_stat(c + 2);
                        if (!ok) return false;
                        tc_fence_after();
                        issue_kk(Cfg::kColS + 64 * b, cross ? k_lo_n : k_lo, kt_lo, q_lo_of(c + 2));       // S^T(s+2)
                        if (leader) umma_commit(&bars.s_full[b]);
                    }
                    ok = mbar_wait(&bars.ds_full[b], ph, &abort_flag);
                    if (!ok) return false;
                    if (first && b == 1 && kIssuers == 2) {
                        ok = mbar_wait(&bars.acc_k, unit_it & 1, &abort_flag);
                        if (!ok) return false;
                    }
                    tc_fence_after();
                    issue_ts(Cfg::kColDK, Cfg::kColDP + 64 * b, q_lo_of(c), !(first && b == 0));          // dK += dS^T Q
                    if (first && b == 0 && kIssuers == 2) {
                        tc_fence_before();
                        if (leader) mbar_arrive(&bars.acc_k);
                    }
                    if (leader) {
                        umma_commit(&bars.qdo_empty[c % NR]);   // folded: also frees the LSE / Delta stage (dS^T(c) has arrived)
                        if (!Cfg::kStatFolded) mbar_arrive(&bars.stat_empty[c % NS]);
                    }
                    if (more) {
                        issue_kk(Cfg::kColDP + 64 * b, cross ? v_lo_n : v_lo, vt_lo, do_lo_of(c + 2));    // dP^T(s+2)
                        if (leader) umma_commit(&bars.dp_full[b]);
                    }
                    if (b == 1) {                                                             // dQ of the 128-query pair
                        if (kIssuers == 2) {   // the other half of dS^T (a single issuer has already waited for it)
                            ok = mbar_wait(&bars.ds_full[0], ph, &abort_flag);
                            if (!ok) return false;
                            if (leader) mbar_arrive(&bars.ds0_seen);   // lets stage 0's warpgroup complete the next phase
                        }
                        ok = mbar_wait(&bars.dq_empty, ((c >> 1) & 1) ^ 1, &abort_flag);
                        if (!ok) return false;
                        tc_fence_after();
                        if (leader) {
#pragma unroll
                            for (int ks = 0; ks < 8; ++ks) {
                                const uint64_t adesc = umma_desc(ds_lo + ph * (Cfg::kDSBytes >> 4) + ks * 128, hi128);
                                umma_ss(tmem + Cfg::kColDQ, adesc, umma_desc(k_lo + ks * 128, hi128), idesc_dq, ks > 0);
                                if (Cfg::kTail)
                                    umma_ss(tmem + Cfg::kColDQ + 64, adesc, umma_desc(kt_lo + ks * 32, hi32), idesc_dq_t, ks > 0);
                            }
                            umma_commit(&bars.dq_full[ph]);
                        }
                    }
                    return true;
                };
                if (kStep == 1) {
                    for (int s = 0; s < n2 && ok; s += 2) {
                        ok = sub_tile(s, std::integral_constant<int, 0>{});
                        if (ok) ok = sub_tile(s + 1, std::integral_constant<int, 1>{});
                    }
                } else {
                    for (int s = b0; s < n2 && ok; s += 2)
                        ok = (b0 == 0) ? sub_tile(s, std::integral_constant<int, 0>{}) : sub_tile(s, std::integral_constant<int, 1>{});
                }
                if (!ok) break;
                if (leader) umma_commit(&bars.dkv_full);
                if (leader) umma_commit(&bars.kv_empty[kb]);
                sc += n2;
            }
        }
        __syncwarp();
    } else if (warp == 2) {
        // ------------------------------------------------------------------ LSE / Delta staging
        setmaxnreg_dec<kRegsService>();
        uint32_t sc = 0;
        bool ok = true;
        mpipe_work_item_t it_next = item_at(unit_of(0));   // one unit ahead: the global load is off the unit's critical path
        for (int ur = 0, u = unit_of(0); u < n_units && ok; ++ur, u = unit_of(ur)) {
            const mpipe_work_item_t it = it_next;
            it_next = item_at(unit_of(ur + 1));
            const int head = u % p.n_heads;
            const int n2 = subtiles_of(it);
            const int q_end = it.kv_start + it.kv_len;
            for (int s = 0; s < n2; ++s, ++sc) {
                const int rs = sc % NS;
                float* dst = reinterpret_cast<float*>(smem + Cfg::kSmemStat + rs * (2 * kQS * 4));
                const int q0 = it.kv_start + s * kQS;
                float val[4];   // read from global memory before the stage is known to be free: the latency overlaps the wait
#pragma unroll
                for (int e = 0; e < 4; ++e) {   // e = 0, 1: -LSE*log2e of 64 query columns; e = 2, 3: -Delta
                    const bool is_lse = (e < 2);
                    const int q = q0 + lane + 32 * (e & 1);
                    if (q < q_end) {   // stored negated: what the softmax warps add
                        val[e] = -__ldg((is_lse ? p.lse : p.delta) + int64_t(head) * p.total_tokens + q);
                        if (is_lse) val[e] *= 1.4426950408889634f;
                    } else {
                        val[e] = is_lse ? -CUDART_INF_F : 0.f;  // P = exp2(-inf) = 0 for query columns past the segment
                    }
                }
                // the stage is free when the MMAs that read the Q / dO sub-tile of four sub-tiles ago have completed
                // (that commit follows the arrival of its dS^T, i.e. the softmax warps' last read of the stage)
                ok = mbar_wait<kSleepAux>(Cfg::kStatFolded ? &bars.qdo_empty[rs] : &bars.stat_empty[rs],
                                                   ((sc / NS) & 1) ^ 1, &abort_flag);
                if (!ok) break;
#pragma unroll
                for (int e = 0; e < 4; ++e) dst[((e < 2) ? 0 : kQS) + lane + 32 * (e & 1)] = val[e];
                __syncwarp();
                if (lane == 0) mbar_arrive(Cfg::kStatFolded ? &bars.qdo_full[rs] : &bars.stat_full[rs]);
            }
        }
    } else if (warp == 3) {
        setmaxnreg_dec<kRegsService>();   // spare warp when one issuer is enough
    } else if (warp < 12) {
        // ------------------------------------------------------------------ softmax / dS warps
        // Warpgroup g owns TMEM stage g, i.e. every other 64-query sub-tile; thread = key row.
        setmaxnreg_inc<kRegsSoftmax>();
        const int g = (warp - 4) >> 2;
        const int r = ((warp & 3) << 5) | lane;
        const uint32_t lane_base = uint32_t((warp & 3) * 32) << 16;
        const uint32_t t_s = tmem + lane_base + Cfg::kColS + g * 64;
        const uint32_t t_dp = tmem + lane_base + Cfg::kColDP + g * 64;
        uint8_t* ds_row = smem + Cfg::kSmemDS + g * (kBT * 128) + r * 128;
        uint32_t sc = 0;   // global sub-tile counter at the start of the unit (always even)
        bool ok = true;
        mpipe_work_item_t it_next = item_at(unit_of(0));   // one unit ahead: the global load is off the unit's critical path
        for (int ur = 0, u = unit_of(0); u < n_units && ok; ++ur, u = unit_of(ur)) {
            const mpipe_work_item_t it = it_next;
            it_next = item_at(unit_of(ur + 1));
            const int n2 = subtiles_of(it);
            const bool key_valid = r < it.row_len;
            const bool ragged_keys = it.row_len < kBT;
            for (int s = g; s < n2; s += 2) {
                const uint32_t c = sc + s;
                const int rs = c % NS;
                const uint32_t ph = (c >> 1) & 1;   // phase of the per-stage barriers = dS^T buffer of the pair
                const float* stat = reinterpret_cast<const float*>(smem + Cfg::kSmemStat + rs * (2 * kQS * 4));
                const float4* lse4 = reinterpret_cast<const float4*>(stat);
                const float4* dl4 = reinterpret_cast<const float4*>(stat + kQS);
                // (the LSE / Delta stage was complete before this S^T was issued)
                ok = mbar_wait(&bars.s_full[g], ph, &abort_flag);
                if (!ok) break;
                tc_fence_after();
                // P^T = exp2(S^T * scale*log2e - LSE*log2e): both 32-column halves are requested before the
                // one wait; multiply-add on packed fp32 pairs
                float pr[64];
                {
                    uint32_t sr[64];
                    tmem_ld32(t_s, *reinterpret_cast<uint32_t(*)[32]>(&sr[0]));
                    tmem_ld32(t_s + 32, *reinterpret_cast<uint32_t(*)[32]>(&sr[32]));
                    tmem_wait_ld();
                    const float2 sc2 = make_float2(p.scale_log2, p.scale_log2);
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        uint32_t pk[16];
#pragma unroll
                        for (int c4 = 0; c4 < 8; ++c4) {
                            const float4 l4 = lse4[h * 8 + c4];
                            const int e = h * 32 + 4 * c4;
                            const float2 x01 = fma2(make_float2(__uint_as_float(sr[e]), __uint_as_float(sr[e + 1])), sc2,
                                                    make_float2(l4.x, l4.y));
                            const float2 x23 = fma2(make_float2(__uint_as_float(sr[e + 2]), __uint_as_float(sr[e + 3])), sc2,
                                                    make_float2(l4.z, l4.w));
                            pr[e] = ex2_approx(x01.x);
                            pr[e + 1] = ex2_approx(x01.y);
                            pr[e + 2] = ex2_approx(x23.x);
                            pr[e + 3] = ex2_approx(x23.y);
                            pk[2 * c4] = pack_bf16(pr[e], pr[e + 1]);
                            pk[2 * c4 + 1] = pack_bf16(pr[e + 2], pr[e + 3]);
                        }
                        tmem_st16(t_s + h * 16, pk);
                    }
                }
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars.p_full[g]);

                ok = mbar_wait(&bars.dp_full[g], ph, &abort_flag);
                if (!ok) break;
                // dS^T buffer (pair & 1) is free once dQ of pair - 2 has completed. With one issuing warp that is implied
                // by s_full above (S^T(c) was issued, in order, after that dQ); with two it is waited for.
                if (kIssuers == 2 && (c >> 1) >= 2) {
                    ok = mbar_wait(&bars.dq_full[ph], ((c >> 2) + 1) & 1, &abort_flag);
                    if (!ok) break;
                }
                tc_fence_after();
                // dS^T = P^T o (dP^T - Delta); key rows past the segment are zeroed on the packed words
                {
                    uint32_t dr[64];
                    tmem_ld32(t_dp, *reinterpret_cast<uint32_t(*)[32]>(&dr[0]));
                    tmem_ld32(t_dp + 32, *reinterpret_cast<uint32_t(*)[32]>(&dr[32]));
                    tmem_wait_ld();
                    uint32_t pk[32];
#pragma unroll
                    for (int c4 = 0; c4 < 16; ++c4) {
                        const float4 d4 = dl4[c4];
                        const int e = 4 * c4;
                        const float2 t01 = add2(make_float2(__uint_as_float(dr[e]), __uint_as_float(dr[e + 1])),
                                                make_float2(d4.x, d4.y));
                        const float2 t23 = add2(make_float2(__uint_as_float(dr[e + 2]), __uint_as_float(dr[e + 3])),
                                                make_float2(d4.z, d4.w));
                        const float2 s01 = mul2(make_float2(pr[e], pr[e + 1]), t01);
                        const float2 s23 = mul2(make_float2(pr[e + 2], pr[e + 3]), t23);
                        pk[2 * c4] = pack_bf16(s01.x, s01.y);
                        pk[2 * c4 + 1] = pack_bf16(s23.x, s23.y);
                    }
                    if (ragged_keys) {   // uniform per unit: only a segment's last key tile has rows to zero
#pragma unroll
                        for (int i = 0; i < 32; ++i) pk[i] = key_valid ? pk[i] : 0u;
                    }
                    tmem_st16(t_dp, *reinterpret_cast<uint32_t(*)[16]>(&pk[0]));
                    tmem_st16(t_dp + 16, *reinterpret_cast<uint32_t(*)[16]>(&pk[16]));
                    // the same 64 values as 8 x 16 bytes of row r of the [key][q] tile (128-byte swizzle)
#pragma unroll
                    for (int chunk = 0; chunk < 8; ++chunk) {
                        *reinterpret_cast<uint4*>(ds_row + ph * Cfg::kDSBytes + ((chunk ^ (r & 7)) << 4)) =
                            make_uint4(pk[4 * chunk], pk[4 * chunk + 1], pk[4 * chunk + 2], pk[4 * chunk + 3]);
                    }
                }
                tmem_wait_st();
                fence_async_smem();
                tc_fence_before();
                __syncwarp();
                // With two issuing warps ds_full[0] has two consumers; the second (stage 1's issuer, before dQ) can lag, and
                // a parity wait cannot tell phase n from n + 2: do not complete a phase before it has seen the last one.
                if (kIssuers == 2 && g == 0 && (c >> 1) >= 1) {
                    ok = mbar_wait(&bars.ds0_seen, ((c >> 1) - 1) & 1, &abort_flag);
                    if (!ok) break;
                }
                if (lane == 0) mbar_arrive(&bars.ds_full[g]);
            }
            sc += n2;
        }
    } else {
        // ------------------------------------------------------------------ dQ reducer + dK/dV epilogue
        // dQ of a 128-query pair: TMEM -> registers -> swizzled staging in shared memory -> one TMA
        // reduce-add per 32 fp32 columns into the global accumulator (the copy engine does the atomics).
        setmaxnreg_dec<kRegsReducer>();
        const int r = ((warp & 3) << 5) | lane;
        const int rt = tid - 12 * 32;   // 0..127 inside the warpgroup
        const uint32_t lane_base = uint32_t((warp & 3) * 32) << 16;
        uint32_t pc = 0, unit_it = 0;   // pair counter
        bool ok = true;
        mpipe_work_item_t it_next = item_at(unit_of(0));   // one unit ahead: the global load is off the unit's critical path
        for (int ur = 0, u = unit_of(0); u < n_units; ++ur, u = unit_of(ur), ++unit_it) {
            const mpipe_work_item_t it = it_next;
            it_next = item_at(unit_of(ur + 1));
            const int head = u % p.n_heads;
            const int npairs = (it.kv_len + kBT - 1) / kBT;
            // No early exit inside this loop: the four warps meet at named barriers, so after a time-out
            // they keep walking the (now empty) iterations together instead of leaving one another behind.
            for (int i = 0; i < npairs; ++i, ++pc) {
                if (ok) ok = mbar_wait<kSleepAux>(&bars.dq_full[pc & 1], (pc >> 1) & 1, &abort_flag);
                tc_fence_after();
                uint8_t* stage = smem + Cfg::kSmemStage;
                const int q0 = it.kv_start + i * kBT;
                // Two steps through one [128 rows][128 B] staging box (128-byte swizzle): columns 0..31, then 32..63; the
                // D = 80 tail (columns 64..79, [128 rows][64 B], 64-byte swizzle) rides with the first step. The second
                // half leaves TMEM before the first is handed to the copy engine, so the next pair's dQ MMA can start.
                if (rt == 0) bulk_wait_group_read<0>();   // the box must have been read before it is overwritten
                named_barrier_sync(1, 128);
                uint32_t v1[2][16];
                if (ok) {
                    uint32_t v0[2][16];
                    tmem_ld16(tmem + lane_base + Cfg::kColDQ, v0[0]);
                    tmem_ld16(tmem + lane_base + Cfg::kColDQ + 16, v0[1]);
                    tmem_wait_ld();
#pragma unroll
                    for (int chunk = 0; chunk < 8; ++chunk)
                        *reinterpret_cast<uint4*>(stage + r * 128 + ((chunk ^ (r & 7)) << 4)) =
                            make_uint4(v0[chunk / 4][4 * (chunk & 3)], v0[chunk / 4][4 * (chunk & 3) + 1],
                                       v0[chunk / 4][4 * (chunk & 3) + 2], v0[chunk / 4][4 * (chunk & 3) + 3]);
                    tmem_ld16(tmem + lane_base + Cfg::kColDQ + 32, v1[0]);
                    tmem_ld16(tmem + lane_base + Cfg::kColDQ + 48, v1[1]);
                    if (Cfg::kTail) {
                        uint32_t vt[16];
                        tmem_ld16(tmem + lane_base + Cfg::kColDQ + 64, vt);
                        tmem_wait_ld();
#pragma unroll
                        for (int chunk = 0; chunk < 4; ++chunk)
                            *reinterpret_cast<uint4*>(stage + Cfg::kStageMain + r * 64 + ((chunk ^ ((r >> 1) & 3)) << 4)) =
                                make_uint4(vt[4 * chunk], vt[4 * chunk + 1], vt[4 * chunk + 2], vt[4 * chunk + 3]);
                    } else {
                        tmem_wait_ld();
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars.dq_empty);   // the whole row has left TMEM
                }
                fence_async_smem();
                named_barrier_sync(1, 128);
                if (ok && rt == 0 && it.seg >= 0) {
                    tma_reduce_add_3d(&maps.dq_acc, stage, 0, head, q0);
                    if (Cfg::kTail) tma_reduce_add_3d(&maps.dq_acc_tail, stage + Cfg::kStageMain, 64, head, q0);
                    bulk_commit_group();
                }
                if (rt == 0) bulk_wait_group_read<0>();
                named_barrier_sync(1, 128);
                if (ok) {
#pragma unroll
                    for (int chunk = 0; chunk < 8; ++chunk)
                        *reinterpret_cast<uint4*>(stage + r * 128 + ((chunk ^ (r & 7)) << 4)) =
                            make_uint4(v1[chunk / 4][4 * (chunk & 3)], v1[chunk / 4][4 * (chunk & 3) + 1],
                                       v1[chunk / 4][4 * (chunk & 3) + 2], v1[chunk / 4][4 * (chunk & 3) + 3]);
                }
                fence_async_smem();
                named_barrier_sync(1, 128);
                if (ok && rt == 0 && it.seg >= 0) {
                    tma_reduce_add_3d(&maps.dq_acc, stage, 32, head, q0);
                    bulk_commit_group();
                }
            }
            if (ok) ok = mbar_wait<kSleepAux>(&bars.dkv_full, unit_it & 1, &abort_flag);
            if (!ok) continue;   // keep walking the units so that the named barriers above stay matched
            tc_fence_after();
            const bool store = r < it.row_len && it.seg >= 0;
            const int64_t tok = int64_t(it.row_start) + r;
            __nv_bfloat16* dv_row = p.dv + tok * p.tok_stride_g + int64_t(head) * p.head_stride_g;
            __nv_bfloat16* dk_row = p.dk + tok * p.tok_stride_g + int64_t(head) * p.head_stride_g;
#pragma unroll
            for (int which = 0; which < 2; ++which) {
                const uint32_t col = which == 0 ? Cfg::kColDV : Cfg::kColDK;
                const float mul = which == 0 ? 1.0f : p.scale;
                __nv_bfloat16* row = which == 0 ? dv_row : dk_row;
#pragma unroll
                for (int c0 = 0; c0 < D; c0 += 32) {   // 32 columns per round trip (16 in the D = 80 tail)
                    uint32_t v[2][16];
                    const bool two = (c0 + 32 <= D);
                    tmem_ld16(tmem + lane_base + col + c0, v[0]);
                    if (two) tmem_ld16(tmem + lane_base + col + c0 + 16, v[1]);
                    tmem_wait_ld();
                    if (which == 1 && c0 + 32 >= D) {   // both accumulators have left TMEM: the next unit may overwrite them
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&bars.dkv_empty);
                    }
#pragma unroll
                    for (int c8 = 0; c8 < (two ? 4 : 2); ++c8) {
                        const uint32_t* w = &v[c8 / 2][(c8 & 1) * 8];
                        uint4 a;
                        a.x = pack_bf16(__uint_as_float(w[0]) * mul, __uint_as_float(w[1]) * mul);
                        a.y = pack_bf16(__uint_as_float(w[2]) * mul, __uint_as_float(w[3]) * mul);
                        a.z = pack_bf16(__uint_as_float(w[4]) * mul, __uint_as_float(w[5]) * mul);
                        a.w = pack_bf16(__uint_as_float(w[6]) * mul, __uint_as_float(w[7]) * mul);
                        if (store) *reinterpret_cast<uint4*>(row + c0 + 8 * c8) = a;
                    }
                }
            }
        }
        if (rt == 0) bulk_wait_group<0>();   // all reductions have landed before the CTA exits
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 2) tmem_dealloc(tmem, 512);
    if (tid == 0 && abort_flag) report_status(p.status_buf, MPIPE_ERR_TIMEOUT, int32_t(blockIdx.x));
}

// Delta[h,t] = sum_d dO[t,h,d] * O[t,h,d], and the fp32 dQ accumulator is cleared.  HBM-bound helper:
// kLanes lanes share one (t,h) row (16 bytes of dO and of O each, coalesced across the row), partial
// dot products are combined with shuffles; the accumulator is cleared with flat 16-byte stores.
template <int D>
__global__ void __launch_bounds__(256)
bwd_prepass_kernel(const __nv_bfloat16* __restrict__ dout, const __nv_bfloat16* __restrict__ o, int64_t tok_stride_o,
                   int64_t head_stride_o, int32_t total_tokens, int32_t n_heads, float* __restrict__ delta,
                   float* __restrict__ dq_acc) {
    constexpr int kLanes = (D == 64) ? 8 : 16;   // lanes per row (D = 80 uses 10 of 16)
    constexpr int kRowsPerBlock = 256 / kLanes;
    const int64_t n_rows = int64_t(total_tokens) * n_heads;
    const int sub = threadIdx.x % kLanes;
    for (int64_t row0 = int64_t(blockIdx.x) * kRowsPerBlock; row0 < n_rows; row0 += int64_t(gridDim.x) * kRowsPerBlock) {
        const int64_t idx = row0 + threadIdx.x / kLanes;
        float acc = 0.f;
        int t = 0, h = 0;
        if (idx < n_rows) {
            t = int(idx / n_heads);
            h = int(idx % n_heads);
            if (sub * 8 < D) {
                const uint4 x = __ldg(reinterpret_cast<const uint4*>(dout + t * tok_stride_o + h * head_stride_o) + sub);
                const uint4 y = __ldg(reinterpret_cast<const uint4*>(o + t * tok_stride_o + h * head_stride_o) + sub);
                const uint32_t xs[4] = {x.x, x.y, x.z, x.w}, ys[4] = {y.x, y.y, y.z, y.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    acc = fmaf(__uint_as_float(xs[e] << 16), __uint_as_float(ys[e] << 16), acc);
                    acc = fmaf(__uint_as_float(xs[e] & 0xFFFF0000u), __uint_as_float(ys[e] & 0xFFFF0000u), acc);
                }
            }
        }
#pragma unroll
        for (int m = kLanes / 2; m > 0; m >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, m);
        if (idx < n_rows && sub == 0) delta[int64_t(h) * total_tokens + t] = acc;
        // clear the accumulator rows of this block: kRowsPerBlock * D floats, contiguous
        const int64_t z0 = row0 * D;
        const int64_t z1 = (row0 + kRowsPerBlock < n_rows ? row0 + kRowsPerBlock : n_rows) * D;
        float4* z = reinterpret_cast<float4*>(dq_acc);
        for (int64_t i = z0 / 4 + threadIdx.x; i < z1 / 4; i += 256) z[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
}

// dQ[t,h,:] = scale * acc[t,h,:] as bf16.  One thread per 8 elements.
__global__ void __launch_bounds__(256)
bwd_dq_convert_kernel(const float* __restrict__ acc, __nv_bfloat16* __restrict__ dq, int64_t tok_stride_g,
                      int64_t head_stride_g, int32_t total_tokens, int32_t n_heads, int32_t head_dim, float scale) {
    const int chunks = head_dim / 8;
    const int64_t idx = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (idx >= int64_t(total_tokens) * n_heads * chunks) return;
    const int c = int(idx % chunks);
    const int64_t th = idx / chunks;
    const int h = int(th % n_heads);
    const int64_t t = th / n_heads;
    const float4* src = reinterpret_cast<const float4*>(acc + th * head_dim + c * 8);
    const float4 x = __ldg(src), y = __ldg(src + 1);
    uint4 out;
    out.x = pack_bf16(x.x * scale, x.y * scale);
    out.y = pack_bf16(x.z * scale, x.w * scale);
    out.z = pack_bf16(y.x * scale, y.y * scale);
    out.w = pack_bf16(y.z * scale, y.w * scale);
    *reinterpret_cast<uint4*>(dq + t * tok_stride_g + h * head_stride_g + c * 8) = out;
}

template <int D>
static int32_t launch_bwd(const void* dout, const void* q, const void* k, const void* v, const void* o, void* dq,
                          int64_t ts_qkv, int64_t hs_qkv, int64_t ts_o, int64_t hs_o, int32_t total_tokens,
                          int32_t n_heads, BwdParams prm, float* delta, float* dq_acc, cudaStream_t stream) {
    using Cfg = BwdCfg<D>;
    BwdMaps m;
    if (!make_tensor_map_thd(&m.q, q, total_tokens, n_heads, D, ts_qkv, hs_qkv, 64, kQS, 128) ||
        !make_tensor_map_thd(&m.k, k, total_tokens, n_heads, D, ts_qkv, hs_qkv, 64, kBT, 128) ||
        !make_tensor_map_thd(&m.v, v, total_tokens, n_heads, D, ts_qkv, hs_qkv, 64, kBT, 128) ||
        !make_tensor_map_thd(&m.dout, dout, total_tokens, n_heads, D, ts_o, hs_o, 64, kQS, 128) ||
        !make_tensor_map_thd(&m.dq_acc, dq_acc, total_tokens, n_heads, D, int64_t(n_heads) * D, D, 32, kBT, 128, 4))
        return MPIPE_ERR_CUDA;
    m.q_tail = m.q, m.k_tail = m.k, m.v_tail = m.v, m.dout_tail = m.dout, m.dq_acc_tail = m.dq_acc;
    if (Cfg::kTail) {
        if (!make_tensor_map_thd(&m.q_tail, q, total_tokens, n_heads, D, ts_qkv, hs_qkv, 16, kQS, 32) ||
            !make_tensor_map_thd(&m.k_tail, k, total_tokens, n_heads, D, ts_qkv, hs_qkv, 16, kBT, 32) ||
            !make_tensor_map_thd(&m.v_tail, v, total_tokens, n_heads, D, ts_qkv, hs_qkv, 16, kBT, 32) ||
            !make_tensor_map_thd(&m.dout_tail, dout, total_tokens, n_heads, D, ts_o, hs_o, 16, kQS, 32) ||
            !make_tensor_map_thd(&m.dq_acc_tail, dq_acc, total_tokens, n_heads, D, int64_t(n_heads) * D, D, 16, kBT, 64, 4))
            return MPIPE_ERR_CUDA;
    }
    if (!ensure_dynamic_smem<attn_bwd_kernel<D>>(Cfg::kSmemAlloc)) return MPIPE_ERR_CUDA;
    const int64_t rows = int64_t(total_tokens) * n_heads;
    const int64_t prepass_blocks = (rows + (D == 64 ? 32 : 16) - 1) / (D == 64 ? 32 : 16);
    const int64_t prepass_cap = int64_t(sm_count()) * 64;
    bwd_prepass_kernel<D><<<unsigned(prepass_blocks < prepass_cap ? prepass_blocks : prepass_cap), 256, 0, stream>>>(
        static_cast<const __nv_bfloat16*>(dout), static_cast<const __nv_bfloat16*>(o), ts_o, hs_o, total_tokens, n_heads,
        delta, dq_acc);
    const int n_units = prm.n_items * prm.n_heads;
    const int grid = n_units < sm_count() ? n_units : sm_count();
    profile_start(kProfileBwdMain, stream);
    attn_bwd_kernel<D><<<grid, kBwdThreads, Cfg::kSmemAlloc, stream>>>(m, prm);
    profile_stop(kProfileBwdMain, stream);
    const int64_t chunks = rows * (D / 8);
    bwd_dq_convert_kernel<<<unsigned((chunks + 255) / 256), 256, 0, stream>>>(
        dq_acc, static_cast<__nv_bfloat16*>(dq), prm.tok_stride_g, prm.head_stride_g, total_tokens, n_heads, D,
        prm.scale);
    return cudaGetLastError() == cudaSuccess ? MPIPE_OK : MPIPE_ERR_CUDA;
}

static size_t round256(size_t x) { return (x + 255) & ~size_t(255); }

}  // namespace mpipe

extern "C" {


int32_t mpipe_bwd_tile_rows(void) { return mpipe::kBT; }

size_t mpipe_attn_workspace_bytes(int32_t total_tokens, int32_t n_heads, int32_t head_dim, int32_t mode) {
    if (mode != MPIPE_ENC_TRAINED || total_tokens <= 0 || n_heads <= 0 || head_dim <= 0) return 0;
    return mpipe::round256(size_t(total_tokens) * n_heads * head_dim * 4) +
           mpipe::round256(size_t(total_tokens) * n_heads * 4);
}

namespace {
// Argument checks shared by the two backward entry points.  Returns MPIPE_OK when the call may go on;
// *nothing_to_do is set when it is complete without a launch (frozen encoder, no tokens, no items).
int32_t bwd_check_args(const void* dout, const void* q, const void* k, const void* v, const void* o, const float* lse,
                       const void* dq, const void* dk, const void* dv, int64_t tok_stride_qkv, int64_t head_stride_qkv,
                       int64_t tok_stride_o, int64_t head_stride_o, int64_t tok_stride_grad, int64_t head_stride_grad,
                       const int32_t* cu_seqlens_dev, int32_t n_seg, int32_t total_tokens, int32_t max_seqlen,
                       const mpipe_work_item_t* bwd_items_dev, int32_t n_bwd_items, int32_t n_heads, int32_t head_dim,
                       float softmax_scale, int32_t mode, bool* nothing_to_do) {
    using namespace mpipe;
    *nothing_to_do = true;
    if (mode != MPIPE_ENC_FROZEN && mode != MPIPE_ENC_TRAINED) return MPIPE_ERR_INVALID_ARG;
    if (mode == MPIPE_ENC_FROZEN) return MPIPE_OK;  // Lemma 1: a frozen encoder has no backward event
    if (n_seg < 0 || total_tokens < 0 || max_seqlen < 0 || n_bwd_items < 0 || n_heads <= 0) return MPIPE_ERR_INVALID_ARG;
    if (head_dim != 64 && head_dim != 80) return MPIPE_ERR_UNSUPPORTED;
    if (total_tokens == 0 || n_bwd_items == 0) return MPIPE_OK;
    if (dout == nullptr || q == nullptr || k == nullptr || v == nullptr || o == nullptr || lse == nullptr ||
        dq == nullptr || dk == nullptr || dv == nullptr || bwd_items_dev == nullptr || cu_seqlens_dev == nullptr)
        return MPIPE_ERR_INVALID_ARG;
    if (!aligned16(dout) || !aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(dq) ||
        !aligned16(dk) || !aligned16(dv))
        return MPIPE_ERR_INVALID_ARG;
    if ((tok_stride_qkv & 7) || (head_stride_qkv & 7) || (tok_stride_o & 7) || (head_stride_o & 7) ||
        (tok_stride_grad & 7) || (head_stride_grad & 7))
        return MPIPE_ERR_INVALID_ARG;
    if (head_stride_qkv < head_dim || head_stride_o < head_dim || head_stride_grad < head_dim ||
        tok_stride_qkv < head_dim || tok_stride_o < head_dim || tok_stride_grad < head_dim)
        return MPIPE_ERR_INVALID_ARG;
    if (!(softmax_scale > 0.f) || !(softmax_scale < 1e30f)) return MPIPE_ERR_INVALID_ARG;
    if (int64_t(n_bwd_items) * n_heads >= (int64_t(1) << 31)) return MPIPE_ERR_INVALID_ARG;
    *nothing_to_do = false;
    return MPIPE_OK;
}
}  // namespace

int32_t mpipe_varlen_attn_bwd(const void* dout, const void* q, const void* k, const void* v, const void* o,
                              const float* lse, void* dq, void* dk, void* dv, int64_t tok_stride_qkv,
                              int64_t head_stride_qkv, int64_t tok_stride_o, int64_t head_stride_o,
                              int64_t tok_stride_grad, int64_t head_stride_grad, const int32_t* cu_seqlens_dev,
                              int32_t n_seg, int32_t total_tokens, int32_t max_seqlen,
                              const mpipe_work_item_t* bwd_items_dev, int32_t n_bwd_items, int32_t n_heads,
                              int32_t head_dim, float softmax_scale, int32_t mode, void* workspace,
                              size_t workspace_bytes, int32_t* status_buf, void* stream) {
    using namespace mpipe;
    bool nothing_to_do = false;
    const int32_t chk = bwd_check_args(dout, q, k, v, o, lse, dq, dk, dv, tok_stride_qkv, head_stride_qkv, tok_stride_o,
                                       head_stride_o, tok_stride_grad, head_stride_grad, cu_seqlens_dev, n_seg,
                                       total_tokens, max_seqlen, bwd_items_dev, n_bwd_items, n_heads, head_dim,
                                       softmax_scale, mode, &nothing_to_do);
    if (chk != MPIPE_OK || nothing_to_do) return chk;
    const size_t need = mpipe_attn_workspace_bytes(total_tokens, n_heads, head_dim, mode);
    if (workspace == nullptr || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0)
        return MPIPE_ERR_WORKSPACE;

    float* dq_acc = static_cast<float*>(workspace);
    float* delta = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) +
                                            round256(size_t(total_tokens) * n_heads * head_dim * 4));
    BwdParams prm;
    prm.items = bwd_items_dev;
    prm.n_items = n_bwd_items;
    prm.n_heads = n_heads;
    prm.total_tokens = total_tokens;
    prm.lse = lse;
    prm.delta = delta;
    prm.dk = static_cast<__nv_bfloat16*>(dk);
    prm.dv = static_cast<__nv_bfloat16*>(dv);
    prm.tok_stride_g = tok_stride_grad;
    prm.head_stride_g = head_stride_grad;
    prm.scale = softmax_scale;
    prm.scale_log2 = softmax_scale * 1.4426950408889634f;
    prm.status_buf = status_buf;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (head_dim == 64)
        return launch_bwd<64>(dout, q, k, v, o, dq, tok_stride_qkv, head_stride_qkv, tok_stride_o, head_stride_o,
                              total_tokens, n_heads, prm, delta, dq_acc, st);
    return launch_bwd<80>(dout, q, k, v, o, dq, tok_stride_qkv, head_stride_qkv, tok_stride_o, head_stride_o,
                          total_tokens, n_heads, prm, delta, dq_acc, st);
}


// ---------------------------------------------------------------------------------------------
// Backward for callers that cannot allocate: the scratch lives inside the library.
// ---------------------------------------------------------------------------------------------
namespace {

// Scratch of mpipe_varlen_attn_bwd_static: fp32 dQ accumulator + Delta of one call.  Every GPU that
// loads this library carries these 32 MiB from load until the process exits.
constexpr size_t kStaticScratchBytes = size_t(32) << 20;
static __device__ __align__(256) unsigned char g_bwd_static_scratch[kStaticScratchBytes];

// Device address of the array, looked up once per device.  On the host the array's name is only a
// stand-in symbol, not a device address, so kernels must be given the looked-up pointer.  The cache is
// plain host memory without a lock: two host threads that make their first call on a device at the same
// time both look the address up and store the same value.
void* g_bwd_static_scratch_ptr[64] = {nullptr};

int32_t static_scratch_for_current_device(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return MPIPE_ERR_CUDA;
    if (g_bwd_static_scratch_ptr[dev] == nullptr) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_bwd_static_scratch) != cudaSuccess || ptr == nullptr) {
            (void)cudaGetLastError();
            return MPIPE_ERR_CUDA;
        }
        g_bwd_static_scratch_ptr[dev] = ptr;
    }
    *out = g_bwd_static_scratch_ptr[dev];
    return MPIPE_OK;
}

}  // namespace

size_t mpipe_attn_bwd_static_scratch_bytes(void) { return kStaticScratchBytes; }

int32_t mpipe_varlen_attn_bwd_static(const void* dout, const void* q, const void* k, const void* v, const void* o,
                                     const float* lse, void* dq, void* dk, void* dv, int64_t tok_stride_qkv,
                                     int64_t head_stride_qkv, int64_t tok_stride_o, int64_t head_stride_o,
                                     int64_t tok_stride_grad, int64_t head_stride_grad,
                                     const int32_t* cu_seqlens_dev, int32_t n_seg, int32_t total_tokens,
                                     int32_t max_seqlen, const mpipe_work_item_t* bwd_items_dev, int32_t n_bwd_items,
                                     int32_t n_heads, int32_t head_dim, float softmax_scale, int32_t mode,
                                     int32_t* status_buf, void* stream) {
    // The same checks, in the same order, as mpipe_varlen_attn_bwd: a bad argument gets the same status from both.
    bool nothing_to_do = false;
    const int32_t chk = bwd_check_args(dout, q, k, v, o, lse, dq, dk, dv, tok_stride_qkv, head_stride_qkv, tok_stride_o,
                                       head_stride_o, tok_stride_grad, head_stride_grad, cu_seqlens_dev, n_seg,
                                       total_tokens, max_seqlen, bwd_items_dev, n_bwd_items, n_heads, head_dim,
                                       softmax_scale, mode, &nothing_to_do);
    if (chk != MPIPE_OK || nothing_to_do) return chk;
    // The problem must fit the built-in scratch; larger ones have to use mpipe_varlen_attn_bwd.
    if (mpipe_attn_workspace_bytes(total_tokens, n_heads, head_dim, mode) > kStaticScratchBytes)
        return MPIPE_ERR_WORKSPACE;
    void* scratch = nullptr;
    const int32_t rc = static_scratch_for_current_device(&scratch);
    if (rc != MPIPE_OK) return rc;
    return mpipe_varlen_attn_bwd(dout, q, k, v, o, lse, dq, dk, dv, tok_stride_qkv, head_stride_qkv, tok_stride_o,
                                 head_stride_o, tok_stride_grad, head_stride_grad, cu_seqlens_dev, n_seg,
                                 total_tokens, max_seqlen, bwd_items_dev, n_bwd_items, n_heads, head_dim,
                                 softmax_scale, mode, scratch, kStaticScratchBytes, status_buf, stream);
}

}  // extern "C"
