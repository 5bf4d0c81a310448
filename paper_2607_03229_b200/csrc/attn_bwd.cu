// mpipe_varlen_attn_bwd: gradient of the per-image softmax attention, the attention part of the
// optional Bwd(enc, r, m) event (it exists only when trainable(enc), Lemma 1).
//
// Three launches on the caller's stream:
//   1. prepass   Delta[h,t] = sum_d dO[t,h,d] O[t,h,d]  and the fp32 dQ accumulator is cleared
//   2. main      one persistent CTA per SM walks (key tile x head) units; a unit keeps one 128-key
//                K/V tile resident and steps through the 128-row query tiles of the same segment
//   3. convert   dQ = softmax_scale * accumulator -> bf16
//
// Main kernel, per step = one [128 keys x 128 queries] block (everything transposed so that the key index is the
// TMEM lane):
//   S^T  = K Q^T            tcgen05, N = 128, operands in shared memory          -> TMEM (128 columns)
//   dP^T = V dO^T           tcgen05, N = 128                                      -> TMEM (128 columns)
//   P^T  = exp2(scale*log2e * (S^T - LSE/scale))     softmax warps, written over S^T as bf16
//   dS^T = P^T o (dP^T - Delta)                      softmax warps, over dP^T as bf16 + to shared memory
// The row terms -LSE_q / scale and -Delta_q are ADDED BY THE TENSOR CORE: each of the two score products runs one
// more 16-element K-step whose key-side operand is a column of ones and whose query-side operand holds the term
// split into three bf16 parts (24 bits, i.e. all of the fp32 value).  The softmax warps then need no per-query
// value at all -- fetching 128 of them per thread and step from shared memory, whose port the operand reads of the
// MMAs keep busy, was the largest single cost of a step (about a sixth of it).
//   dV  += P^T dO           tcgen05, A operand read from TMEM, dO as MN-major B, N = head_dim
//   dK  += dS^T Q           tcgen05, A operand read from TMEM, Q as MN-major B
//   dQ_i = dS K             tcgen05, dS^T in shared memory read as an MN-major A, K as MN-major B
// dQ_i is read back from TMEM by a reducer warpgroup, staged in shared memory and added to the global fp32
// accumulator by the copy engine (cp.reduce.async.bulk.tensor, fp32 add): the order of those additions is not
// fixed, so the low bits of dQ can differ from run to run.  dK (x softmax_scale) and dV leave TMEM once per unit.
//
// The block is as large as the TMEM budget allows (S^T 128 + dP^T 128 + dV, dK, dQ head_dim columns each) because
// the kernel is bound by the NUMBER of tcgen05.mma instructions its one issuing thread gets through and by the
// barrier hops between that thread and the softmax warps, not by the tensor pipe: a 128 x 128 step takes 32 MMAs
// (34 at head_dim 80) and four hops; two 64-query half steps took 40 (68) and eight.
//
// Warp roles (512 threads): 0 TMA producer, 1 tcgen05 issuer, 2 TMEM allocation and LSE/Delta staging, 4-11 softmax
// (thread = key row; warps 4-7 take query columns 0-63 of the block, warps 8-11 columns 64-127), 12-15 dQ reducer
// and epilogue.  Every wait is bounded (see sm100_ptx.cuh); expiry sets status_buf and drains the CTA.
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
constexpr int kBQ = 128;  // query rows per step
constexpr int kQH = 64;   // query columns of a step handled by one softmax warpgroup

// Shared-memory layout of a [128 rows x head_dim] bf16 tile.  head_dim 64: one TMA box, rows of 128 bytes, 128-byte
// swizzle.  head_dim 80: three boxes of 32 elements (rows of 64 bytes, 64-byte swizzle) 8 KB apart, the last one half
// beyond the tensor and zero-filled by TMA; with a single swizzle mode over the whole row a tile serves as a K-major
// operand (five 16-element K-steps) and, as an MN-major operand, as ONE N = 80 operand (two and a half 32-element
// atoms) -- a 64 + 16 split needs two MMA instructions for every product over the head dimension.
template <int D>
struct BwdCfg {
    static constexpr int kBoxElems = (D == 64) ? 64 : 32;
    static constexpr int kBoxes = (D == 64) ? 1 : 3;
    static constexpr int kRowBytes = kBoxElems * 2;
    static constexpr int kBoxBytes = 128 * kRowBytes;             // 16 KB / 8 KB
    static constexpr int kTile = kBoxes * kBoxBytes;              // K, V, Q, dO tiles: 16 KB / 24 KB
    static constexpr uint32_t kSwz = (D == 64) ? kSwizzle128 : kSwizzle64;
    static constexpr uint32_t kSBO = 8 * kRowBytes;               // 8 rows of one box
    static constexpr int kKSteps = D / 16;                        // K-steps of a product over the head dimension
    static constexpr int kKVBufs = (D == 64) ? 2 : 1;             // 2: the next unit's K/V tiles load during the current unit
    static constexpr int kRing = 2;                               // Q / dO / row-term stages
    // One more 16-element K-step carries the per-query row terms into the two score products (see the staging warp):
    // [128 rows][32 bytes] operands, 32-byte swizzle.
    static constexpr int kExtra = 128 * 32;
    // dQ staging for the TMA reduction: 16 fp32 columns at a time through three rotating [128 q][16 fp32] boxes
    // (rows of 64 bytes, 64-byte swizzle), so that the copy engine reads two boxes while the third is being filled
    static constexpr int kStageBox = kBQ * 64;
    static constexpr int kStageBoxes = 3;
    static constexpr int kStageBytes = kStageBoxes * kStageBox;
    static constexpr int kSmemK = 0;                              // buffer i at i * 2 * kTile (K then V)
    static constexpr int kSmemV = kTile;
    static constexpr int kSmemQ = kKVBufs * 2 * kTile;
    static constexpr int kSmemDO = kSmemQ + kRing * kTile;
    static constexpr int kDSBytes = 2 * kBT * 128;                // dS^T of a step as [key][q]: two 64-query atoms of 16 KB
    static constexpr int kSmemDS = kSmemDO + kRing * kTile;
    static constexpr int kSmemStage = kSmemDS + kDSBytes;
    static constexpr int kSmemOnes = kSmemStage + kStageBytes;    // the key-side operand of the extra K-step (constant)
    static constexpr int kSmemQX = kSmemOnes + kExtra;            // kRing x query-side operand for S^T (-LSE / softmax_scale)
    static constexpr int kSmemDOX = kSmemQX + kRing * kExtra;     // kRing x query-side operand for dP^T (-Delta)
    static constexpr int kSmemTotal = kSmemDOX + kRing * kExtra;
    static constexpr int kSmemAlloc = kSmemTotal + 1024;
    // TMEM columns; P^T / dS^T (bf16) overlay the first 32 columns of each warpgroup's 64-column half of S^T / dP^T
    static constexpr int kColS = 0, kColDP = 128, kColDV = 256, kColDK = 256 + D, kColDQ = 256 + 2 * D;
    // head_dim 64 leaves 64 columns: P^T (128 queries as bf16) gets them instead of overlaying S^T.  The next step's
    // S^T can then be issued as soon as the softmax warps have READ the current one, not only after dV has consumed
    // P^T, which takes the issuing thread and the tensor pipe out of the softmax warps' step-to-step loop.
    static constexpr bool kPSeparate = (kColDQ + D + kBQ / 2 <= 512);
    static constexpr int kColP = kPSeparate ? kColDQ + D : kColS;
    static constexpr int kPStride = kPSeparate ? kQH / 2 : kQH;   // columns between the two warpgroups' halves of P^T
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
    uint64_t kv_full[2], kv_empty[2], dkv_full, dkv_empty;
    uint64_t qdo_full[4], qdo_empty[4];
    uint64_t s_full, s_read, p_full, pv_done, dp_full, ds_full, dq_full, dq_empty;
};

struct BwdMaps {
    CUtensorMap q, k, v, dout, dq_acc;
};

template <int D>
__global__ void __maxnreg__(kRegsLaunch)
attn_bwd_kernel(const __grid_constant__ BwdMaps maps, const BwdParams p) {
    using Cfg = BwdCfg<D>;
    constexpr int NR = Cfg::kRing;
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
            mbar_init(&bars.kv_empty[i], 1);
        }
        mbar_init(&bars.dkv_full, 1);
        mbar_init(&bars.dkv_empty, 4);
        for (int s = 0; s < 4; ++s) {
            mbar_init(&bars.qdo_full[s], 2);    // the producer's expect_tx arrival + the staging warp
            mbar_init(&bars.qdo_empty[s], 1);
        }
        mbar_init(&bars.s_full, 1);
        mbar_init(&bars.s_read, 8);             // (separate P^T only) S^T is in the softmax warps' registers
        mbar_init(&bars.pv_done, 1);            // (separate P^T only) dV has consumed P^T
        mbar_init(&bars.p_full, 8);             // one arrival per softmax warp
        mbar_init(&bars.dp_full, 1);
        mbar_init(&bars.ds_full, 8);
        mbar_init(&bars.dq_full, 1);
        mbar_init(&bars.dq_empty, 4);           // one arrival per reducer warp
        fence_mbar_init();
    }
    if (warp == 2) {
        tmem_alloc(&tmem_base_slot, 512);
        tmem_relinquish();
    }
    if (tid >= 128 && tid < 256) {
        // Key-side operand of the extra K-step: every row is (1, 1, 1, 0 x 5 | 1, 1, 1, 0 x 5).  The query-side rows carry
        // their three parts in the first 16-byte half only and zeros in the second, so the dot product is the sum of
        // the three parts whichever way the 32-byte swizzle orders a row's two halves.
        uint4* row = reinterpret_cast<uint4*>(smem + Cfg::kSmemOnes + (tid - 128) * 32);
        row[0] = row[1] = make_uint4(0x3F803F80u, 0x00003F80u, 0u, 0u);
        fence_async_smem();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_slot;
    // The plan comes from device memory: it is checked as a whole before any role starts (see plan_ok_cta); a
    // rejected plan leaves every role with nothing to do.
    __shared__ int plan_flag;
    const int n_units = plan_ok_cta(p.items, p.n_items, kBT, p.total_tokens, p.status_buf, &plan_flag) ? p.n_items * p.n_heads : 0;
    // Units are sorted by decreasing cost; CTAs walk them in boustrophedon order (0..G-1, then G-1..0, ...) so
    // that the CTA that got the most expensive unit of one round gets the cheapest of the next.
    auto unit_of = [&](int round) {
        const int g = int(gridDim.x), i = int(blockIdx.x);
        return round * g + ((round & 1) ? g - 1 - i : i);
    };
    // Unit u -> (work item, head).  The items of one segment are consecutive in the list (tile 0, 1, ...), and their
    // units occupy the same stretch of the unit sequence whichever way it is ordered inside.  Short segments: tile by
    // tile, heads innermost.  Segments of more than kHeadMajorTiles key tiles: head by head, so that the CTAs running
    // at the same time share the Q / dO tiles and the dQ accumulator of one or two heads through L2 instead of all
    // heads' at once (16 heads x 16 384 tokens of Q, dO and fp32 dQ do not fit in L2 beside K and V; DRAM traffic of
    // the Qwen2-VL-like backward was 6.4 x the algorithmic bytes).  The head is returned in the item's `seg` field,
    // which the kernel does not otherwise use.
    constexpr int kHeadMajorTiles = 32;
    auto item_at = [&](int u) {
        mpipe_work_item_t z = {0, 0, 0, 0, 0, 0};
        if (u >= n_units) return z;
        const int i0 = u / p.n_heads;
        const mpipe_work_item_t a = p.items[i0];
        const int nt = (a.kv_len + kBT - 1) / kBT;                   // key tiles of this item's segment
        if (nt <= kHeadMajorTiles) {
            z = a;
            z.seg = u % p.n_heads;
            return z;
        }
        const int first = i0 - a.tile;                               // the segment's first item
        const int l = u - first * p.n_heads;
        const int head = l / nt;
        z = p.items[min(max(first + (l - head * nt), 0), p.n_items - 1)];
        z.seg = min(max(head, 0), p.n_heads - 1);
        return z;
    };
    // Steps of a unit: the 128-query tiles of the segment; rows of the last one past the segment end contribute
    // nothing because their probabilities are forced to zero.
    auto steps_of = [](const mpipe_work_item_t& it) { return (it.kv_len + kBQ - 1) / kBQ; };
    // The j-th step of a unit works on query tile (j + key tile index) mod steps: the CTAs that hold the key tiles of
    // one (segment, head) run at the same time, and started on the same query tile they would all add to the same rows
    // of the dQ accumulator at once (fp32 adds to one address serialise in L2) and ask for the same Q / dO tile.
    auto q_tile_of = [](const mpipe_work_item_t& it, int j, int nq) { return (j + (it.tile >= 0 ? it.tile : 0)) % nq; };

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        setmaxnreg_dec<kRegsService>();
        if (lane == 0) {
            uint32_t unit_it = 0, sc = 0;
            bool ok = true;
            auto load_tile = [&](uint8_t* dst, const CUtensorMap* map, uint64_t* bar, int head, int row) {
#pragma unroll
                for (int bx = 0; bx < Cfg::kBoxes; ++bx)
                    tma_load_3d(dst + bx * Cfg::kBoxBytes, map, bar, bx * Cfg::kBoxElems, head, row);
            };
            mpipe_work_item_t it_next = item_at(unit_of(0));   // one unit ahead: the global load is off the unit's critical path
            for (int ur = 0, u = unit_of(0); u < n_units && ok; ++ur, u = unit_of(ur), ++unit_it) {
                const mpipe_work_item_t it = it_next;
                it_next = item_at(unit_of(ur + 1));
                const int head = it.seg;
                const int nq = steps_of(it);
                const int kb = unit_it % Cfg::kKVBufs;            // K/V buffer of this unit
                uint8_t* kv = smem + kb * (2 * Cfg::kTile);
                ok = mbar_wait<kSleepAux>(&bars.kv_empty[kb], ((unit_it / Cfg::kKVBufs) & 1) ^ 1, &abort_flag);
                if (!ok) break;
                mbar_expect_tx(&bars.kv_full[kb], 2 * Cfg::kTile);
                load_tile(kv + Cfg::kSmemK, &maps.k, &bars.kv_full[kb], head, it.row_start);
                load_tile(kv + Cfg::kSmemV, &maps.v, &bars.kv_full[kb], head, it.row_start);
                for (int j = 0; j < nq; ++j, ++sc) {
                    const int rs = sc % NR;
                    const int row = it.kv_start + q_tile_of(it, j, nq) * kBQ;
                    ok = mbar_wait<kSleepAux>(&bars.qdo_empty[rs], ((sc / NR) & 1) ^ 1, &abort_flag);
                    if (!ok) break;
                    mbar_expect_tx(&bars.qdo_full[rs], 2 * Cfg::kTile);
                    load_tile(smem + Cfg::kSmemQ + rs * Cfg::kTile, &maps.q, &bars.qdo_full[rs], head, row);
                    load_tile(smem + Cfg::kSmemDO + rs * Cfg::kTile, &maps.dout, &bars.qdo_full[rs], head, row);
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ tcgen05 issuer
        // The whole warp walks the loop (uniform control flow); one elected lane issues and commits.
        // Descriptors are precomputed halves: a K-step only adds a constant to the low word.
        // Issue order per step j:  dV(j), S^T(j+1) | dK(j), dQ(j), dP^T(j+1).  S^T(j+1) goes out as soon as the P^T that
        // overlays S^T(j) has been consumed, so that the softmax warps find it ready when they return from dS^T(j).
        setmaxnreg_dec<kRegsService>();
        {
            const bool leader = elect_one();
            const uint32_t sbase = smem_u32(smem);
            constexpr uint32_t hi_t = umma_desc_hi(Cfg::kSBO, Cfg::kSwz);      // Q / K / V / dO tiles
            constexpr uint32_t hi128 = umma_desc_hi(1024, kSwizzle128);        // the dS^T tile
            constexpr uint32_t idesc_s = umma_idesc_bf16(kBT, kBQ, 0, 0);      // K-major x K-major, N = 128 queries
            constexpr uint32_t idesc_ts = umma_idesc_bf16(kBT, D, 0, 1);       // A in TMEM, MN-major B, N = head_dim
            constexpr uint32_t idesc_dq = umma_idesc_bf16(kBQ, D, 1, 1);       // MN-major A and B
            // low descriptor words (16-byte units).  K-major use of a tile: K-step ks starts (ks % per_box) * 32 bytes into
            // box ks / per_box.  MN-major use: rows are the contraction index, 16 rows per K-step; LBO = box stride.
            constexpr uint32_t kPerBox = Cfg::kBoxElems / 16;
            auto kmaj = [&](uint32_t lo, int ks) { return lo + uint32_t(ks / kPerBox) * (Cfg::kBoxBytes >> 4) + uint32_t(ks % kPerBox) * 2; };
            constexpr uint32_t kMnStep = (16 * Cfg::kRowBytes) >> 4;
            const uint32_t ds_lo = umma_desc_lo(sbase + Cfg::kSmemDS, kBT * 128);   // two 64-query atoms 16 KB apart
            const uint32_t q_lo0 = umma_desc_lo(sbase + Cfg::kSmemQ, 0), do_lo0 = umma_desc_lo(sbase + Cfg::kSmemDO, 0);
            const uint32_t q_mn0 = umma_desc_lo(sbase + Cfg::kSmemQ, Cfg::kBoxBytes), do_mn0 = umma_desc_lo(sbase + Cfg::kSmemDO, Cfg::kBoxBytes);
            auto stage_off = [&](uint32_t c) { return (c % NR) * uint32_t(Cfg::kTile >> 4); };
            constexpr uint32_t hi32 = umma_desc_hi(256, kSwizzle32);           // the extra K-step's operands
            const uint32_t ones_lo = umma_desc_lo(sbase + Cfg::kSmemOnes, 0);
            const uint32_t qx_lo0 = umma_desc_lo(sbase + Cfg::kSmemQX, 0), dox_lo0 = umma_desc_lo(sbase + Cfg::kSmemDOX, 0);
            auto extra_off = [&](uint32_t c) { return (c % NR) * uint32_t(Cfg::kExtra >> 4); };
            // dst[128 keys x 128 q] = A[128 x D] * B[128 x D]^T + 1 * x[q]: both K-major, then the row-term K-step
            auto issue_kk = [&](uint32_t dcol, uint32_t a_lo, uint32_t b_lo, uint32_t x_lo) {
                if (leader) {
#pragma unroll
                    for (int ks = 0; ks < Cfg::kKSteps; ++ks)
                        umma_ss(tmem + dcol, umma_desc(kmaj(a_lo, ks), hi_t), umma_desc(kmaj(b_lo, ks), hi_t), idesc_s, ks > 0);
                    umma_ss(tmem + dcol, umma_desc(ones_lo, hi32), umma_desc(x_lo, hi32), idesc_s, 1);
                }
            };
            // dst[128 keys x D] (+)= A^T-in-TMEM[128 keys x 128 q] * B[128 q x D] (B rows = q, MN-major)
            auto issue_ts = [&](uint32_t dcol, uint32_t acol, uint32_t astride, uint32_t b_mn, bool acc) {
                if (leader) {
#pragma unroll
                    for (int ks = 0; ks < kBQ / 16; ++ks)
                        umma_ts(tmem + dcol, tmem + acol + (ks >> 2) * astride + (ks & 3) * 8, umma_desc(b_mn + ks * kMnStep, hi_t), idesc_ts,
                                (acc || ks > 0) ? 1u : 0u);
                }
            };
            uint32_t unit_it = 0, sc = 0;   // sc: global step counter at the start of the unit
            bool ok = true;
            mpipe_work_item_t it_next = item_at(unit_of(0));   // one unit ahead: the global load is off the unit's critical path
            for (int ur = 0, u = unit_of(0); u < n_units && ok; ++ur, u = unit_of(ur), ++unit_it) {
                const mpipe_work_item_t it = it_next;
                it_next = item_at(unit_of(ur + 1));
                const int nq = steps_of(it);
                const int kb = unit_it % Cfg::kKVBufs;
                const uint32_t kvb = sbase + kb * (2 * Cfg::kTile);
                const uint32_t k_lo = umma_desc_lo(kvb + Cfg::kSmemK, 0), v_lo = umma_desc_lo(kvb + Cfg::kSmemV, 0);
                const uint32_t k_mn = umma_desc_lo(kvb + Cfg::kSmemK, Cfg::kBoxBytes);
                // With two K/V buffers the stream of steps runs on across the unit boundary: S^T / dP^T of the next unit's
                // first step are issued inside this unit's last step, from the other (prefetched) buffer, so the softmax
                // warps never see the pipeline drain between units.
                constexpr bool kStream = (Cfg::kKVBufs == 2);
                const bool has_next = kStream && unit_of(ur + 1) < n_units;
                const uint32_t kvb_n = sbase + (kb ^ 1) * (2 * Cfg::kTile);
                const uint32_t k_lo_n = umma_desc_lo(kvb_n + Cfg::kSmemK, 0), v_lo_n = umma_desc_lo(kvb_n + Cfg::kSmemV, 0);
                ok = mbar_wait(&bars.kv_full[kb], (unit_it / Cfg::kKVBufs) & 1, &abort_flag);
                if (!ok) break;
                if (!kStream || unit_it == 0) {   // prologue: S^T and dP^T of the unit's first step
                    ok = mbar_wait(&bars.qdo_full[sc % NR], (sc / NR) & 1, &abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    issue_kk(Cfg::kColS, k_lo, q_lo0 + stage_off(sc), qx_lo0 + extra_off(sc));
                    if (leader) umma_commit(&bars.s_full);
                    issue_kk(Cfg::kColDP, v_lo, do_lo0 + stage_off(sc), dox_lo0 + extra_off(sc));
                    if (leader) umma_commit(&bars.dp_full);
                }
                for (int j = 0; j < nq && ok; ++j) {
                    const uint32_t c = sc + j;
                    const uint32_t ph = c & 1;
                    const bool cross = (j + 1 == nq) && has_next;   // step j+1 is the next unit's first
                    const bool more = (j + 1 < nq) || cross;
                    auto issue_next_s = [&]() -> bool {   // S^T(j+1), from the next unit's K tile at a unit's last step
                        if (cross) {   // the next unit's K/V tiles (loaded while this unit ran)
                            if (!mbar_wait(&bars.kv_full[kb ^ 1], ((unit_it + 1) / Cfg::kKVBufs) & 1, &abort_flag)) return false;
                        }
                        if (!mbar_wait(&bars.qdo_full[(c + 1) % NR], ((c + 1) / NR) & 1, &abort_flag)) return false;
                        tc_fence_after();
                        issue_kk(Cfg::kColS, cross ? k_lo_n : k_lo, q_lo0 + stage_off(c + 1), qx_lo0 + extra_off(c + 1));
                        if (leader) umma_commit(&bars.s_full);
                        return true;
                    };
                    if (Cfg::kPSeparate && more) {   // S^T(j) has been read: S^T(j+1) may replace it at once
                        ok = mbar_wait(&bars.s_read, ph, &abort_flag);
                        if (ok) ok = issue_next_s();
                        if (!ok) break;
                    }
                    ok = mbar_wait(&bars.p_full, ph, &abort_flag);
                    if (!ok) break;
                    if (j == 0) {   // the accumulators are free: the previous unit's epilogue has read them
                        ok = mbar_wait(&bars.dkv_empty, (unit_it & 1) ^ 1, &abort_flag);
                        if (!ok) break;
                    }
                    tc_fence_after();
                    issue_ts(Cfg::kColDV, Cfg::kColP, Cfg::kPStride, do_mn0 + stage_off(c), j > 0);               // dV += P^T dO
                    if (Cfg::kPSeparate) {
                        if (leader) umma_commit(&bars.pv_done);
                    } else if (more) {   // P^T overlays S^T: only now may S^T(j+1) be written
                        ok = issue_next_s();
                        if (!ok) break;
                    }
                    ok = mbar_wait(&bars.ds_full, ph, &abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    issue_ts(Cfg::kColDK, Cfg::kColDP, kQH, q_mn0 + stage_off(c), j > 0);                              // dK += dS^T Q
                    if (leader) umma_commit(&bars.qdo_empty[c % NR]);   // also frees the LSE / Delta stage (dS^T(j) has arrived)
                    ok = mbar_wait(&bars.dq_empty, ph ^ 1, &abort_flag);   // the reducer has taken dQ(j-1) out of TMEM
                    if (!ok) break;
                    tc_fence_after();
                    if (leader) {                                                                                 // dQ(j) = dS K
#pragma unroll
                        for (int ks = 0; ks < kBT / 16; ++ks)
                            umma_ss(tmem + Cfg::kColDQ, umma_desc(ds_lo + ks * 128, hi128), umma_desc(k_mn + ks * kMnStep, hi_t), idesc_dq, ks > 0);
                        umma_commit(&bars.dq_full);
                    }
                    if (more) {   // after dQ(j): its completion then implies that the dS^T tile in shared memory has been read
                        issue_kk(Cfg::kColDP, cross ? v_lo_n : v_lo, do_lo0 + stage_off(c + 1), dox_lo0 + extra_off(c + 1));   // dP^T(j+1)
                        if (leader) umma_commit(&bars.dp_full);
                    }
                }
                if (!ok) break;
                if (leader) umma_commit(&bars.dkv_full);
                if (leader) umma_commit(&bars.kv_empty[kb]);
                sc += nq;
            }
        }
        __syncwarp();
    } else if (warp == 2) {
        // ------------------------------------------------------------------ row-term staging
        // Per step and query q: x_q = -LSE_q / softmax_scale and y_q = -Delta_q, each split into three bf16 parts
        // (hi, then the remainder, then its remainder: together the fp32 value), written as the first three elements
        // of row q of the step's two extra-K-step operands.  Query rows past the segment end get a hugely negative x
        // (their probabilities become exp2(-large) = 0) and y = 0.
        setmaxnreg_dec<kRegsService>();
        uint32_t sc = 0;
        bool ok = true;
        const float inv_scale = 1.0f / p.scale;
        auto split3 = [](float a) {
            const __nv_bfloat16 h = __float2bfloat16_rn(a);
            const float r1 = a - __bfloat162float(h);
            const __nv_bfloat16 m = __float2bfloat16_rn(r1);
            const __nv_bfloat16 l = __float2bfloat16_rn(r1 - __bfloat162float(m));
            return make_uint4(uint32_t(__bfloat16_as_ushort(h)) | (uint32_t(__bfloat16_as_ushort(m)) << 16),
                              uint32_t(__bfloat16_as_ushort(l)), 0u, 0u);
        };
        mpipe_work_item_t it_next = item_at(unit_of(0));   // one unit ahead: the global load is off the unit's critical path
        for (int ur = 0, u = unit_of(0); u < n_units && ok; ++ur, u = unit_of(ur)) {
            const mpipe_work_item_t it = it_next;
            it_next = item_at(unit_of(ur + 1));
            const int head = it.seg;
            const int nq = steps_of(it);
            const int q_end = it.kv_start + it.kv_len;
            for (int j = 0; j < nq; ++j, ++sc) {
                const int rs = sc % NR;
                uint4* qx = reinterpret_cast<uint4*>(smem + Cfg::kSmemQX + rs * Cfg::kExtra);
                uint4* dox = reinterpret_cast<uint4*>(smem + Cfg::kSmemDOX + rs * Cfg::kExtra);
                const int q0 = it.kv_start + q_tile_of(it, j, nq) * kBQ;
                float xv[4], yv[4];   // read from global memory before the stage is known to be free: the latency overlaps the wait
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int q = q0 + lane + 32 * e;
                    const bool valid = q < q_end;
                    xv[e] = valid ? -__ldg(p.lse + int64_t(head) * p.total_tokens + q) * inv_scale : -3.0e38f;
                    yv[e] = valid ? -__ldg(p.delta + int64_t(head) * p.total_tokens + q) : 0.f;
                }
                // the stage is free when the MMAs that read the Q / dO tile it travels with have completed
                ok = mbar_wait<kSleepAux>(&bars.qdo_empty[rs], ((sc / NR) & 1) ^ 1, &abort_flag);
                if (!ok) break;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int row = lane + 32 * e;
                    qx[2 * row] = split3(xv[e]);
                    qx[2 * row + 1] = make_uint4(0u, 0u, 0u, 0u);
                    dox[2 * row] = split3(yv[e]);
                    dox[2 * row + 1] = make_uint4(0u, 0u, 0u, 0u);
                }
                fence_async_smem();   // generic-proxy writes, read by the tensor core
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars.qdo_full[rs]);
            }
        }
    } else if (warp == 3) {
        setmaxnreg_dec<kRegsService>();   // spare warp
    } else if (warp < 12) {
        // ------------------------------------------------------------------ softmax / dS warps
        // Thread = key row; warpgroup g takes query columns [64 g, 64 g + 64) of every step.
        setmaxnreg_inc<kRegsSoftmax>();
        const int g = (warp - 4) >> 2;
        const int r = ((warp & 3) << 5) | lane;
        const uint32_t lane_base = uint32_t((warp & 3) * 32) << 16;
        const uint32_t t_s = tmem + lane_base + Cfg::kColS + g * kQH;
        const uint32_t t_p = tmem + lane_base + Cfg::kColP + g * Cfg::kPStride;
        const uint32_t t_dp = tmem + lane_base + Cfg::kColDP + g * kQH;
        uint8_t* ds_row = smem + Cfg::kSmemDS + g * (kBT * 128) + r * 128;
        uint32_t sc = 0;   // global step counter at the start of the unit
        bool ok = true;
        mpipe_work_item_t it_next = item_at(unit_of(0));   // one unit ahead: the global load is off the unit's critical path
        for (int ur = 0, u = unit_of(0); u < n_units && ok; ++ur, u = unit_of(ur)) {
            const mpipe_work_item_t it = it_next;
            it_next = item_at(unit_of(ur + 1));
            const int nq = steps_of(it);
            const bool key_valid = r < it.row_len;
            const bool ragged_keys = it.row_len < kBT;
            for (int j = 0; j < nq; ++j) {
                const uint32_t c = sc + j;
                const uint32_t ph = c & 1;
                ok = mbar_wait(&bars.s_full, ph, &abort_flag);
                if (!ok) break;
                tc_fence_after();
                // P^T = exp2(scale*log2e * S'^T), S' already holding the row term: both 32-column halves are requested
                // before the one wait; packed fp32 pairs for the multiply
                float pr[64];
                {
                    uint32_t sr[64];
                    tmem_ld32(t_s, *reinterpret_cast<uint32_t(*)[32]>(&sr[0]));
                    tmem_ld32(t_s + 32, *reinterpret_cast<uint32_t(*)[32]>(&sr[32]));
                    tmem_wait_ld();
                    if (Cfg::kPSeparate) {   // the scores are in registers: the next step's S^T may be written
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&bars.s_read);
                    }
                    const float2 sc2 = make_float2(p.scale_log2, p.scale_log2);
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        uint32_t pk[16];
#pragma unroll
                        for (int c4 = 0; c4 < 8; ++c4) {
                            const int e = h * 32 + 4 * c4;
                            const float2 x01 = mul2(make_float2(__uint_as_float(sr[e]), __uint_as_float(sr[e + 1])), sc2);
                            const float2 x23 = mul2(make_float2(__uint_as_float(sr[e + 2]), __uint_as_float(sr[e + 3])), sc2);
                            pr[e] = ex2_approx(x01.x);
                            pr[e + 1] = ex2_approx(x01.y);
                            pr[e + 2] = ex2_approx(x23.x);
                            pr[e + 3] = ex2_approx(x23.y);
                            pk[2 * c4] = pack_bf16(pr[e], pr[e + 1]);
                            pk[2 * c4 + 1] = pack_bf16(pr[e + 2], pr[e + 3]);
                        }
                        if (Cfg::kPSeparate && h == 0 && c > 0) {   // dV(j-1) has read the previous P^T (long since, as a rule)
                            ok = mbar_wait(&bars.pv_done, (c - 1) & 1, &abort_flag);
                            tc_fence_after();
                        }
                        tmem_st16(t_p + h * 16, pk);   // (overlay: over this thread's own scores, which are in registers)
                    }
                    if (!ok) break;
                }
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars.p_full);

                // dP^T(j) complete also means dQ(j-1) has completed (issued before it, same thread): the dS^T tile in
                // shared memory may be overwritten
                ok = mbar_wait(&bars.dp_full, ph, &abort_flag);
                if (!ok) break;
                tc_fence_after();
                // dS^T = P^T o dP'^T (dP' already holding -Delta); key rows past the segment are zeroed on the packed words
                {
                    uint32_t dr[64];
                    tmem_ld32(t_dp, *reinterpret_cast<uint32_t(*)[32]>(&dr[0]));
                    tmem_ld32(t_dp + 32, *reinterpret_cast<uint32_t(*)[32]>(&dr[32]));
                    tmem_wait_ld();
                    uint32_t pk[32];
#pragma unroll
                    for (int c4 = 0; c4 < 16; ++c4) {
                        const int e = 4 * c4;
                        const float2 s01 = mul2(make_float2(pr[e], pr[e + 1]), make_float2(__uint_as_float(dr[e]), __uint_as_float(dr[e + 1])));
                        const float2 s23 = mul2(make_float2(pr[e + 2], pr[e + 3]), make_float2(__uint_as_float(dr[e + 2]), __uint_as_float(dr[e + 3])));
                        pk[2 * c4] = pack_bf16(s01.x, s01.y);
                        pk[2 * c4 + 1] = pack_bf16(s23.x, s23.y);
                    }
                    if (ragged_keys) {   // uniform per unit: only a segment's last key tile has rows to zero
#pragma unroll
                        for (int i = 0; i < 32; ++i) pk[i] = key_valid ? pk[i] : 0u;
                    }
                    tmem_st16(t_dp, *reinterpret_cast<uint32_t(*)[16]>(&pk[0]));
                    tmem_st16(t_dp + 16, *reinterpret_cast<uint32_t(*)[16]>(&pk[16]));
                    // the same 64 values as 8 x 16 bytes of row r of this warpgroup's [key][64 q] atom (128-byte swizzle)
#pragma unroll
                    for (int chunk = 0; chunk < 8; ++chunk) {
                        *reinterpret_cast<uint4*>(ds_row + ((chunk ^ (r & 7)) << 4)) =
                            make_uint4(pk[4 * chunk], pk[4 * chunk + 1], pk[4 * chunk + 2], pk[4 * chunk + 3]);
                    }
                }
                tmem_wait_st();
                fence_async_smem();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars.ds_full);
            }
            sc += nq;
        }
    } else {
        // ------------------------------------------------------------------ dQ reducer + dK/dV epilogue
        // dQ of a step: TMEM -> registers -> swizzled staging in shared memory -> one TMA reduce-add per 16 fp32
        // columns into the global accumulator (the copy engine does the atomics).
        setmaxnreg_dec<kRegsReducer>();
        const int r = ((warp & 3) << 5) | lane;
        const int rt = tid - 12 * 32;   // 0..127 inside the warpgroup
        const uint32_t lane_base = uint32_t((warp & 3) * 32) << 16;
        uint32_t pc = 0, gc = 0, unit_it = 0;   // step counter, staging-chunk counter
        bool ok = true;
        mpipe_work_item_t it_next = item_at(unit_of(0));   // one unit ahead: the global load is off the unit's critical path
        for (int ur = 0, u = unit_of(0); u < n_units; ++ur, u = unit_of(ur), ++unit_it) {
            const mpipe_work_item_t it = it_next;
            it_next = item_at(unit_of(ur + 1));
            const int head = it.seg;
            const int nq = steps_of(it);
            // No early exit inside this loop: the four warps meet at named barriers, so after a time-out
            // they keep walking the (now empty) iterations together instead of leaving one another behind.
            for (int i = 0; i < nq; ++i, ++pc) {
                if (ok) ok = mbar_wait<kSleepAux>(&bars.dq_full, pc & 1, &abort_flag);
                tc_fence_after();
                const int q0 = it.kv_start + q_tile_of(it, i, nq) * kBQ;
                // One round per 16 columns: read them from TMEM, write this thread's 64-byte row of box gc % 3, and
                // after the warpgroup's barrier hand the box to the copy engine.  Box gc % 3 was last used three rounds
                // ago; before each barrier the issuing thread waits until at most ONE reduction is still reading its
                // box, so the box of the next round is free when the barrier opens -- one barrier per round.
#pragma unroll
                for (int ch = 0; ch < D / 16; ++ch, ++gc) {
                    uint8_t* box = smem + Cfg::kSmemStage + (gc % Cfg::kStageBoxes) * Cfg::kStageBox;
                    if (ok) {
                        uint32_t v[16];
                        tmem_ld16(tmem + lane_base + Cfg::kColDQ + 16 * ch, v);
                        tmem_wait_ld();
                        if (ch == D / 16 - 1) {   // the whole row has left TMEM: the next step's dQ may be issued
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(&bars.dq_empty);
                        }
#pragma unroll
                        for (int c4 = 0; c4 < 4; ++c4)
                            *reinterpret_cast<uint4*>(box + r * 64 + ((c4 ^ ((r >> 1) & 3)) << 4)) =
                                make_uint4(v[4 * c4], v[4 * c4 + 1], v[4 * c4 + 2], v[4 * c4 + 3]);
                    }
                    fence_async_smem();
                    if (rt == 0) bulk_wait_group_read<1>();
                    named_barrier_sync(1, 128);
                    if (rt == 0) {
                        if (ok) tma_reduce_add_3d(&maps.dq_acc, box, 16 * ch, head, q0);
                        bulk_commit_group();   // (an empty group after a time-out keeps the round count in step)
                    }
                }
            }
            if (ok) ok = mbar_wait<kSleepAux>(&bars.dkv_full, unit_it & 1, &abort_flag);
            if (!ok) continue;   // keep walking the units so that the named barriers above stay matched
            tc_fence_after();
            const bool store = r < it.row_len;
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
    constexpr uint32_t box = Cfg::kBoxElems;
    constexpr int swz = Cfg::kRowBytes;
    if (!make_tensor_map_thd(&m.q, q, total_tokens, n_heads, D, ts_qkv, hs_qkv, box, kBQ, swz) ||
        !make_tensor_map_thd(&m.k, k, total_tokens, n_heads, D, ts_qkv, hs_qkv, box, kBT, swz) ||
        !make_tensor_map_thd(&m.v, v, total_tokens, n_heads, D, ts_qkv, hs_qkv, box, kBT, swz) ||
        !make_tensor_map_thd(&m.dout, dout, total_tokens, n_heads, D, ts_o, hs_o, box, kBQ, swz) ||
        !make_tensor_map_thd(&m.dq_acc, dq_acc, total_tokens, n_heads, D, int64_t(n_heads) * D, D, 16, kBQ, 64, 4))
        return MPIPE_ERR_CUDA;
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
