// Shared host-side helpers of libmpipe_enc (argument checks, status reporting).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include "../../include/mpipe_enc.h"

namespace mpipe {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline int cdiv(int a, int b) { return (a + b - 1) / b; }

// Number of SMs of the current device (cached per device id).
int sm_count();

// A kernel that uses more than 48 KB of dynamic shared memory must opt in once per device; doing it on every
// launch costs host time that shows on small microbatches.  The kernel is a template VALUE argument, so every
// kernel (every instantiation of a kernel template) has its own function-local table of the devices set up.
template <auto kernel>
inline bool ensure_dynamic_smem(int bytes) {
    static bool done[64] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) return false;
    if (dev < 64 && done[dev]) return true;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return false;
    if (dev < 64) done[dev] = true;
    return true;
}

// Defined in gemm.cu, used by the layer forward: one projection that stores both GELU(u) and u.
int32_t linear_fwd_gelu_keep_preact(const void* a, const void* w, const void* bias, void* act, void* pre, int32_t M, int32_t N,
                                    int32_t K, int64_t lda, int64_t ldw, int64_t ldact, int64_t ldpre, int32_t* status_buf,
                                    void* stream);

// Optional measurement aid (mpipe_set_profile_events): events recorded around one kernel launch.  The slots
// are thread-local: they affect only launches made by the thread that set them, so concurrent callers of the
// library share no mutable state.
struct ProfileEvents {
    cudaEvent_t start = nullptr, stop = nullptr;
};
enum { kProfileFwd = 0, kProfileBwdMain = 1, kProfileMerge = 2, kProfileLinear = 3, kProfileLayerNorm = 4, kProfileSlots = 5 };
extern thread_local ProfileEvents g_profile[kProfileSlots];
inline void profile_start(int which, cudaStream_t st) {
    if (g_profile[which].start != nullptr) cudaEventRecord(g_profile[which].start, st);
}
inline void profile_stop(int which, cudaStream_t st) {
    if (g_profile[which].stop != nullptr) cudaEventRecord(g_profile[which].stop, st);
}

// Device-side: record the first finding in the caller's status buffer.
__device__ __forceinline__ void report_status(int32_t* status_buf, int32_t code, int32_t detail) {
    if (status_buf != nullptr && atomicCAS(status_buf, 0, code) == 0) status_buf[1] = detail;
}

// Work items are read from device memory that the host cannot inspect when it launches, so every CTA checks
// the whole list before it does anything else: an item is acceptable if its row range and its key range are
// non-empty, lie inside [0, T) and the row range is at most one tile.  One bad item rejects the plan as a whole --
// the kernel reports MPIPE_ERR_INDEX with the item's index and returns without reading or writing a tensor --
// which keeps every check out of the pipeline's loops.  A plan made by mpipe_seg_plan for the same total_tokens
// always passes.
__device__ __forceinline__ bool plan_item_ok(const mpipe_work_item_t& it, int32_t tile_rows, int32_t T) {
    return it.row_start >= 0 && it.row_len >= 1 && it.row_len <= tile_rows && it.row_start <= T - it.row_len &&
           it.kv_start >= 0 && it.kv_len >= 1 && it.kv_start <= T - it.kv_len;
}
// Returns true if every item passes.  All threads of the CTA must call it; `flag` is a shared-memory word.
static __device__ __noinline__ bool plan_ok_cta(const mpipe_work_item_t* items, int32_t n_items, int32_t tile_rows, int32_t T,
                                            int32_t* status_buf, int* flag) {
    if (threadIdx.x == 0) *flag = -1;
    __syncthreads();
    for (int i = threadIdx.x; i < n_items; i += blockDim.x)
        if (!plan_item_ok(items[i], tile_rows, T)) atomicMax(flag, i);
    __syncthreads();
    const int bad = *flag;
    if (bad >= 0 && blockIdx.x == 0 && threadIdx.x == 0) report_status(status_buf, MPIPE_ERR_INDEX, bad);
    return bad < 0;
}

}  // namespace mpipe
