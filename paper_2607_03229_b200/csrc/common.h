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

// Work items are read from device memory that the host cannot inspect when it launches.  Every range of an
// item is therefore clamped to the tensors (token rows [0, T), at most tile_rows rows per item), so that no
// load, store or reduction derived from it can leave them.  An item that is empty after clamping is replaced
// by a one-token stand-in whose results are not stored (seg = -1): the pipeline then runs a regular unit and
// every role keeps the same trip counts.  Returns true if the item had to be altered; the caller reports
// MPIPE_ERR_INDEX.  A plan made by mpipe_seg_plan for the same total_tokens is never altered.
__device__ __forceinline__ bool sanitize_item(mpipe_work_item_t& it, int32_t tile_rows, int32_t T) {
    const mpipe_work_item_t in = it;
    // intersection of [start, start + len) with [0, T), in 64-bit so that no sum wraps
    const int64_t r0 = max(int64_t(in.row_start), int64_t(0)), r1 = min(int64_t(in.row_start) + in.row_len, int64_t(T));
    const int64_t k0 = max(int64_t(in.kv_start), int64_t(0)), k1 = min(int64_t(in.kv_start) + in.kv_len, int64_t(T));
    it.row_start = int32_t(min(r0, int64_t(T)));
    it.row_len = int32_t(min(max(r1 - r0, int64_t(0)), int64_t(tile_rows)));
    it.kv_start = int32_t(min(k0, int64_t(T)));
    it.kv_len = int32_t(max(k1 - k0, int64_t(0)));
    bool altered = in.seg < 0 || it.row_start != in.row_start || it.row_len != in.row_len ||
                   it.kv_start != in.kv_start || it.kv_len != in.kv_len;
    if (it.row_len == 0 || it.kv_len == 0 || in.seg < 0) {
        it.seg = -1;
        it.row_start = it.kv_start = 0;
        it.row_len = it.kv_len = 1;
        altered = true;
    }
    return altered;
}

}  // namespace mpipe
