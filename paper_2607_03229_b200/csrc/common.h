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

// Optional measurement aid (mpipe_set_profile_events): events recorded around one kernel launch.
struct ProfileEvents {
    cudaEvent_t start = nullptr, stop = nullptr;
};
enum { kProfileFwd = 0, kProfileBwdMain = 1, kProfileMerge = 2, kProfileLinear = 3, kProfileLayerNorm = 4, kProfileSlots = 5 };
extern ProfileEvents g_profile[kProfileSlots];
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

}  // namespace mpipe
