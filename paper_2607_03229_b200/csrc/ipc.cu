// Peer mapping for the Replicated -> Sharded seam across ranks (Table 2: Gather forward, Scatter backward).
// The encoder output of a microbatch lives on its ByMicrobatch owner; the first pipeline stage owns the LLM input
// sequence.  Instead of a send followed by a local scatter, the owner's merge kernel stores its rows straight into the
// first stage's buffer through a peer mapping (plain stores over NVLink; no TMA, no multicast), and the reverse seam
// reads the gradient rows the same way.  These helpers only export / open / close that mapping (CUDA IPC).
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include "common.h"

extern "C" {

int32_t mpipe_ipc_handle_bytes(void) { return int32_t(sizeof(cudaIpcMemHandle_t)); }

int32_t mpipe_ipc_export(const void* dev_ptr, void* handle_out) {
    if (dev_ptr == nullptr || handle_out == nullptr) return MPIPE_ERR_INVALID_ARG;
    cudaIpcMemHandle_t h;
    if (cudaIpcGetMemHandle(&h, const_cast<void*>(dev_ptr)) != cudaSuccess) {
        cudaGetLastError();
        return MPIPE_ERR_CUDA;
    }
    memcpy(handle_out, &h, sizeof(h));
    return MPIPE_OK;
}

int32_t mpipe_ipc_open(const void* handle, void** dev_ptr_out) {
    if (handle == nullptr || dev_ptr_out == nullptr) return MPIPE_ERR_INVALID_ARG;
    cudaIpcMemHandle_t h;
    memcpy(&h, handle, sizeof(h));
    void* p = nullptr;
    if (cudaIpcOpenMemHandle(&p, h, cudaIpcMemLazyEnablePeerAccess) != cudaSuccess) {
        cudaGetLastError();
        return MPIPE_ERR_CUDA;
    }
    *dev_ptr_out = p;
    return MPIPE_OK;
}

int32_t mpipe_ipc_close(void* dev_ptr) {
    if (dev_ptr == nullptr) return MPIPE_ERR_INVALID_ARG;
    if (cudaIpcCloseMemHandle(dev_ptr) != cudaSuccess) {
        cudaGetLastError();
        return MPIPE_ERR_CUDA;
    }
    return MPIPE_OK;
}

}  // extern "C"
