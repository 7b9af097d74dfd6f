// qlora_bwd_lora_static: the LoRA-gradient call for callers that cannot hand the library a scratch buffer.
//
// Some hosts of this library may not allocate device memory when they call it: a training framework that has already
// given the whole device to its own memory pool (a fresh cudaMalloc then fails), or a step loop whose rules forbid
// allocation calls because cudaMalloc / cudaFree synchronise the device.  For them the scratch that qlora_bwd_lora
// takes from its `workspace` argument lives here instead, in one file-scope device array that is part of the loaded
// library: every GPU that loads the library holds QLORA_STATIC_SCRATCH_BYTES of it until the process exits.
//
// The array's name is only a host-side handle in host code, not a device address; handing it to a kernel would fault
// (or, where the GPU can reach host memory, quietly use the wrong memory).  Its device address is looked up once per
// device with cudaGetSymbolAddress, with that device current, and that pointer is what the kernels receive.
#include <cuda_runtime.h>

#include <mutex>

#include "launch.h"
#include "qlora.h"

namespace {

static __device__ __align__(256) unsigned char g_static_scratch[QLORA_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void* g_scratch_ptr[kMaxDevices] = {};   // device address of g_static_scratch on each device, filled on first use

// Device address of the scratch array on the current device (set-up on the first call per device).
int static_scratch_for_current_device(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return QLORA_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (g_scratch_ptr[dev] == nullptr) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) return QLORA_ERR_CUDA;
        g_scratch_ptr[dev] = ptr;
    }
    *out = g_scratch_ptr[dev];
    return QLORA_OK;
}

}  // namespace

extern "C" int qlora_bwd_lora_static(const qlora_desc* desc, int M, const void* X, const void* dY, const void* A,
                                     const void* B, const float* H, const float* G, float* dA, float* dB,
                                     int accumulate, void* cuda_stream) {
    size_t need = 0;
    const int rc = qlora_workspace_bytes(desc, M, &need);   // also validates the descriptor and M
    if (rc != QLORA_OK) return rc;
    need = qlora::required_workspace_bytes(*desc, M);         // (the part of it that qlora_bwd_lora can use)
    if (need > (size_t)QLORA_STATIC_SCRATCH_BYTES) return QLORA_ERR_STATIC_LIMIT;
    void* scratch = nullptr;
    const int rs = static_scratch_for_current_device(&scratch);
    if (rs != QLORA_OK) return rs;
    // Same kernels, same order as qlora_bwd_lora; only the scratch differs.  Every scratch element that a kernel of the
    // call reads has been written earlier in the same call (H / G are recomputed in full, every partial-sum slice is
    // stored before the reduction reads it), so nothing left behind by the previous call needs clearing.
    return qlora_bwd_lora(desc, M, X, dY, A, B, H, G, dA, dB, accumulate, scratch, (size_t)QLORA_STATIC_SCRATCH_BYTES,
                          cuda_stream);
}
