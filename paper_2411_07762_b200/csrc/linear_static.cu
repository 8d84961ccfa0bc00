// aser_linear_w4a8_lr_static: the tensor-core linear for callers that cannot provide a
// workspace.  The scratch the kernel needs (status word, tile counters, partial sums of tiles
// shared between CTAs) lives in a fixed array that is part of the library image.
#include <stdio.h>

#include <atomic>

#include "aser_common.cuh"

namespace aser {
namespace {

constexpr size_t kStaticScratchBytes = 8u << 20;  // 8 MiB: enough for up to 32 tokens per call

// One copy per GPU that loads the library, resident until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// Device address of g_static_scratch per CUDA device ordinal.  In host code the array's name
// only identifies the symbol; the address a kernel can use comes from cudaGetSymbolAddress.
// Threads may race to fill a slot; they store the same value, atomically.  An address stays
// valid for the life of the device's primary context: after cudaDeviceReset it is stale.
std::atomic<void*> g_scratch_addr[kMaxDevices];

int scratch_for_current_device(void** out) {
    int dev = 0;
    const int rc = current_device(&dev);
    if (rc != ASER_OK) return rc;
    void* addr = g_scratch_addr[dev].load(std::memory_order_acquire);
    if (addr == nullptr) {
        int major = 0;
        cudaError_t e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
        if (e != cudaSuccess) return record_cuda_error(e, "cudaDeviceGetAttribute");
        if (major != 10) return record_error(ASER_ERR_DEVICE, "device is not compute capability 10.x");
        void* ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess) return record_cuda_error(e, "cudaGetSymbolAddress(static scratch)");
        g_scratch_addr[dev].store(ptr, std::memory_order_release);
        addr = ptr;
    }
    *out = addr;
    return ASER_OK;
}

}  // namespace
}  // namespace aser

using namespace aser;

extern "C" int aser_linear_w4a8_lr_static(const int8_t* Xq, const float* a_scale, const void* Wk,
                                          const float* w_scale, const void* T_bf16,
                                          const void* LB_f16, int M, int N, int K, int r,
                                          void* Y_f16, int32_t* acc_debug, void* stream) {
    const size_t need = aser_workspace_bytes(M, N, K, r);   // 0 for an unsupported shape
    if (M < 0 || N < 0 || need == 0)
        return record_error(ASER_ERR_SHAPE, "unsupported M, N, K or r");
    if (M == 0 || N == 0) return ASER_OK;
    if (need > kStaticScratchBytes) {
        char msg[200];
        snprintf(msg, sizeof(msg),
                 "this problem needs %zu bytes of scratch but the built-in array holds %zu "
                 "(at most 32 tokens per call); use aser_linear_w4a8_lr with a workspace",
                 need, kStaticScratchBytes);
        return record_error(ASER_ERR_WORKSPACE, msg);
    }
    const void* required[] = {Xq, a_scale, Wk, w_scale, Y_f16};
    for (const void* ptr : required) {
        if (ptr == nullptr) return record_error(ASER_ERR_NULL, "a required pointer is NULL");
        if (misaligned16(ptr)) return record_error(ASER_ERR_ALIGN, "a pointer is not 16-byte aligned");
    }
    if (r > 0) {
        if (T_bf16 == nullptr || LB_f16 == nullptr)
            return record_error(ASER_ERR_NULL, "T_bf16 or LB_f16 is NULL with r > 0");
        if (misaligned16(T_bf16) || misaligned16(LB_f16))
            return record_error(ASER_ERR_ALIGN, "a pointer is not 16-byte aligned");
    }
    if (acc_debug != nullptr && misaligned16(acc_debug))
        return record_error(ASER_ERR_ALIGN, "acc_debug is not 16-byte aligned");

    void* scratch = nullptr;
    int rc = scratch_for_current_device(&scratch);
    if (rc != ASER_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // The array still holds whatever the previous call left: the status word and the tile
    // counters must read zero when the kernel starts (partial sums are written before use).
    cudaError_t e = cudaMemsetAsync(scratch, 0, linear_tc_zeroed_prefix_bytes(M, N, K, r), st);
    if (e != cudaSuccess) return record_cuda_error(e, "cudaMemsetAsync(static scratch)");
    return launch_linear_tc(Xq, a_scale, static_cast<const uint8_t*>(Wk), w_scale,
                            static_cast<const __nv_bfloat16*>(T_bf16),
                            static_cast<const __half*>(LB_f16), M, N, K, r,
                            static_cast<__half*>(Y_f16), acc_debug, scratch, kStaticScratchBytes, st);
}
