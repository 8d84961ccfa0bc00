// Shared host/device helpers of the ASER linear library (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "aser.h"

namespace aser {

// ---- host side -------------------------------------------------------------
// Records the text of a CUDA error for aser_last_error() and returns ASER_ERR_LAUNCH.
int record_cuda_error(cudaError_t e, const char* where);
// Records a plain message for aser_last_error() and returns `code`.
int record_error(int code, const char* msg);
// cudaGetLastError() after a launch -> ASER_OK or ASER_ERR_LAUNCH.
int check_launch(const char* where);

// Per-device caches (shared-memory opt-ins, SM counts, occupancy answers) are arrays indexed by
// the CUDA device ordinal: a process may drive several GPUs, and function attributes belong to
// a device's context.  current_device returns ASER_OK and the ordinal, or an error code.
constexpr int kMaxDevices = 64;
int current_device(int* dev);
// Number of SMs of the current device.
int device_sm_count(int* num_sms);

inline bool misaligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

// Kernel launchers (one per .cu file); arguments are already validated.
int launch_pack_w4(const __half* W, const float* s, int N, int K, uint8_t* Wq, float* w_scale,
                   cudaStream_t st);
int launch_repack_w4(const uint8_t* Wq, int N, int K, uint8_t* Wk, bool inverse, cudaStream_t st);
// act_bits: width of the symmetric activation codes (2..8); they are stored in int8 either way.
// t_pair: T is written as [M, 2r], a bf16 value and the bf16 remainder of each entry.
int launch_quant_act(const __half* X, const float* s, const __half* LA, int M, int K, int r,
                     int8_t* Xq, float* a_scale, __nv_bfloat16* T, cudaStream_t st, int act_bits = 8,
                     bool t_pair = false);
// The same with caller-provided scratch (quant_act_ws_scratch_bytes): the two-kernel path for more
// than 32 tokens, ranks up to 512 (stacked down projections of layers that share X).
size_t quant_act_ws_scratch_bytes(int M, int K, int r);
int quant_act_ws_launches(int M, int K);     // kernels one call enqueues
int launch_quant_act_ws(const __half* X, const float* s, const __half* LA, int M, int K, int r,
                        int8_t* Xq, float* a_scale, __nv_bfloat16* T, void* scratch, size_t scratch_bytes,
                        cudaStream_t st, int act_bits = 8, bool t_pair = false);
// Device-side construction of a layer's factors (construct.cu); synchronises the stream.
size_t construct_workspace_bytes(int N, int K, int Tcal, int r, int n_split);
int launch_construct(const __half* W, const float* s, const __half* Xcal, int N, int K, int Tcal, int r,
                     double damping, int iters, uint8_t* Wq, float* w_scale, __half* LA, __half* LB,
                     double* sigma_out, double* S_out, const int* split_idx, int n_split, void* workspace,
                     cudaStream_t st);
int launch_linear_simt(const int8_t* Xq, const float* a_scale, const uint8_t* Wq,
                       const float* w_scale, const __nv_bfloat16* T, const __half* LB,
                       int M, int N, int K, int r, __half* Y, int32_t* acc_debug, cudaStream_t st);
// Several layers stacked along N that read the same activations, served by one launch: rows
// [0, b1) are layer 0, [b1, b2) layer 1, ... (bounds are multiples of 128; at most four layers, all
// of rank r); layer l takes the columns [l r, (l + 1) r) of T.  The default is a single layer.
struct CatSplit {
    int layers = 1;
    int b1 = 0x7fffffff, b2 = 0x7fffffff, b3 = 0x7fffffff;
};
__host__ __device__ inline int cat_layer(const CatSplit& c, int row) {
    return (row >= c.b1 ? 1 : 0) + (row >= c.b2 ? 1 : 0) + (row >= c.b3 ? 1 : 0);
}
// `ldt`: elements between rows of T (0 = r; larger when T is a column range of a wider matrix).
// `overlap_prev`: the kernel launched before this one on `st` is this library's quant_act for
// the same step.  The linear kernel may then start while that one still runs: it streams the
// weights (which that kernel does not write) and waits for its completion before it touches
// Xq, a_scale or T.  Must be false when anything else precedes the launch.
int launch_linear_tc(const int8_t* Xq, const float* a_scale, const uint8_t* Wk,
                     const float* w_scale, const __nv_bfloat16* T, const __half* LB,
                     int M, int N, int K, int r, __half* Y, int32_t* acc_debug,
                     void* workspace, size_t workspace_bytes, cudaStream_t st,
                     bool overlap_prev = false, int ldt = 0, CatSplit cat = CatSplit());
// Few-token kernel (M <= kLinearDecodeMaxTokens): streams the weights once, no workspace.
// linear_decode_prefers: the shapes for which it is faster than the tensor-core kernel.
constexpr int kLinearDecodeMaxTokens = 16;
bool linear_decode_prefers(int M, int N, int K);
int launch_linear_decode(const int8_t* Xq, const float* a_scale, const uint8_t* Wk,
                         const float* w_scale, const __nv_bfloat16* T, const __half* LB,
                         int M, int N, int K, int r, __half* Y, int32_t* acc_debug,
                         cudaStream_t st, bool overlap_prev = false, int ldt = 0, CatSplit cat = CatSplit());
size_t linear_tc_workspace_bytes(int M, int N, int K, int r);
// The range checks launch_linear_tc makes before it launches (workspace size, index widths), for
// callers that must reject a call before they enqueue anything else.  Records the error text.
int linear_tc_check(int M, int N, int K, int r, size_t workspace_bytes);
// Leading bytes of the workspace (status word + tile counters) that must be zero at launch.
size_t linear_tc_zeroed_prefix_bytes(int M, int N, int K, int r);

// Layout of the repacked weight: [N/128 row blocks][K/128 column blocks][8 KiB].
// Inside a block: 4 sub-blocks of 32 columns; each holds 128 rows x 16 bytes.
// The 16 bytes of a row are four 32-bit words; word w covers columns c0 = 32*sub + 8*w .. +7
// with column c0+i   in nibble 2*i   (i = 0..3)  -> bytes of (word << 4) & 0xF0F0F0F0
// and  column c0+4+i in nibble 2*i+1 (i = 0..3)  -> bytes of  word       & 0xF0F0F0F0,
// so two ALU operations turn a word into eight int8 values equal to 16*q, already in
// column order.
constexpr int kWkRows = 128;
constexpr int kWkCols = 128;
constexpr int kWkBlockBytes = kWkRows * kWkCols / 2;  // 8192

// Workspace header (first 256 bytes): word 0 = status, rest reserved.  The tile counters of the
// tensor-core kernel follow; header and counters (kWsZeroedBytes in all) must read zero when a
// kernel starts, everything behind them is written before it is read.
constexpr size_t kWsHeaderBytes = 256;
constexpr size_t kWsZeroedBytes = 1024;

#ifdef __CUDACC__
// ---- device side -----------------------------------------------------------
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
// Round-half-to-even to an integer-valued float, then clamp; returns the int.
__device__ __forceinline__ int rne_clamp(float v, float lo, float hi) {
    float c = rintf(v);
    c = fminf(fmaxf(c, lo), hi);
    return (int)c;
}
#endif

}  // namespace aser
