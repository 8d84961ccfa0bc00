// CUDA-core (dp4a) version of the ASER linear: integer product of int8 activations with
// canonical packed int4 weights, dequantisation, and the up projection L_B T (Sec. 4.2,
// "W_q X + L_A L_B X").  Slow and simple on purpose: it is the on-device cross-check of the
// tensor-core kernel and never the timed path.
#include "aser_common.cuh"

namespace aser {

namespace {

constexpr int kTok = 8;    // tokens per warp
constexpr int kWarps = 8;  // output channels per CTA (one warp each)

// Sign-extend the eight nibbles of a canonical word (column c+t in nibble t) into two
// int8x4 words: lo = columns c..c+3, hi = columns c+4..c+7.
__device__ __forceinline__ void nibbles_to_int8(uint32_t w, uint32_t& lo, uint32_t& hi) {
    uint32_t b[8];
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        int v = (int)((w >> (4 * t)) & 0xF);
        v = (v ^ 8) - 8;
        b[t] = (uint32_t)(v & 0xFF);
    }
    lo = b[0] | (b[1] << 8) | (b[2] << 16) | (b[3] << 24);
    hi = b[4] | (b[5] << 8) | (b[6] << 16) | (b[7] << 24);
}

// grid = (ceil(N / kWarps), ceil(M / kTok)); warp w of a CTA owns channel n = bx*kWarps + w and
// kTok tokens; lanes stride over K in steps of 8 columns.
__global__ void __launch_bounds__(kWarps * 32)
linear_simt_kernel(const int8_t* __restrict__ Xq, const float* __restrict__ a_scale,
                   const uint8_t* __restrict__ Wq, const float* __restrict__ w_scale,
                   const __nv_bfloat16* __restrict__ T, const __half* __restrict__ LB,
                   int M, int N, int K, int r, __half* __restrict__ Y,
                   int32_t* __restrict__ acc_debug) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n = blockIdx.x * kWarps + warp;
    const int m0 = blockIdx.y * kTok;
    if (n >= N) return;
    int acc[kTok];
#pragma unroll
    for (int i = 0; i < kTok; ++i) acc[i] = 0;
    const uint8_t* wrow = Wq + (size_t)n * (K / 2);
    for (int c = lane * 8; c < K; c += 32 * 8) {
        uint32_t w = *reinterpret_cast<const uint32_t*>(wrow + c / 2);
        uint32_t lo, hi;
        nibbles_to_int8(w, lo, hi);
#pragma unroll
        for (int i = 0; i < kTok; ++i) {
            if (m0 + i < M) {
                uint2 x = *reinterpret_cast<const uint2*>(Xq + (size_t)(m0 + i) * K + c);
                acc[i] = __dp4a((int)x.x, (int)lo, acc[i]);
                acc[i] = __dp4a((int)x.y, (int)hi, acc[i]);
            }
        }
    }
#pragma unroll
    for (int i = 0; i < kTok; ++i) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], o);
    }
    const float ws = w_scale[n];
#pragma unroll
    for (int i = 0; i < kTok; ++i) {
        const int m = m0 + i;
        if (m < M) {
            float lr = 0.f;
            for (int j = lane; j < r; j += 32)
                lr = fmaf(__half2float(LB[(size_t)n * r + j]), __bfloat162float(T[(size_t)m * r + j]), lr);
            lr = warp_sum(lr);
            if (lane == 0) {
                float y = (float)acc[i] * a_scale[m] * ws + lr;
                Y[(size_t)m * N + n] = __float2half_rn(y);
                if (acc_debug) acc_debug[(size_t)m * N + n] = acc[i];
            }
        }
    }
}

}  // namespace

int launch_linear_simt(const int8_t* Xq, const float* a_scale, const uint8_t* Wq,
                       const float* w_scale, const __nv_bfloat16* T, const __half* LB,
                       int M, int N, int K, int r, __half* Y, int32_t* acc_debug, cudaStream_t st) {
    if (M == 0 || N == 0) return ASER_OK;
    dim3 grid((N + kWarps - 1) / kWarps, (M + kTok - 1) / kTok);
    if (grid.y > 65535) return ASER_ERR_SHAPE;
    linear_simt_kernel<<<grid, kWarps * 32, 0, st>>>(Xq, a_scale, Wq, w_scale, T, LB, M, N, K, r, Y,
                                                     acc_debug);
    return check_launch("linear_simt_kernel");
}

}  // namespace aser
