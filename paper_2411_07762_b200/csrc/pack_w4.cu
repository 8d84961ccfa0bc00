// Offline weight path: smoothing multiply, per-output-channel int4 round-to-nearest,
// nibble packing (Sec. 4.2 Eq. 10/12 Q(W_s); Sec. 5.1 per-channel RTN), plus the
// permutation between the canonical packed form and the tensor-core kernel's layout.
#include "aser_common.cuh"

namespace aser {

namespace {

constexpr int kPackThreads = 256;

__device__ __forceinline__ void load_s8(const float* s, int c, float (&sv)[8]) {
    float4 s0 = *reinterpret_cast<const float4*>(s + c * 8);
    float4 s1 = *reinterpret_cast<const float4*>(s + c * 8 + 4);
    sv[0] = s0.x; sv[1] = s0.y; sv[2] = s0.z; sv[3] = s0.w;
    sv[4] = s1.x; sv[5] = s1.y; sv[6] = s1.z; sv[7] = s1.w;
}

// One CTA per output channel (row).  Pass 1: row absmax of fp32(W)*s.  Pass 2: re-read the
// row (it is in L1/L2), divide, round half-to-even, clamp, pack two codes per byte.
__global__ void __launch_bounds__(kPackThreads)
pack_w4_kernel(const __half* __restrict__ W, const float* __restrict__ s, int N, int K,
               uint8_t* __restrict__ Wq, float* __restrict__ w_scale) {
    const int n = blockIdx.x;
    const __half* row = W + (size_t)n * K;
    const int chunks = K / 8;  // 8 halves = 16 bytes
    __shared__ float red[kPackThreads / 32];

    float amax = 0.f;
    for (int c = threadIdx.x; c < chunks; c += kPackThreads) {
        uint4 raw = *reinterpret_cast<const uint4*>(row + c * 8);
        const __half* h = reinterpret_cast<const __half*>(&raw);
        float sv[8];
        if (s) load_s8(s, c, sv);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            float w = __half2float(h[i]);
            float v = s ? __fmul_rn(w, sv[i]) : w;
            amax = fmaxf(amax, fabsf(v));
        }
    }
    amax = warp_max(amax);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = amax;
    __syncthreads();
    amax = red[0];
#pragma unroll
    for (int i = 1; i < kPackThreads / 32; ++i) amax = fmaxf(amax, red[i]);

    const float sc = __fdiv_rn(amax, 7.0f);
    if (threadIdx.x == 0) w_scale[n] = sc;

    uint8_t* out = Wq + (size_t)n * (K / 2);
    for (int c = threadIdx.x; c < chunks; c += kPackThreads) {
        uint4 raw = *reinterpret_cast<const uint4*>(row + c * 8);
        const __half* h = reinterpret_cast<const __half*>(&raw);
        float sv[8];
        if (s) load_s8(s, c, sv);
        uint32_t word = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            float w = __half2float(h[i]);
            float v = s ? __fmul_rn(w, sv[i]) : w;
            int q = 0;
            if (amax > 0.f) q = rne_clamp(__fdiv_rn(v, sc), -8.f, 7.f);
            word |= (uint32_t)(q & 0xF) << (4 * i);  // column 2j -> low nibble of byte j
        }
        *reinterpret_cast<uint32_t*>(out + c * 4) = word;
    }
}

// Canonical [N, K/2] <-> blocked layout (see aser_common.cuh).  One thread per 32-bit word
// of the blocked layout (8 codes).  Rows >= N of the last block are zero codes.
__global__ void repack_w4_kernel(uint8_t* __restrict__ Wq, int N, int K,
                                 uint8_t* __restrict__ Wk, bool inverse, size_t n_words) {
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= n_words) return;
    const int kblocks = K / kWkCols;
    size_t blk = idx / (kWkBlockBytes / 4);
    int in_blk = (int)(idx % (kWkBlockBytes / 4));
    int nb = (int)(blk / kblocks), kb = (int)(blk % kblocks);
    int sub = in_blk / (kWkRows * 4);  // 32-column sub-block
    int row = (in_blk / 4) % kWkRows;
    int w = in_blk % 4;
    int n = nb * kWkRows + row;
    int c0 = kb * kWkCols + sub * 32 + w * 8;  // first of the 8 columns of this word
    uint32_t* blocked = reinterpret_cast<uint32_t*>(Wk) + idx;
    uint32_t* canon = reinterpret_cast<uint32_t*>(Wq + (size_t)(n < N ? n : 0) * (K / 2) + c0 / 2);
    if (!inverse) {
        uint32_t out = 0;
        if (n < N) {
            uint32_t can = *canon;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                uint32_t a = (can >> (4 * i)) & 0xF;        // column c0 + i
                uint32_t b = (can >> (4 * (i + 4))) & 0xF;  // column c0 + 4 + i
                out |= a << (8 * i);
                out |= b << (8 * i + 4);
            }
        }
        *blocked = out;
    } else {
        if (n >= N) return;
        uint32_t blkw = *blocked;
        uint32_t can = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            uint32_t a = (blkw >> (8 * i)) & 0xF;
            uint32_t b = (blkw >> (8 * i + 4)) & 0xF;
            can |= a << (4 * i);
            can |= b << (4 * (i + 4));
        }
        *canon = can;
    }
}

}  // namespace

int launch_pack_w4(const __half* W, const float* s, int N, int K, uint8_t* Wq, float* w_scale,
                   cudaStream_t st) {
    if (N == 0) return ASER_OK;
    pack_w4_kernel<<<N, kPackThreads, 0, st>>>(W, s, N, K, Wq, w_scale);
    return check_launch("pack_w4_kernel");
}

// `inverse` false: reads Wq, writes Wk.  true: reads Wk, writes Wq.
int launch_repack_w4(const uint8_t* Wq, int N, int K, uint8_t* Wk, bool inverse, cudaStream_t st) {
    if (N == 0) return ASER_OK;
    size_t n_words = aser_repacked_bytes(N, K) / 4;
    int threads = 256;
    size_t blocks = (n_words + threads - 1) / threads;
    repack_w4_kernel<<<(unsigned)blocks, threads, 0, st>>>(const_cast<uint8_t*>(Wq), N, K, Wk, inverse,
                                                           n_words);
    return check_launch("repack_w4_kernel");
}

}  // namespace aser
