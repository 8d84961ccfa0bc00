// Few-token kernel of the ASER linear (Sec. 4.2, "W_q X + L_A L_B X") for M <= 16 tokens:
//   acc = Xq Wq^T (int8 x int4 -> int32),  Y = fp16(acc * a_scale[m] * w_scale[n] + T L_B^T).
//
// With so few tokens the layer is a stream of packed weights through HBM (4 M operations per
// byte) and what matters is how many bytes are in flight and how short the dependent chain of a
// CTA is, not the tensor-core rate.  So this kernel has no shared-memory pipeline, no
// barriers and no cross-CTA reduction:
//   * a CTA owns 16 or 32 output channels for the WHOLE of K, its eight warps take every eighth
//     128-column block; the only exchange is one shared-memory sum over the eight warps;
//   * every thread keeps 128 bytes of packed weights in flight as 16-byte loads into registers
//     (issued before anything else, refilled as they are consumed); the loads of a warp cover
//     whole 128-byte lines of the blocked weight layout (eight rows x 16 bytes per 32-column
//     sub-block).  A per-thread cp.async ring in shared memory (twice the bytes in flight) was
//     measured 20-50 % slower: the shared memory it takes is L1 capacity that the activation
//     fragments then miss;
//   * the packed word is turned into two int8x4 registers (16 * q) by two logic operations and
//     fed to mma.sync m16n8k32 (weights on the 16-row side, tokens on the 8-column side).  An
//     integer dot product does not care about the order of k, so a thread's k positions are
//     simply the 32 columns it loaded; the activation fragment reads the same 32 columns of
//     its token's row of Xq (32 contiguous bytes, served by L1/L2: Xq is at most 16 x K bytes);
//   * the low-rank term is a (16 or 32) x M x r product per CTA: warp w takes the 16-wide slices
//     w and w + 8 of r on mma.sync m16n8k16 (L_B rows from global memory, T converted bf16 ->
//     fp16 in registers); its few loads are issued right behind the first weight loads and it is
//     finished before the first weights arrive;
//   * very large weight matrices (above 64 MB packed) are better served by the bulk-copy pipeline
//     of the tensor-core kernel, which keeps more bytes in flight per SM; the dispatch is in
//     linear_decode_prefers().
//   * the weight loads precede griddepcontrol.wait, so under a programmatic dependent launch
//     they overlap the activation kernel; Xq, a_scale and T are read after it.
#include "aser_common.cuh"

namespace aser {

namespace {

constexpr int kDecWarps = 8;
constexpr int kDecThreads = kDecWarps * 32;
constexpr int kDecRows = 16;      // output channels per CTA
constexpr int kDecBatch = 4;      // column blocks per thread whose weight loads are in flight

__device__ __forceinline__ uint4 ld_stream16(const uint8_t* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
__device__ __forceinline__ void dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// c += A(16 x 16, fp16, row) * B(16 x 8, fp16, col), fp32 accumulation
__device__ __forceinline__ void mma_f16_16x8x16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                                uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// two bf16 in a word -> two fp16 in a word (exact inside the fp16 normal range)
__device__ __forceinline__ uint32_t bf16x2_to_f16x2(uint32_t v) {
    const __half2 h = __floats2half2_rn(__uint_as_float(v << 16), __uint_as_float(v & 0xFFFF0000u));
    return *reinterpret_cast<const uint32_t*>(&h);
}

// c += A(16 x 32, int8, row) * B(32 x 8, int8, col)
__device__ __forceinline__ void mma_s8_16x8x32(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                               uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// NT = number of 8-token groups (1 for M <= 8, 2 for M <= 16).  R = 16-row tiles per warp: a
// CTA owns 16 R output channels; the activation fragment of a column block is loaded once and
// used for all R tiles, which is what keeps the L1 traffic (two bytes of activations per byte of
// packed weights at R = 1, sixteen tokens) below the weight stream's.  B column blocks per warp
// are in flight: B * R * 32 bytes of packed weights per thread (128 bytes at three CTAs per SM,
// 256 bytes at two).
template <int NT, int R, int B>
struct DecCfg {
    static constexpr int Batch = B;
    static constexpr int Rows = 16 * R;
    static constexpr int Regs = R * NT * 4;          // accumulator registers per thread
    static constexpr int MinCtas = (R * B <= 4) ? 3 : 2;
};

template <int NT, int R, int B>
__global__ void __launch_bounds__(kDecThreads, DecCfg<NT, R, B>::MinCtas)
linear_decode_kernel(const int8_t* Xq, const float* a_scale, const uint8_t* __restrict__ Wk,
                     const float* __restrict__ w_scale, const __nv_bfloat16* T,
                     const __half* __restrict__ LB, int M, int N, int K, int r, int ldt,
                     __half* __restrict__ Y, int32_t* __restrict__ acc_debug, const CatSplit cat) {
    using C = DecCfg<NT, R, B>;
    constexpr int BATCH = C::Batch;
    // partial sums of the eight warps: integer accumulators and fp32 accumulators of the low-rank term
    __shared__ int red[kDecWarps][C::Regs][32];
    __shared__ float red_lr[kDecWarps][C::Regs][32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;       // fragment row group / k quarter
    const int KB = K / kWkCols;
    const int n0 = blockIdx.x * C::Rows;
    T += cat_layer(cat, n0) * r;        // a CTA's rows lie inside one layer (16 R divides 128)
    // Rows n0 + 16 rt + g and + 8 of sub-block t (columns 32 t .. 32 t + 31 of a block).  The
    // blocked layout pads the last 128-row tile with zero codes, so rows past N inside that tile
    // read as zeros; a CTA never reaches past the tile (16 R divides 128).
    const uint8_t* wbase = Wk + ((size_t)(n0 >> 7) * KB) * kWkBlockBytes + t * (kWkRows * 16) +
                           ((n0 & 127) + g) * 16;

    uint4 wa[BATCH][R][2];
#pragma unroll
    for (int i = 0; i < BATCH; ++i) {
        const int kbi = warp + i * kDecWarps;
        if (kbi < KB) {
#pragma unroll
            for (int rt = 0; rt < R; ++rt) {
                wa[i][rt][0] = ld_stream16(wbase + (size_t)kbi * kWkBlockBytes + rt * 256);
                wa[i][rt][1] = ld_stream16(wbase + (size_t)kbi * kWkBlockBytes + rt * 256 + 128);
            }
        }
    }
    // L_B fragments of the low-rank term (constant data: may precede the dependency wait)
    uint2 la[2][R][2];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
        const int k0 = (warp + u * kDecWarps) * 16 + 4 * t;
#pragma unroll
        for (int rt = 0; rt < R; ++rt) {
            const int row0 = n0 + rt * 16 + g;
            la[u][rt][0] = la[u][rt][1] = make_uint2(0, 0);
            if (k0 < r) {
                if (row0 < N) la[u][rt][0] = __ldg(reinterpret_cast<const uint2*>(LB + (size_t)row0 * r + k0));
                if (row0 + 8 < N) la[u][rt][1] = __ldg(reinterpret_cast<const uint2*>(LB + (size_t)(row0 + 8) * r + k0));
            }
        }
    }
    dep_wait();

    // ---- low-rank term, while the weight loads are in flight: warp w takes the 16-wide slices
    // w and w + 8 of r; a thread's k positions inside a slice are 4 t .. 4 t + 3 ----
    const int lr_warps = (r / 16 < kDecWarps) ? r / 16 : kDecWarps;
    if (warp < lr_warps) {
        uint2 tv[2][NT];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int k0 = (warp + u * kDecWarps) * 16 + 4 * t;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                tv[u][nt] = make_uint2(0, 0);
                if (k0 < r && g + 8 * nt < M)
                    tv[u][nt] = *reinterpret_cast<const uint2*>(T + (size_t)(g + 8 * nt) * ldt + k0);
            }
        }
#pragma unroll
        for (int rt = 0; rt < R; ++rt) {
            float cf[NT][4];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int e = 0; e < 4; ++e) cf[nt][e] = 0.f;
#pragma unroll
            for (int u = 0; u < 2; ++u)
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
                    mma_f16_16x8x16(cf[nt], la[u][rt][0].x, la[u][rt][1].x, la[u][rt][0].y, la[u][rt][1].y,
                                    bf16x2_to_f16x2(tv[u][nt].x), bf16x2_to_f16x2(tv[u][nt].y));
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int e = 0; e < 4; ++e) red_lr[warp][(rt * NT + nt) * 4 + e][lane] = cf[nt][e];
        }
    }

    // ---- integer product ----
    int c[R][NT][4];
#pragma unroll
    for (int rt = 0; rt < R; ++rt)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) c[rt][nt][e] = 0;
    // activation fragment: 32 bytes of token g (+ 8 nt) at the columns this thread loaded
    const int8_t* xrow[NT];
    bool x_ok[NT];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        x_ok[nt] = g + 8 * nt < M;
        xrow[nt] = Xq + (size_t)(x_ok[nt] ? g + 8 * nt : 0) * K + t * 32;
    }
    for (int kb0 = warp; kb0 < KB; kb0 += kDecWarps * BATCH) {
#pragma unroll
        for (int i = 0; i < BATCH; ++i) {
            const int kbi = kb0 + i * kDecWarps;
            if (kbi < KB) {
                uint32_t b[NT][8];
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    uint4 lo = make_uint4(0, 0, 0, 0), hi = make_uint4(0, 0, 0, 0);
                    if (x_ok[nt]) {
                        const uint4* xp = reinterpret_cast<const uint4*>(xrow[nt] + kbi * kWkCols);
                        lo = xp[0];
                        hi = xp[1];
                    }
                    b[nt][0] = lo.x; b[nt][1] = lo.y; b[nt][2] = lo.z; b[nt][3] = lo.w;
                    b[nt][4] = hi.x; b[nt][5] = hi.y; b[nt][6] = hi.z; b[nt][7] = hi.w;
                }
                const int kbn = kbi + kDecWarps * BATCH;
#pragma unroll
                for (int rt = 0; rt < R; ++rt) {
                    const uint32_t w0[4] = {wa[i][rt][0].x, wa[i][rt][0].y, wa[i][rt][0].z, wa[i][rt][0].w};
                    const uint32_t w1[4] = {wa[i][rt][1].x, wa[i][rt][1].y, wa[i][rt][1].z, wa[i][rt][1].w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        // word j: columns 8 j .. 8 j + 3 in the low nibbles, 8 j + 4 .. 8 j + 7 in the high
                        const uint32_t a0 = (w0[j] << 4) & 0xF0F0F0F0u, a2 = w0[j] & 0xF0F0F0F0u;
                        const uint32_t a1 = (w1[j] << 4) & 0xF0F0F0F0u, a3 = w1[j] & 0xF0F0F0F0u;
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt)
                            mma_s8_16x8x32(c[rt][nt], a0, a1, a2, a3, b[nt][2 * j], b[nt][2 * j + 1]);
                    }
                    if (kbn < KB) {
                        wa[i][rt][0] = ld_stream16(wbase + (size_t)kbn * kWkBlockBytes + rt * 256);
                        wa[i][rt][1] = ld_stream16(wbase + (size_t)kbn * kWkBlockBytes + rt * 256 + 128);
                    }
                }
            }
        }
    }

    // Output element (channel row, token column) of tile rt sits in accumulator register
    // (row % 16 / 8) * 2 + column % 2 of lane (row % 8) * 4 + (column % 8) / 2, token group
    // column / 8.  A thread finishes the elements idx = tid, tid + 256, ...; idx % (16 R) is the
    // channel, so consecutive threads store consecutive channels.
    constexpr int kOutPerThread = (C::Rows * 8 * NT + kDecThreads - 1) / kDecThreads;
    int sums[kOutPerThread];
#pragma unroll
    for (int rt = 0; rt < R; ++rt)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) red[warp][(rt * NT + nt) * 4 + e][lane] = c[rt][nt][e];
    __syncthreads();
#pragma unroll
    for (int o = 0; o < kOutPerThread; ++o) {
        const int idx = threadIdx.x + o * kDecThreads;
        const int row = idx % C::Rows, om = idx / C::Rows, col = om & 7;
        const int reg = ((row >> 4) * NT + (om >> 3)) * 4 + ((row >> 3) & 1) * 2 + (col & 1);
        const int ln = (row & 7) * 4 + (col >> 1);
        int sum = 0;
        if (om < 8 * NT) {
#pragma unroll
            for (int w = 0; w < kDecWarps; ++w) sum += red[w][reg][ln];
        }
        sums[o] = sum;
    }

    // ---- scale, add, store ----
#pragma unroll
    for (int o = 0; o < kOutPerThread; ++o) {
        const int idx = threadIdx.x + o * kDecThreads;
        const int row = idx % C::Rows, om = idx / C::Rows, col = om & 7;
        const int on = n0 + row;
        if (om < M && on < N) {
            const int reg = ((row >> 4) * NT + (om >> 3)) * 4 + ((row >> 3) & 1) * 2 + (col & 1);
            const int ln = (row & 7) * 4 + (col >> 1);
            float lr = 0.f;
            for (int w = 0; w < lr_warps; ++w) lr += red_lr[w][reg][ln];
            // the weights were unpacked as 16 q: 1/16 is folded into the scale (exact)
            const float y = fmaf((float)sums[o], a_scale[om] * (__ldg(w_scale + on) * 0.0625f), lr);
            Y[(size_t)om * N + on] = __float2half_rn(y);
            if (acc_debug) acc_debug[(size_t)om * N + on] = sums[o] >> 4;
        }
    }
}

template <int NT, int R, int B>
int launch_cfg(const int8_t* Xq, const float* a_scale, const uint8_t* Wk, const float* w_scale,
               const __nv_bfloat16* T, const __half* LB, int M, int N, int K, int r, __half* Y,
               int32_t* acc_debug, cudaStream_t st, bool overlap_prev, int ldt, CatSplit cat) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((N + DecCfg<NT, R, B>::Rows - 1) / DecCfg<NT, R, B>::Rows, 1, 1);
    cfg.blockDim = dim3(kDecThreads, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap_prev ? 1 : 0;
    cudaError_t e = cudaLaunchKernelEx(&cfg, linear_decode_kernel<NT, R, B>, Xq, a_scale, Wk, w_scale, T, LB,
                                       M, N, K, r, ldt, Y, acc_debug, cat);
    if (e != cudaSuccess) return record_cuda_error(e, "linear_decode_kernel");
    return check_launch("linear_decode_kernel");
}

template <int NT>
int launch_nt(const int8_t* Xq, const float* a_scale, const uint8_t* Wk, const float* w_scale,
              const __nv_bfloat16* T, const __half* LB, int M, int N, int K, int r, __half* Y,
              int32_t* acc_debug, cudaStream_t st, bool overlap_prev, int ldt, CatSplit cat) {
    // Rows per CTA: 32 where that still gives every SM about one and a half CTAs (activation
    // fragments reused twice), else 16 (few output channels: latency matters, every SM gets work).
    int num_sms = 0;
    {
        const int rc = device_sm_count(&num_sms);
        if (rc != ASER_OK) return rc;
    }
    // (Four blocks in flight per warp at 32 rows, i.e. 256 bytes per thread and two CTAs per SM,
    // measured 7 % slower at 8192 x 8192 than two blocks and three CTAs per SM.)
    if (N >= 32 * 3 * num_sms / 2)
        return launch_cfg<NT, 2, 2>(Xq, a_scale, Wk, w_scale, T, LB, M, N, K, r, Y, acc_debug, st, overlap_prev, ldt, cat);
    return launch_cfg<NT, 1, 4>(Xq, a_scale, Wk, w_scale, T, LB, M, N, K, r, Y, acc_debug, st, overlap_prev, ldt, cat);
}

}  // namespace

bool linear_decode_prefers(int M, int N, int K) {
    return M <= kLinearDecodeMaxTokens && (long long)N * K / 2 <= (64ll << 20);
}

int launch_linear_decode(const int8_t* Xq, const float* a_scale, const uint8_t* Wk,
                         const float* w_scale, const __nv_bfloat16* T, const __half* LB,
                         int M, int N, int K, int r, __half* Y, int32_t* acc_debug,
                         cudaStream_t st, bool overlap_prev, int ldt, CatSplit cat) {
    if (ldt <= 0) ldt = r * cat.layers;
    if (M > kLinearDecodeMaxTokens) return record_error(ASER_ERR_SHAPE, "linear_decode: more than 16 tokens");
    if (M <= 8) return launch_nt<1>(Xq, a_scale, Wk, w_scale, T, LB, M, N, K, r, Y, acc_debug, st, overlap_prev, ldt, cat);
    return launch_nt<2>(Xq, a_scale, Wk, w_scale, T, LB, M, N, K, r, Y, acc_debug, st, overlap_prev, ldt, cat);
}

}  // namespace aser
