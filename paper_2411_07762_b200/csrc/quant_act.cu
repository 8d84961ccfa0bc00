// Fused activation kernel: smoothing divide (Sec. 4.2, the M^-1 X factor of Eq. 9),
// per-token int8 round-to-nearest (Sec. 5.1) and the down projection T = X~ L_A^T of the
// error-reconstruction branch (Sec. 4.1).
//
// Two launch shapes:
//   * few tokens (decode): one CTA per (token, group of L_A rows) so that the L_A stream is
//     spread over many SMs; CUDA-core FMAs in fp32.
//   * many tokens (prefill): one CTA per 16 tokens; x~ is rounded to fp16 and multiplied with
//     L_A on the tensor cores (mma.sync m16n8k16, fp32 accumulation) while the row absmax is
//     collected; a second sweep over the (L2-resident) rows writes the int8 codes.
#include "aser_common.cuh"

namespace aser {

namespace {

struct RawChunk {  // 8 activations and their 8 smoothing divisors
    uint4 x;
    float4 s0, s1;
};

__device__ __forceinline__ RawChunk load_raw(const __half* xrow, const float* s, int col, bool ok) {
    RawChunk rc;
    rc.x = ok ? *reinterpret_cast<const uint4*>(xrow + col) : make_uint4(0, 0, 0, 0);
    if (s) {
        rc.s0 = *reinterpret_cast<const float4*>(s + col);
        rc.s1 = *reinterpret_cast<const float4*>(s + col + 4);
    } else {
        rc.s0 = make_float4(1.f, 1.f, 1.f, 1.f);
        rc.s1 = rc.s0;
    }
    return rc;
}

// x~ = fp32(x) / s, one IEEE division each.  Dividing by 1 is the identity, and s is 1 on all
// but the few outlier channels, so the (long) division sequence is skipped for such groups.
__device__ __forceinline__ void smooth8(const RawChunk& rc, float (&v)[8]) {
    const __half* h = reinterpret_cast<const __half*>(&rc.x);
    const bool ones = rc.s0.x == 1.f && rc.s0.y == 1.f && rc.s0.z == 1.f && rc.s0.w == 1.f &&
                      rc.s1.x == 1.f && rc.s1.y == 1.f && rc.s1.z == 1.f && rc.s1.w == 1.f;
    if (ones) {
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = __half2float(h[i]);
        return;
    }
    v[0] = __fdiv_rn(__half2float(h[0]), rc.s0.x); v[1] = __fdiv_rn(__half2float(h[1]), rc.s0.y);
    v[2] = __fdiv_rn(__half2float(h[2]), rc.s0.z); v[3] = __fdiv_rn(__half2float(h[3]), rc.s0.w);
    v[4] = __fdiv_rn(__half2float(h[4]), rc.s1.x); v[5] = __fdiv_rn(__half2float(h[5]), rc.s1.y);
    v[6] = __fdiv_rn(__half2float(h[6]), rc.s1.z); v[7] = __fdiv_rn(__half2float(h[7]), rc.s1.w);
}

// Eight int8 codes rne(x~ / scale) clamped to +-127, packed low column first.
// The definition uses the IEEE quotient.  |x~ / scale| <= 127 (1 + 2^-23), so x~ * (1/scale)
// differs from the rounded quotient by less than 4 * 2^-24 * 127 < 3.1e-5: whenever that product
// is at least 1e-4 away from every half-integer, both round to the same integer and the
// multiplication stands in for the division.  Only the rare near-ties take the real division.
__device__ __forceinline__ uint2 quant8(const float (&v)[8], float sc, bool nonzero) {
    uint32_t w[2] = {0, 0};
    const float rcp = nonzero ? __frcp_rn(sc) : 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        int q = 0;
        if (nonzero) {
            const float t = v[i] * rcp;
            const float fr = fabsf(t) - floorf(fabsf(t));          // fractional part in [0, 1)
            if (fabsf(fr - 0.5f) >= 1e-4f && fabsf(t) < 1e6f) q = rne_clamp(t, -127.f, 127.f);
            else q = rne_clamp(__fdiv_rn(v[i], sc), -127.f, 127.f);
        }
        w[i >> 2] |= (uint32_t)(q & 0xFF) << (8 * (i & 3));
    }
    return make_uint2(w[0], w[1]);
}

// Same codes as quant8 with fewer, cheaper instructions.  Conversions between float and int
// run on a narrow pipe, so rounding uses the 1.5 * 2^23 constant instead: for |t| < 2^22,
// t + 12582912.0f is rounded to the nearest-even integer and its low bits hold that integer in
// two's complement.  The distance of t to that integer tells near-ties (within 1e-4 of a
// half-integer), which alone take the real division.  |x~ / scale| <= 127.00002, so the fast
// path needs no clamp.
__device__ __forceinline__ uint2 quant8_fast(const float (&v)[8], float sc, float rcp) {
    const float kMagic = 12582912.0f;   // 1.5 * 2^23
    uint32_t q[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const float t = v[i] * rcp;
        const float u = __fadd_rn(t, kMagic);
        q[i] = __float_as_uint(u);      // low byte = code
        if (fabsf(t - __fadd_rn(u, -kMagic)) > 0.4999f)
            q[i] = (uint32_t)rne_clamp(__fdiv_rn(v[i], sc), -127.f, 127.f);
    }
    // gather the low bytes of eight words
    const uint32_t a01 = __byte_perm(q[0], q[1], 0x0040), a23 = __byte_perm(q[2], q[3], 0x0040);
    const uint32_t a45 = __byte_perm(q[4], q[5], 0x0040), a67 = __byte_perm(q[6], q[7], 0x0040);
    return make_uint2(__byte_perm(a01, a23, 0x5410), __byte_perm(a45, a67, 0x5410));
}

// ---------------------------------------------------------------------------
// few tokens
// ---------------------------------------------------------------------------
constexpr int kSmallThreads = 256;
constexpr int kRowsPerCta = 4;  // L_A rows handled by one projection CTA

// grid = (1 + ceil(r / kRowsPerCta), M).  blockIdx.x == 0 quantizes token blockIdx.y,
// the others compute kRowsPerCta entries of T for that token.
// dynamic smem: K floats (the smoothed row).
__global__ void __launch_bounds__(kSmallThreads)
quant_act_small_kernel(const __half* __restrict__ X, const float* __restrict__ s,
                       const __half* __restrict__ LA, int M, int K, int r,
                       int8_t* __restrict__ Xq, float* __restrict__ a_scale,
                       __nv_bfloat16* __restrict__ T) {
    extern __shared__ __align__(16) float xs[];
    __shared__ float red[kRowsPerCta][kSmallThreads / 32];
    const int m = blockIdx.y;
    const int chunks = K / 8;
    const __half* row = X + (size_t)m * K;

    float amax = 0.f;
    for (int c = threadIdx.x; c < chunks; c += kSmallThreads) {
        RawChunk rc = load_raw(row, s, c * 8, true);
        float v[8];
        smooth8(rc, v);
#pragma unroll
        for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(v[i]));
        *reinterpret_cast<float4*>(xs + c * 8) = make_float4(v[0], v[1], v[2], v[3]);
        *reinterpret_cast<float4*>(xs + c * 8 + 4) = make_float4(v[4], v[5], v[6], v[7]);
    }

    if (blockIdx.x == 0) {
        // ---- quantize this token ----
        amax = warp_max(amax);
        if ((threadIdx.x & 31) == 0) red[0][threadIdx.x >> 5] = amax;
        __syncthreads();
        amax = red[0][0];
#pragma unroll
        for (int i = 1; i < kSmallThreads / 32; ++i) amax = fmaxf(amax, red[0][i]);
        const float sc = __fdiv_rn(amax, 127.0f);
        if (threadIdx.x == 0) a_scale[m] = sc;
        int8_t* out = Xq + (size_t)m * K;
        for (int c = threadIdx.x; c < chunks; c += kSmallThreads) {
            float v[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = xs[c * 8 + i];
            *reinterpret_cast<uint2*>(out + c * 8) = quant8(v, sc, amax > 0.f);
        }
        return;
    }

    // ---- down projection: kRowsPerCta rows of L_A against the smoothed token ----
    __syncthreads();
    const int j0 = (blockIdx.x - 1) * kRowsPerCta;
    float acc[kRowsPerCta];
#pragma unroll
    for (int jj = 0; jj < kRowsPerCta; ++jj) acc[jj] = 0.f;
    for (int c = threadIdx.x; c < chunks; c += kSmallThreads) {
        float4 x0 = *reinterpret_cast<const float4*>(xs + c * 8);
        float4 x1 = *reinterpret_cast<const float4*>(xs + c * 8 + 4);
#pragma unroll
        for (int jj = 0; jj < kRowsPerCta; ++jj) {
            if (j0 + jj < r) {
                uint4 raw = *reinterpret_cast<const uint4*>(LA + (size_t)(j0 + jj) * K + c * 8);
                const __half2* h2 = reinterpret_cast<const __half2*>(&raw);
                float2 a = __half22float2(h2[0]), b = __half22float2(h2[1]);
                float2 cc = __half22float2(h2[2]), d = __half22float2(h2[3]);
                float t = acc[jj];
                t = fmaf(a.x, x0.x, t); t = fmaf(a.y, x0.y, t);
                t = fmaf(b.x, x0.z, t); t = fmaf(b.y, x0.w, t);
                t = fmaf(cc.x, x1.x, t); t = fmaf(cc.y, x1.y, t);
                t = fmaf(d.x, x1.z, t); t = fmaf(d.y, x1.w, t);
                acc[jj] = t;
            }
        }
    }
#pragma unroll
    for (int jj = 0; jj < kRowsPerCta; ++jj) {
        float t = warp_sum(acc[jj]);
        if ((threadIdx.x & 31) == 0) red[jj][threadIdx.x >> 5] = t;
    }
    __syncthreads();
    if (threadIdx.x < kRowsPerCta && j0 + threadIdx.x < r) {
        float t = 0.f;
#pragma unroll
        for (int i = 0; i < kSmallThreads / 32; ++i) t += red[threadIdx.x][i];
        T[(size_t)m * r + j0 + threadIdx.x] = __float2bfloat16_rn(t);
    }
}

// ---------------------------------------------------------------------------
// many tokens
// ---------------------------------------------------------------------------
constexpr int kTileM = 16;          // tokens per CTA (one mma.sync M tile)
constexpr int kChunkK = 128;        // columns staged per pipeline step
constexpr int kLargeThreads = 256;  // 16 threads per token row
constexpr int kRowBytes = kChunkK * 2 + 16;  // padded smem row (272 B): conflict-free ldmatrix

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dst), "l"(src));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& a, uint32_t& b, uint32_t& c,
                                            uint32_t& d) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(a), "=r"(b), "=r"(c), "=r"(d)
                 : "r"(addr)
                 : "memory");
}
__device__ __forceinline__ void mma_f16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                        uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
        "{%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// grid = ceil(M / 16).  dynamic smem: 2 stages x (16 + r) rows x 272 B.
// MAXT = tiles of 8 T-columns per warp = ceil(r / 64).
template <int MAXT>
__global__ void __launch_bounds__(kLargeThreads)
quant_act_large_kernel(const __half* __restrict__ X, const float* __restrict__ s,
                       const __half* __restrict__ LA, int M, int K, int r,
                       int8_t* __restrict__ Xq, float* __restrict__ a_scale,
                       __nv_bfloat16* __restrict__ T) {
    extern __shared__ __align__(16) uint8_t smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int m0 = blockIdx.x * kTileM;
    const int trow = tid >> 4;  // token row of this thread (0..15)
    const int tcol = tid & 15;  // 16-byte column chunk within the 128-column step
    const int m = m0 + trow;
    const bool row_ok = m < M;
    const __half* xrow = X + (size_t)(row_ok ? m : 0) * K;
    const int nch = K / kChunkK;
    const int stage_bytes = (kTileM + r) * kRowBytes;
    const uint32_t smem_base = (uint32_t)__cvta_generic_to_shared(smem);
    const int ntiles = r / 8;

    auto issue_la = [&](int c, int stage) {  // r rows x 16 chunks of 16 B
        const uint32_t dst0 = smem_base + stage * stage_bytes + kTileM * kRowBytes;
        for (int i = tid; i < r * 16; i += kLargeThreads) {
            int j = i >> 4, cc = i & 15;
            cp_async16(dst0 + j * kRowBytes + cc * 16, LA + (size_t)j * K + c * kChunkK + cc * 8);
        }
    };

    float acc[MAXT][4];
#pragma unroll
    for (int t = 0; t < MAXT; ++t)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[t][i] = 0.f;

    float amax = 0.f;
    if (r > 0) issue_la(0, 0);
    cp_async_commit();
    RawChunk rc = load_raw(xrow, s, tcol * 8, row_ok);

    for (int c = 0; c < nch; ++c) {
        const int stage = c & 1;
        if (r > 0 && c + 1 < nch) issue_la(c + 1, stage ^ 1);
        cp_async_commit();
        {
            float v[8];
            smooth8(rc, v);
#pragma unroll
            for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(v[i]));
            if (r > 0) {
                __half2 p0 = __floats2half2_rn(v[0], v[1]), p1 = __floats2half2_rn(v[2], v[3]);
                __half2 p2 = __floats2half2_rn(v[4], v[5]), p3 = __floats2half2_rn(v[6], v[7]);
                uint4 pk;
                pk.x = *reinterpret_cast<uint32_t*>(&p0); pk.y = *reinterpret_cast<uint32_t*>(&p1);
                pk.z = *reinterpret_cast<uint32_t*>(&p2); pk.w = *reinterpret_cast<uint32_t*>(&p3);
                *reinterpret_cast<uint4*>(smem + stage * stage_bytes + trow * kRowBytes + tcol * 16) = pk;
            }
        }
        if (c + 1 < nch) rc = load_raw(xrow, s, (c + 1) * kChunkK + tcol * 8, row_ok);
        if (r > 0) {
            cp_async_wait<1>();
            __syncthreads();
            const uint32_t a_base = smem_base + stage * stage_bytes;
            const uint32_t b_base = a_base + kTileM * kRowBytes;
            // A fragment: lanes 0-15 give rows 0-15 at k, lanes 16-31 rows 0-15 at k+8
            const uint32_t a_addr = a_base + (lane & 15) * kRowBytes + (lane >> 4) * 16;
#pragma unroll
            for (int kk = 0; kk < kChunkK / 32; ++kk) {
                uint32_t a0, a1, a2, a3, a4, a5, a6, a7;
                ldmatrix_x4(a_addr + kk * 64, a0, a1, a2, a3);
                ldmatrix_x4(a_addr + kk * 64 + 32, a4, a5, a6, a7);
#pragma unroll
                for (int t = 0; t < MAXT; ++t) {
                    int nt = warp + t * 8;
                    if (nt < ntiles) {
                        // B: 8 rows of L_A (T columns) x 32 k = four 8x8 matrices along k
                        uint32_t b_addr = b_base + (nt * 8 + (lane & 7)) * kRowBytes + kk * 64 +
                                          (lane >> 3) * 16;
                        uint32_t b0, b1, b2, b3;
                        ldmatrix_x4(b_addr, b0, b1, b2, b3);
                        mma_f16(acc[t], a0, a1, a2, a3, b0, b1);
                        mma_f16(acc[t], a4, a5, a6, a7, b2, b3);
                    }
                }
            }
            __syncthreads();
        }
    }
    cp_async_wait<0>();

    // ---- per-token scale: the 16 threads of a row are 16 consecutive lanes ----
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    const float sc = __fdiv_rn(amax, 127.0f);
    if (tcol == 0 && row_ok) a_scale[m] = sc;

    // ---- T tile (fp32 accumulators -> bf16) ----
    if (r > 0) {
        const int g = lane >> 2, tq = lane & 3;
#pragma unroll
        for (int t = 0; t < MAXT; ++t) {
            int nt = warp + t * 8;
            if (nt < ntiles) {
                int j = nt * 8 + tq * 2;
                if (m0 + g < M)
                    *reinterpret_cast<__nv_bfloat162*>(T + (size_t)(m0 + g) * r + j) =
                        __floats2bfloat162_rn(acc[t][0], acc[t][1]);
                if (m0 + g + 8 < M)
                    *reinterpret_cast<__nv_bfloat162*>(T + (size_t)(m0 + g + 8) * r + j) =
                        __floats2bfloat162_rn(acc[t][2], acc[t][3]);
            }
        }
    }

    // ---- second sweep: int8 codes ----
    if (!row_ok) return;
    int8_t* out = Xq + (size_t)m * K;
    rc = load_raw(xrow, s, tcol * 8, true);
    for (int c = 0; c < nch; ++c) {
        RawChunk cur = rc;
        if (c + 1 < nch) rc = load_raw(xrow, s, (c + 1) * kChunkK + tcol * 8, true);
        float v[8];
        smooth8(cur, v);
        *reinterpret_cast<uint2*>(out + c * kChunkK + tcol * 8) = quant8(v, sc, amax > 0.f);
    }
}

// ---------------------------------------------------------------------------
// many tokens, single pass over X: thread-block cluster split along K
// ---------------------------------------------------------------------------
// A cluster of CK CTAs owns 32 tokens; CTA `rank` owns the K-slice [rank*Kc, (rank+1)*Kc) with
// Kc <= 2048, small enough to keep the raw fp16 activations of the slice in shared memory.
// Sweep 1 (per 64-column chunk): x~ = x / s, row absmax, x~ rounded to fp16 and multiplied with
// the L_A chunk on the tensor cores.  Then the CTAs exchange row maxima and partial T through
// distributed shared memory, and sweep 2 quantizes the resident slice, so X is read from HBM
// exactly once and L_A is re-read once per 32 tokens.
constexpr int kCTok = 32;                   // tokens per cluster
constexpr int kCThreads = 512;              // 16 threads per token row; 16 warps hide latencies
constexpr int kCChunk = 128;                // columns per pipeline step
constexpr int kCRow = kCChunk * 2 + 16;     // padded row of a staged fp16 chunk (272 B)
// L_A chunks in flight: as many as shared memory allows beside the resident activations
__host__ __device__ constexpr int cluster_stages(int r) { return r <= 64 ? 3 : 2; }

struct ClusterSmem {
    int x_raw, s_vec, ones, a_stage, la_stage, t_part, amax_part, scale, total;
};
__host__ __device__ inline ClusterSmem cluster_smem(int Kc, int r) {
    ClusterSmem L;
    int off = 0;
    L.x_raw = off;      off += kCTok * (Kc * 2 + 16);          // raw fp16 activations (padded rows)
    L.s_vec = off;      off += Kc * 4;                         // smoothing divisors of the slice
    L.ones = off;       off += ((Kc / 8 + 15) / 16) * 16;      // per 8 columns: all divisors are 1
    L.a_stage = off;    off += 2 * kCTok * kCRow;              // x~ as fp16, double buffered
    L.la_stage = off;                                          // L_A chunks; afterwards this CTA's
    L.t_part = off;                                            // partial T (fp32) reuses the space
    {
        const int la = cluster_stages(r) * r * kCRow, tp = kCTok * r * 4;
        off += (la > tp ? la : tp) + 16;
    }
    L.amax_part = off;  off += kCTok * 4;
    L.scale = off;      off += kCTok * 4;
    L.total = off;
    return L;
}

__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Read a float from the same shared-memory offset in CTA `rank` of the cluster.
__device__ __forceinline__ float dsmem_ld_f32(uint32_t local_addr, uint32_t rank) {
    uint32_t remote;
    float v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(remote) : "memory");
    return v;
}

// grid = (CK, ceil(M / 32)), cluster = (CK, 1, 1).  NTW = 8-column tiles of T per warp,
// STG = L_A pipeline depth (cluster_stages(r)).
template <int NTW, int STG>
__global__ void __launch_bounds__(kCThreads)
quant_act_cluster_kernel(const __half* __restrict__ X, const float* __restrict__ s,
                         const __half* __restrict__ LA, int M, int K, int Kc, int r, int CK,
                         int8_t* __restrict__ Xq, float* __restrict__ a_scale,
                         __nv_bfloat16* __restrict__ T) {
    extern __shared__ __align__(16) uint8_t smem[];
    const ClusterSmem L = cluster_smem(Kc, r);
    const int xrow_bytes = Kc * 2 + 16;            // padded: rows of a warp fall in different banks
    const uint32_t sb = (uint32_t)__cvta_generic_to_shared(smem);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_rank();
    const int m0 = blockIdx.y * kCTok;
    const int k0 = (int)rank * Kc;
    const int nch = Kc / kCChunk;
    const int trow = tid >> 4, tcg = tid & 15;     // this thread's token row and 8-column group
    const bool row_ok = m0 + trow < M;
    float* s_sm = reinterpret_cast<float*>(smem + L.s_vec);
    float* t_part = reinterpret_cast<float*>(smem + L.t_part);
    float* amax_part = reinterpret_cast<float*>(smem + L.amax_part);
    float* scale_sm = reinterpret_cast<float*>(smem + L.scale);

    // smoothing divisors of the slice (plain loads; ones when s is absent) and, per group of 8
    // columns, whether all of them are 1: there x~ is the fp16 input itself
    uint8_t* ones_sm = smem + L.ones;
    for (int i = tid; i < Kc; i += kCThreads) s_sm[i] = s ? s[k0 + i] : 1.f;
    for (int g8 = tid; g8 < Kc / 8; g8 += kCThreads) {
        bool one = true;
        if (s)
            for (int i = 0; i < 8; ++i) one = one && (s[k0 + g8 * 8 + i] == 1.f);
        ones_sm[g8] = one ? 1 : 0;
    }

    // Activations go to their final place, so they can be requested far ahead of use (the L_A
    // ring cannot): kXAhead chunks = 64 KiB in flight per SM, what an HBM-bound stream needs.
    constexpr int kXAhead = 8;
    auto issue_x = [&](int c) {
        // 32 rows x 256 B, one 16-byte copy per thread (zero rows past M)
        const uint32_t xdst = sb + L.x_raw + trow * xrow_bytes + c * (kCChunk * 2) + tcg * 16;
        if (row_ok) cp_async16(xdst, X + (size_t)(m0 + trow) * K + k0 + c * kCChunk + tcg * 8);
        else *reinterpret_cast<uint4*>(smem + L.x_raw + trow * xrow_bytes + c * (kCChunk * 2) + tcg * 16) = make_uint4(0, 0, 0, 0);
    };
    auto issue_chunk = [&](int c) {
        if (c + kXAhead < nch) issue_x(c + kXAhead);
        // L_A chunk: r rows x 256 B
        const uint32_t ldst = sb + L.la_stage + (c % STG) * r * kCRow;
        for (int i = tid; i < r * 16; i += kCThreads) {
            const int j = i >> 4, cc = i & 15;
            cp_async16(ldst + j * kCRow + cc * 16, LA + (size_t)j * K + k0 + c * kCChunk + cc * 8);
        }
    };

    float acc[NTW][4];
#pragma unroll
    for (int i = 0; i < NTW; ++i)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[i][e] = 0.f;
    const int mt = warp & 1, nq = warp >> 1;
    const int ntiles = r / 8;

    for (int c = 0; c < kXAhead && c < nch; ++c) issue_x(c);   // joins the first commit group
    for (int c = 0; c < STG - 1; ++c) {
        if (c < nch) issue_chunk(c);
        cp_async_commit();
    }
    float amax = 0.f;
    __half2 hamax = __float2half2_rn(0.f);
    for (int c = 0; c < nch; ++c) {
        cp_async_wait<STG - 2>();      // chunk c has landed (for this thread's copies)
        __syncthreads();                    // ... and for everyone's; chunk c-1 is fully consumed
        if (c + STG - 1 < nch) issue_chunk(c + STG - 1);   // refills the stage of chunk c-1
        cp_async_commit();
        // x~ for this thread's 8 columns
        {
            const uint4 raw = *reinterpret_cast<const uint4*>(smem + L.x_raw + trow * xrow_bytes + c * (kCChunk * 2) + tcg * 16);
            uint4 pk;
            if (ones_sm[c * (kCChunk / 8) + tcg]) {
                // x~ == x: maximum of |x| in fp16 arithmetic is exact, the MMA operand is the input
                const __half2* h2 = reinterpret_cast<const __half2*>(&raw);
#pragma unroll
                for (int i = 0; i < 4; ++i) hamax = __hmax2(hamax, __habs2(h2[i]));
                pk = raw;
            } else {
                const float4 s0 = *reinterpret_cast<const float4*>(s_sm + c * kCChunk + tcg * 8);
                const float4 s1 = *reinterpret_cast<const float4*>(s_sm + c * kCChunk + tcg * 8 + 4);
                RawChunk rc{raw, s0, s1};
                float v[8];
                smooth8(rc, v);
#pragma unroll
                for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(v[i]));
                __half2 p0 = __floats2half2_rn(v[0], v[1]), p1 = __floats2half2_rn(v[2], v[3]);
                __half2 p2 = __floats2half2_rn(v[4], v[5]), p3 = __floats2half2_rn(v[6], v[7]);
                pk.x = *reinterpret_cast<uint32_t*>(&p0); pk.y = *reinterpret_cast<uint32_t*>(&p1);
                pk.z = *reinterpret_cast<uint32_t*>(&p2); pk.w = *reinterpret_cast<uint32_t*>(&p3);
            }
            if (r > 0)
                *reinterpret_cast<uint4*>(smem + L.a_stage + (c & 1) * kCTok * kCRow + trow * kCRow + tcg * 16) = pk;
        }
        if (r > 0) {
            __syncthreads();
            const uint32_t a_base = sb + L.a_stage + (c & 1) * kCTok * kCRow + (mt * 16 + (lane & 15)) * kCRow + (lane >> 4) * 16;
            const uint32_t b_base = sb + L.la_stage + (c % STG) * r * kCRow + (lane & 7) * kCRow + (lane >> 3) * 16;
#pragma unroll
            for (int kk = 0; kk < kCChunk / 32; ++kk) {
                uint32_t a0, a1, a2, a3, a4, a5, a6, a7;
                ldmatrix_x4(a_base + kk * 64, a0, a1, a2, a3);
                ldmatrix_x4(a_base + kk * 64 + 32, a4, a5, a6, a7);
#pragma unroll
                for (int i = 0; i < NTW; ++i) {
                    const int nt = nq + 8 * i;
                    if (nt < ntiles) {
                        uint32_t b0, b1, b2, b3;
                        ldmatrix_x4(b_base + nt * 8 * kCRow + kk * 64, b0, b1, b2, b3);
                        mma_f16(acc[i], a0, a1, a2, a3, b0, b1);
                        mma_f16(acc[i], a4, a5, a6, a7, b2, b3);
                    }
                }
            }
        }
    }
    cp_async_wait<0>();
    __syncthreads();        // every warp is done with the L_A stages: their space now holds T

    // ---- publish this CTA's partial results for the cluster ----
    amax = fmaxf(amax, fmaxf(__low2float(hamax), __high2float(hamax)));
    // row maximum over this thread's 8-column groups: the 16 threads of a row are adjacent lanes
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    if (tcg == 0) amax_part[trow] = amax;
    if (r > 0) {
        const int g = lane >> 2, tq = lane & 3;
#pragma unroll
        for (int i = 0; i < NTW; ++i) {
            const int nt = nq + 8 * i;
            if (nt < ntiles) {
                const int j = nt * 8 + tq * 2;
                *reinterpret_cast<float2*>(t_part + (mt * 16 + g) * r + j) = make_float2(acc[i][0], acc[i][1]);
                *reinterpret_cast<float2*>(t_part + (mt * 16 + g + 8) * r + j) = make_float2(acc[i][2], acc[i][3]);
            }
        }
    }
    cluster_sync_all();

    // ---- row scales: maximum over the K-slices (every CTA needs them for its own slice) ----
    if (tid < kCTok) {
        float a = 0.f;
        for (int q = 0; q < CK; ++q) a = fmaxf(a, dsmem_ld_f32(sb + L.amax_part + tid * 4, q));
        const float sc = __fdiv_rn(a, 127.0f);
        scale_sm[tid] = sc;
        if (rank == 0 && m0 + tid < M) a_scale[m0 + tid] = sc;
    }
    // ---- T: sum of the partial products; the cluster's CTAs share the elements ----
    if (r > 0) {
        for (int e = (int)rank * kCThreads + tid; e < kCTok * r; e += CK * kCThreads) {
            float sum = 0.f;
            for (int q = 0; q < CK; ++q) sum += dsmem_ld_f32(sb + L.t_part + e * 4, q);
            const int row = e / r, j = e - row * r;
            if (m0 + row < M) T[(size_t)(m0 + row) * r + j] = __float2bfloat16_rn(sum);
        }
    }
    cluster_sync_all();      // nobody leaves (or reuses shared memory) while peers still read it

    // ---- sweep 2: int8 codes of the resident slice ----
    if (!row_ok) return;
    const float sc = scale_sm[trow];
    int8_t* out = Xq + (size_t)(m0 + trow) * K + k0;
    if (!(sc > 0.f)) {   // all-zero token: codes 0
        for (int c = 0; c < nch; ++c) *reinterpret_cast<uint2*>(out + c * kCChunk + tcg * 8) = make_uint2(0, 0);
        return;
    }
    const float rcp = __frcp_rn(sc);
    for (int c = 0; c < nch; ++c) {
        const uint4 raw = *reinterpret_cast<const uint4*>(smem + L.x_raw + trow * xrow_bytes + c * (kCChunk * 2) + tcg * 16);
        float v[8];
        if (ones_sm[c * (kCChunk / 8) + tcg]) {
            const __half2* h2 = reinterpret_cast<const __half2*>(&raw);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 f = __half22float2(h2[i]);
                v[2 * i] = f.x; v[2 * i + 1] = f.y;
            }
        } else {
            const float4 s0 = *reinterpret_cast<const float4*>(s_sm + c * kCChunk + tcg * 8);
            const float4 s1 = *reinterpret_cast<const float4*>(s_sm + c * kCChunk + tcg * 8 + 4);
            RawChunk rc{raw, s0, s1};
            smooth8(rc, v);
        }
        *reinterpret_cast<uint2*>(out + c * kCChunk + tcg * 8) = quant8_fast(v, sc, rcp);
    }
}

// Smallest cluster size (<= 8) whose K-slice fits shared memory and is a whole number of chunks.
int pick_cluster(int K, int r) {
    for (int ck = 1; ck <= 8; ++ck) {
        if (K % ck) continue;
        const int kc = K / ck;
        if (kc % kCChunk) continue;
        if (cluster_smem(kc, r).total <= 226 * 1024 && kc <= 2048) return ck;
    }
    return 0;
}

template <int NTW, int STG>
int launch_cluster(const __half* X, const float* s, const __half* LA, int M, int K, int r, int ck,
                   int8_t* Xq, float* a_scale, __nv_bfloat16* T, cudaStream_t st) {
    const int kc = K / ck;
    const size_t smem = (size_t)cluster_smem(kc, r).total;
    static size_t configured = 0;
    if (smem > configured) {
        cudaError_t e = cudaFuncSetAttribute(quant_act_cluster_kernel<NTW, STG>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return record_cuda_error(e, "quant_act_cluster smem attribute");
        configured = smem;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(ck, (M + kCTok - 1) / kCTok, 1);
    cfg.blockDim = dim3(kCThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = ck;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, quant_act_cluster_kernel<NTW, STG>, X, s, LA, M, K, kc, r, ck,
                                       Xq, a_scale, T);
    if (e != cudaSuccess) return record_cuda_error(e, "quant_act_cluster_kernel");
    return check_launch("quant_act_cluster_kernel");
}

template <int MAXT>
int launch_large(const __half* X, const float* s, const __half* LA, int M, int K, int r,
                 int8_t* Xq, float* a_scale, __nv_bfloat16* T, cudaStream_t st) {
    size_t smem = 2 * (size_t)(kTileM + r) * kRowBytes;
    static size_t configured = 0;   // largest dynamic shared memory size opted into so far
    if (smem > configured) {
        cudaError_t e = cudaFuncSetAttribute(quant_act_large_kernel<MAXT>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return record_cuda_error(e, "quant_act_large smem attribute");
        configured = smem;
    }
    int grid = (M + kTileM - 1) / kTileM;
    quant_act_large_kernel<MAXT><<<grid, kLargeThreads, smem, st>>>(X, s, LA, M, K, r, Xq, a_scale, T);
    return check_launch("quant_act_large_kernel");
}

}  // namespace

int launch_quant_act(const __half* X, const float* s, const __half* LA, int M, int K, int r,
                     int8_t* Xq, float* a_scale, __nv_bfloat16* T, cudaStream_t st) {
    if (M == 0) return ASER_OK;
    if (M <= 32) {
        size_t smem = (size_t)K * sizeof(float);
        static size_t configured = 48 * 1024;
        if (smem > configured) {
            cudaError_t e = cudaFuncSetAttribute(quant_act_small_kernel,
                                                 cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return record_cuda_error(e, "quant_act_small smem attribute");
            configured = smem;
        }
        dim3 grid(1 + (r + kRowsPerCta - 1) / kRowsPerCta, M);
        quant_act_small_kernel<<<grid, kSmallThreads, smem, st>>>(X, s, LA, M, K, r, Xq, a_scale, T);
        return check_launch("quant_act_small_kernel");
    }
    const int ck = pick_cluster(K, r);
    if (ck > 0 && (long long)((M + kCTok - 1) / kCTok) <= 65535) {
        if (r <= 64) return launch_cluster<1, 3>(X, s, LA, M, K, r, ck, Xq, a_scale, T, st);
        if (r <= 128) return launch_cluster<2, 2>(X, s, LA, M, K, r, ck, Xq, a_scale, T, st);
        return launch_cluster<4, 2>(X, s, LA, M, K, r, ck, Xq, a_scale, T, st);
    }
    if (r <= 64) return launch_large<1>(X, s, LA, M, K, r, Xq, a_scale, T, st);
    if (r <= 128) return launch_large<2>(X, s, LA, M, K, r, Xq, a_scale, T, st);
    return launch_large<4>(X, s, LA, M, K, r, Xq, a_scale, T, st);
}

}  // namespace aser
