// Fused activation kernel: smoothing divide (Sec. 4.2, the M^-1 X factor of Eq. 10),
// per-token int8 round-to-nearest (Sec. 5.1) and the down projection T = X~ L_A^T of the
// error-reconstruction branch (Sec. 4.1).
//
// Launch shapes:
//   * few tokens (decode): one CTA per (token, group of L_A rows) so that the L_A stream is
//     spread over many SMs; CUDA-core FMAs in fp32.
//   * many tokens (prefill): clusters of CTAs own 128 tokens each and split K; TMA streams the
//     activations through shared memory twice (row maxima + tcgen05 down projection, then the
//     int8 codes, written back by TMA stores).  See the section below.
//   * a plain mma.sync kernel (16 tokens per CTA) remains for shapes the cluster kernel
//     cannot take.
#include "act_math.cuh"
#include "aser_common.cuh"
#include "sm100_ptx.cuh"

namespace aser {

namespace {

// Eight int8 codes rne(x~ / scale) clamped to +-127, packed low column first.
// The definition uses the IEEE quotient.  |x~ / scale| <= 127 (1 + 2^-23), so x~ * (1/scale)
// differs from the rounded quotient by less than 4 * 2^-24 * 127 < 3.1e-5: whenever that product
// is at least 1e-4 away from every half-integer, both round to the same integer and the
// multiplication stands in for the division.  Only the rare near-ties take the real division.
__device__ __forceinline__ uint2 quant8(const float (&v)[8], float sc, bool nonzero, float qmax) {
    uint32_t w[2] = {0, 0};
    const float rcp = nonzero ? __frcp_rn(sc) : 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        int q = 0;
        if (nonzero) {
            const float t = v[i] * rcp;
            const float fr = fabsf(t) - floorf(fabsf(t));          // fractional part in [0, 1)
            if (fabsf(fr - 0.5f) >= 1e-4f && fabsf(t) < 1e6f) q = rne_clamp(t, -qmax, qmax);
            else q = rne_clamp(__fdiv_rn(v[i], sc), -qmax, qmax);
        }
        w[i >> 2] |= (uint32_t)(q & 0xFF) << (8 * (i & 3));
    }
    return make_uint2(w[0], w[1]);
}

// ---------------------------------------------------------------------------
// few tokens
// ---------------------------------------------------------------------------
constexpr int kSmallThreads = 256;
constexpr int kRowsPerCta = 4;  // L_A rows handled by one projection CTA

// grid = (1 + ceil(r / kRowsPerCta), M).  blockIdx.x == 0 quantizes token blockIdx.y,
// the others compute kRowsPerCta entries of T for that token.
// dynamic smem: K floats (the smoothed row; used by the quantizing CTA).
__global__ void __launch_bounds__(kSmallThreads)
quant_act_small_kernel(const __half* __restrict__ X, const float* __restrict__ s,
                       const __half* __restrict__ LA, int M, int K, int r,
                       int8_t* __restrict__ Xq, float* __restrict__ a_scale,
                       __nv_bfloat16* __restrict__ T, int ldt, int lo_off, float qmax) {
    extern __shared__ __align__(16) float xs[];
    grid_dep_launch();      // a dependent linear kernel may start streaming its weights
    __shared__ float red[kRowsPerCta][kSmallThreads / 32];
    const int m = blockIdx.y;
    const int chunks = K / 8;
    const __half* row = X + (size_t)m * K;

    if (blockIdx.x == 0) {
        // ---- quantize this token: x~ to shared memory with the row maximum, then the codes ----
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
        amax = warp_max(amax);
        if ((threadIdx.x & 31) == 0) red[0][threadIdx.x >> 5] = amax;
        __syncthreads();
        amax = red[0][0];
#pragma unroll
        for (int i = 1; i < kSmallThreads / 32; ++i) amax = fmaxf(amax, red[0][i]);
        const float sc = __fdiv_rn(amax, qmax);
        if (threadIdx.x == 0) a_scale[m] = sc;
        int8_t* out = Xq + (size_t)m * K;
        for (int c = threadIdx.x; c < chunks; c += kSmallThreads) {
            float v[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = xs[c * 8 + i];
            *reinterpret_cast<uint2*>(out + c * 8) = quant8(v, sc, amax > 0.f, qmax);
        }
        return;
    }

    // ---- down projection: kRowsPerCta rows of L_A against the smoothed token.  A thread
    // smooths the chunks it multiplies, so all of its loads (activations, divisors, L_A rows)
    // are in flight together and no barrier separates them. ----
    const int j0 = (blockIdx.x - 1) * kRowsPerCta;
    float acc[kRowsPerCta];
#pragma unroll
    for (int jj = 0; jj < kRowsPerCta; ++jj) acc[jj] = 0.f;
#pragma unroll 2
    for (int c = threadIdx.x; c < chunks; c += kSmallThreads) {
        const RawChunk rc = load_raw(row, s, c * 8, true);
        uint4 la[kRowsPerCta];
#pragma unroll
        for (int jj = 0; jj < kRowsPerCta; ++jj)
            la[jj] = (j0 + jj < r) ? *reinterpret_cast<const uint4*>(LA + (size_t)(j0 + jj) * K + c * 8)
                                   : make_uint4(0, 0, 0, 0);
        float v[8];
        smooth8(rc, v);
#pragma unroll
        for (int jj = 0; jj < kRowsPerCta; ++jj) {
            const __half2* h2 = reinterpret_cast<const __half2*>(&la[jj]);
            const float2 a = __half22float2(h2[0]), b = __half22float2(h2[1]);
            const float2 cc = __half22float2(h2[2]), d = __half22float2(h2[3]);
            float t = acc[jj];
            t = fmaf(a.x, v[0], t); t = fmaf(a.y, v[1], t);
            t = fmaf(b.x, v[2], t); t = fmaf(b.y, v[3], t);
            t = fmaf(cc.x, v[4], t); t = fmaf(cc.y, v[5], t);
            t = fmaf(d.x, v[6], t); t = fmaf(d.y, v[7], t);
            acc[jj] = t;
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
        store_t(T + (size_t)m * ldt, j0 + threadIdx.x, t, lo_off);
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
                       __nv_bfloat16* __restrict__ T, int ldt, int lo_off, float qmax) {
    extern __shared__ __align__(16) uint8_t smem[];
    grid_dep_launch();
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
    const float sc = __fdiv_rn(amax, qmax);
    if (tcol == 0 && row_ok) a_scale[m] = sc;

    // ---- T tile (fp32 accumulators -> bf16) ----
    if (r > 0) {
        const int g = lane >> 2, tq = lane & 3;
#pragma unroll
        for (int t = 0; t < MAXT; ++t) {
            int nt = warp + t * 8;
            if (nt < ntiles) {
                int j = nt * 8 + tq * 2;
                if (m0 + g < M) store_t2(T + (size_t)(m0 + g) * ldt, j, acc[t][0], acc[t][1], lo_off);
                if (m0 + g + 8 < M) store_t2(T + (size_t)(m0 + g + 8) * ldt, j, acc[t][2], acc[t][3], lo_off);
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
        *reinterpret_cast<uint2*>(out + c * kChunkK + tcol * 8) = quant8(v, sc, amax > 0.f, qmax);
    }
}

// ---------------------------------------------------------------------------
// many tokens: TMA ring + tcgen05 down projection, thread-block cluster split along K
// ---------------------------------------------------------------------------
// A cluster of CK CTAs owns 64 tokens; CTA `rank` owns the K-slice [rank*Kc, (rank+1)*Kc) and
// streams it twice through a ring of 128-column stages filled by TMA (two 64-column tiles per
// stage, 128-byte swizzle, rows past M read as zero).
//   Sweep 1: the consumer warps scan each stage for the row maximum of |x~|.  Where all 16
//   divisors of a (row, 16-column) unit are 1 (all but the outlier channels), x~ is the fp16
//   input itself and the stage is left as TMA wrote it; elsewhere x~ = x / s is computed in
//   fp32 and written back as fp16 in place.  One thread then issues tcgen05.mma (kind::f16)
//   with the L_A tile (TMA) on the M side and the stage's 64 tokens on the N side, so the
//   partial T accumulates transposed, D[j, token], in tensor memory.  L_A has fewer than 128
//   rows when r < 128; the MMA then also reads the shared memory behind the tile and the
//   accumulator rows j >= r are never looked at.
//   Exchange: every CTA stores its row maxima into all CTAs of the cluster and its partial T
//   into the CTA that owns the token (64 / CK tokens each), through distributed shared memory;
//   one cluster barrier publishes both.  The owner sums the CK partials and writes T.
//   Sweep 2: the slice is streamed again (it was just read, so it comes from L2), quantized,
//   staged in shared memory and written by TMA stores, which also clip rows past M.
// The 16 consumer warps form two groups that take alternate stages; inside its stage a warp
// handles one 16-column group for all 64 rows (lane = row and row + 32), so whether a unit needs
// the division is uniform across the warp and the swizzled 16-byte accesses are conflict-free.
// A kernel that allocates tensor memory gets one CTA per SM, so the CTA uses most of the SM's
// shared memory: the ring is as deep as fits (up to six stages).
constexpr int kTTok = 64;                   // tokens per cluster (the MMA's N)
constexpr int kTAtom = 64;                  // columns of one swizzled tile: 128 bytes of fp16
constexpr int kTCols = 128;                 // columns per stage (two tiles)
constexpr int kTConsumerWarps = 16;         // two groups of eight: warp = (stage parity, 16-column group)
constexpr int kTGroupWarps = 8;
constexpr int kTConsumers = kTConsumerWarps * 32;
constexpr int kTWarpProd = kTConsumerWarps;         // TMA producer warp
constexpr int kTWarpMma = kTConsumerWarps + 1;      // MMA issuer warp, owns the tensor memory
constexpr int kTThreads = kTConsumers + 64;
constexpr int kTMaxStages = 6;              // deepest activation / L_A ring
constexpr int kTOut = 4;                    // int8 output tiles in flight
constexpr int kTMaxRank = 128;              // larger r takes the mma.sync kernel
constexpr int kXAtomBytes = kTTok * 128;    // 64 rows x 64 fp16
constexpr int kXStageBytes = 2 * kXAtomBytes;
constexpr int kOutTileBytes = kTTok * kTCols;   // 64 rows x 128 int8
constexpr long long kQaWaitLimitClocks = 400000000ll;   // about 0.2 s of SM clocks per wait
constexpr long long kTL2Budget = 72ll << 20;    // bytes of X the second sweep can expect to find in L2
constexpr int kTCacheUnits = 62;            // 16-column units with a divisor whose divisors are kept in shared memory
constexpr int kTUncached = 255;             // tag of such a unit beyond the cache: its divisors are read from global memory

// Ring depth: as many stages (activation tile + L_A tile) as fit beside the exchange buffers.
// A stage takes about 3 k cycles to go round (HBM latency plus the hand-overs between TMA,
// consumers and MMA), so the depth sets the pace of sweep 1.
__host__ __device__ constexpr int tma_stages(int r, int CK) {
    const int per_stage = kXStageBytes + 256 * r;
    const int exch = (CK > 1) ? 2 * kTTok * r * 4 : 0;
    const int fixed = (exch > 16 * 1024 ? exch : 16 * 1024) + 16 * 1024;
    int ns = (227 * 1024 - fixed) / per_stage;
    if (ns * per_stage < kTOut * kOutTileBytes + kXStageBytes * ns) {      // region B must hold the output tiles
        ns = (227 * 1024 - fixed - kTOut * kOutTileBytes) / kXStageBytes;
    }
    return ns > kTMaxStages ? kTMaxStages : (ns < 2 ? 2 : ns);
}

struct TmaSmem {
    int x_ring, region_b, la_atom_bytes, la_stage_bytes, t_slots, t_stage, ones, amax_cg, amax_stage,
        amax_slots, s_cache, bars, tmem_slot, abort_flag, n_cached, total;
};
// Offsets from the 1 KiB-aligned base.  Region B holds the L_A ring in sweep 1 and the output
// tiles in sweep 2.  t_slots receives the partial T of the tokens this CTA owns from every CTA
// of the cluster, as [source CTA][token][r] floats (64 * r floats in all).  It follows region B
// so that an MMA whose L_A tile has fewer than 128 rows still reads inside the allocation.
__host__ __device__ inline TmaSmem tma_smem(int Kc, int r, int CK) {
    TmaSmem L;
    const int ns = tma_stages(r, CK);
    int off = 0;
    L.x_ring = off;     off += ns * kXStageBytes;
    L.region_b = off;
    L.la_atom_bytes = r * 128;
    L.la_stage_bytes = 2 * L.la_atom_bytes;
    {
        int b = ns * L.la_stage_bytes;
        if (kTOut * kOutTileBytes > b) b = kTOut * kOutTileBytes;
        off += (b + 1023) / 1024 * 1024;
    }
    L.t_slots = off;
    {
        int b = (CK > 1) ? kTTok * r * 4 : 0;
        if (b < 16 * 1024) b = 16 * 1024;                      // readable space behind the L_A ring
        off += b;
    }
    L.t_stage = off;    off += (CK > 1) ? kTTok * r * 4 : 0;   // this CTA's partial T, [token][r]
    L.ones = off;       off += (Kc / 16 + 15) / 16 * 16;       // per 16 columns: 0 = all divisors are 1, else a tag
    L.amax_cg = off;    off += 16 * kTTok * 4;                 // row maxima per (stage parity, 16-column group)
    L.amax_stage = off; off += kTTok * 4;                      // row maxima of this CTA's slice
    L.amax_slots = off; off += 16 * kTTok * 4;                 // row maxima copied in by each CTA
    L.s_cache = off;    off += kTCacheUnits * 16 * 4;          // the divisors of the tagged units
    L.bars = off;       off += (4 * kTMaxStages + 2 * kTOut + 3) * 8;
    L.tmem_slot = off;  off += 8;
    L.abort_flag = off; off += 4;
    L.n_cached = off;   off += 4;
    L.total = off + 1024;                                      // slack for the alignment
    return L;
}

__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_arrive() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait() {
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Address of the same shared-memory offset in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t dsmem_addr(uint32_t local_addr, uint32_t rank) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
    return remote;
}
// Bulk copy from this CTA's shared memory into a peer's; the bytes are counted on the peer's
// mbarrier, which is how the peer learns that they have landed.
__device__ __forceinline__ void dsmem_bulk_copy(uint32_t remote_dst, uint32_t local_src, uint32_t bytes,
                                                uint32_t remote_bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(remote_dst), "r"(local_src), "r"(bytes), "r"(remote_bar)
        : "memory");
}

// Bounded wait on an mbarrier phase.  On expiry (or when another thread of the CTA has given
// up) it sets the CTA's abort flag and returns false; the caller leaves its loop.
__device__ __noinline__ bool qa_wait_slow(uint32_t bar, uint32_t parity, volatile int* flag) {
    uint32_t spins = 0;
    long long t0 = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 255u) == 0) {
            if (*flag) return false;
            if (t0 == 0) {
                t0 = clock64();
            } else if (clock64() - t0 > kQaWaitLimitClocks) {
                *flag = 1;
                return false;
            }
        }
    }
    return true;
}
__device__ __forceinline__ bool qa_wait(uint32_t bar, uint32_t parity, volatile int* flag) {
    if (mbar_try_wait(bar, parity)) return true;
    return qa_wait_slow(bar, parity, flag);
}
// Warp-collective form: lane 0 polls, the outcome is broadcast.
__device__ __forceinline__ bool qa_warp_wait(uint32_t bar, uint32_t parity, volatile int* flag, int lane) {
    int ok = 1;
    if (lane == 0) ok = qa_wait(bar, parity, flag) ? 1 : 0;
    return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, int x, int y, uint32_t src) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                 ::"l"(map), "r"(x), "r"(y), "r"(src)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, uint4 v) {
    asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// 8 fp16 -> 8 fp32
__device__ __forceinline__ void cvt8(const uint4& raw, float (&v)[8]) {
    const __half2* h2 = reinterpret_cast<const __half2*>(&raw);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 f = __half22float2(h2[i]);
        v[2 * i] = f.x; v[2 * i + 1] = f.y;
    }
}
// x~ = fp32(x) / s for 8 columns (IEEE divisions).  A column's divisor is the same for every
// lane of the warp (lanes are rows), so skipping the division where it is 1 does not diverge.
__device__ __forceinline__ void div8(const uint4& raw, const float4& s0, const float4& s1, float (&v)[8]) {
    cvt8(raw, v);
    if (s0.x != 1.f) v[0] = __fdiv_rn(v[0], s0.x);
    if (s0.y != 1.f) v[1] = __fdiv_rn(v[1], s0.y);
    if (s0.z != 1.f) v[2] = __fdiv_rn(v[2], s0.z);
    if (s0.w != 1.f) v[3] = __fdiv_rn(v[3], s0.w);
    if (s1.x != 1.f) v[4] = __fdiv_rn(v[4], s1.x);
    if (s1.y != 1.f) v[5] = __fdiv_rn(v[5], s1.y);
    if (s1.z != 1.f) v[6] = __fdiv_rn(v[6], s1.z);
    if (s1.w != 1.f) v[7] = __fdiv_rn(v[7], s1.w);
}

// grid = (CK, ceil(M / 64)), cluster = (CK, 1, 1) with CK a power of two <= 16, kTThreads threads,
// r <= 128.  T has `ldt` elements per row (the launch may cover a column range of a wider T).
// map_x: X as fp16 [K / 64 blocks][M][64], box 2 blocks x 64 rows, 128-byte swizzle.
// map_la: L_A as fp16 [K / 64 blocks][r][64], box 2 blocks x r rows (unused when r == 0).
// map_q: Xq as bytes [M, K], box 64 rows x 128 columns, 128-byte swizzle.
__global__ void __launch_bounds__(kTThreads, 1)
quant_act_tma_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_la,
                     const __grid_constant__ CUtensorMap map_q, const float* __restrict__ s,
                     int M, int K, int Kc, int r, int CK, float* __restrict__ a_scale,
                     __nv_bfloat16* __restrict__ T, int ldt, int lo_off, float qmax) {
    extern __shared__ uint8_t smem_raw[];
    grid_dep_launch();      // a dependent linear kernel may start streaming its weights
    const uint32_t sraw = smem_u32(smem_raw);
    const uint32_t sb = (sraw + 1023u) & ~1023u;            // swizzled tiles need 1 KiB alignment
    uint8_t* smem = smem_raw + (sb - sraw);
    const TmaSmem L = tma_smem(Kc, r, CK);
    const int NS = tma_stages(r, CK);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_rank();
    const int m0 = blockIdx.y * kTTok;
    const int k0 = (int)rank * Kc;
    const int nst = Kc / kTCols;                            // stages per sweep
    const int rows_owned = kTTok / CK;                      // tokens whose T this CTA sums and writes
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L.abort_flag);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L.tmem_slot);
    uint8_t* ones_sm = smem + L.ones;
    float* s_cache = reinterpret_cast<float*>(smem + L.s_cache);
    int* n_cached = reinterpret_cast<int*>(smem + L.n_cached);
    float* amax_cg = reinterpret_cast<float*>(smem + L.amax_cg);
    float* amax_stage = reinterpret_cast<float*>(smem + L.amax_stage);
    float* amax_slots = reinterpret_cast<float*>(smem + L.amax_slots);
    float* t_slots = reinterpret_cast<float*>(smem + L.t_slots);
    float* t_stage = reinterpret_cast<float*>(smem + L.t_stage);
    auto bar_full = [&](int st) { return sb + L.bars + st * 8; };
    auto bar_ready = [&](int st) { return sb + L.bars + (kTMaxStages + st) * 8; };
    auto bar_free1 = [&](int st) { return sb + L.bars + (2 * kTMaxStages + st) * 8; };
    auto bar_free2 = [&](int st) { return sb + L.bars + (3 * kTMaxStages + st) * 8; };
    auto bar_out_full = [&](int o) { return sb + L.bars + (4 * kTMaxStages + o) * 8; };
    auto bar_out_free = [&](int o) { return sb + L.bars + (4 * kTMaxStages + kTOut + o) * 8; };
    const uint32_t bar_acc = sb + L.bars + (4 * kTMaxStages + 2 * kTOut) * 8;
    const uint32_t bar_amax = bar_acc + 8;      // the peers' row maxima have landed
    const uint32_t bar_t = bar_acc + 16;        // the peers' partial T have landed
    constexpr uint32_t kTmemCols = 64;                      // D[j, token]: 64 token columns
    // The two consumer groups take alternate uses of the ring.  A wait on a phase PARITY is only
    // sound for a waiter that observes every phase of its barrier.  With an even ring a stage
    // always comes back to the same group, which therefore sees each of its phases.  With an odd
    // ring the groups alternate on a stage; a warp that only waited for its own uses could find
    // the barrier one phase behind (the other group's load still in flight), read that as "my
    // phase is complete", work on a stage that has not landed and arrive on a barrier out of
    // turn.  So with an odd ring every consumer warp waits for EVERY use of the ring and the
    // warps of the idle group hand the stage on at once: the hand-over barriers then count all
    // sixteen warps.
    const bool all_observe = (NS & 1) != 0;
    const uint32_t ring_arrivals = all_observe ? kTConsumerWarps : kTGroupWarps;

    // Use i of the ring: i < nst is sweep 1 (X and L_A tiles), the rest sweep 2 (X only).
    // A stage's previous use was released by the MMAs (sweep 1) or the consumers (sweep 2).
    auto load_use = [&](int i) -> bool {
        const int st = i % NS;
        if (i >= NS) {
            const int prev = i - NS;
            bool ok;
            if (prev < nst) {
                ok = qa_wait(bar_free1(st), (uint32_t)(prev / NS) & 1u, abort_flag);
            } else {
                const int first = nst + ((st - nst % NS + NS) % NS);
                ok = qa_wait(bar_free2(st), (uint32_t)((prev - first) / NS) & 1u, abort_flag);
            }
            if (!ok) return false;
        }
        const uint32_t xdst = sb + L.x_ring + st * kXStageBytes;
        if (i < nst) {
            const int kcol = k0 + i * kTCols;
            mbar_arrive_expect_tx(bar_full(st), (uint32_t)(kXStageBytes + L.la_stage_bytes));
            tma_load_3d(xdst, &map_x, 0, m0, kcol / kTAtom, bar_full(st));
            if (r > 0) tma_load_3d(sb + L.region_b + st * L.la_stage_bytes, &map_la, 0, 0, kcol / kTAtom, bar_full(st));
        } else {
            const int kcol = k0 + (i - nst) * kTCols;
            mbar_arrive_expect_tx(bar_full(st), (uint32_t)kXStageBytes);
            tma_load_3d(xdst, &map_x, 0, m0, kcol / kTAtom, bar_full(st));
        }
        return true;
    };

    // ---- setup ----
    if (warp == kTWarpProd) {
        // The producer sets up the barriers and fills the ring before anyone else is ready.
        if (lane == 0) {
            for (int st = 0; st < kTMaxStages; ++st) {
                mbar_init(bar_full(st), 1);                     // the producer's expect_tx arrival
                mbar_init(bar_ready(st), ring_arrivals);        // the consumers are done with the stage
                mbar_init(bar_free1(st), 1);                    // sweep 1: the MMAs have read it
                mbar_init(bar_free2(st), ring_arrivals);        // sweep 2: the consumers have read it
            }
            for (int o = 0; o < kTOut; ++o) {
                mbar_init(bar_out_full(o), kTGroupWarps);       // an output tile is written
                mbar_init(bar_out_free(o), 1);                  // its store has read it
            }
            mbar_init(bar_acc, 1);
            mbar_init(bar_amax, 1);
            mbar_init(bar_t, 1);
            *abort_flag = 0;
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
            fence_proxy_async_smem();
            if (CK > 1) {       // bytes the cluster's CTAs will copy in
                mbar_arrive_expect_tx(bar_amax, (uint32_t)(CK * kTTok * 4));
                if (r > 0) mbar_arrive_expect_tx(bar_t, (uint32_t)(kTTok * r * 4));
            }
            for (int i = 0; i < NS && i < 2 * nst; ++i) load_use(i);      // no waits yet
        }
        __syncwarp();
    } else if (warp == kTWarpMma) {
        if (r > 0) {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols)
                         : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
        if (lane == 0) prefetch_tensormap(&map_q);
    } else {
        // Per 16 columns of the slice: are all smoothing divisors 1?  They are on all but the few
        // outlier channels; a unit that has a divisor keeps its sixteen in shared memory, so that
        // the two sweeps never wait for global memory.
        if (tid == 0) *n_cached = 0;
        named_bar_sync(1, kTConsumers);
        for (int g = tid; g < Kc / 16; g += kTConsumers) {
            int tag = 0;
            if (s) {
                const float4* sp = reinterpret_cast<const float4*>(s + k0 + g * 16);
                float4 v[4];
                bool one = true;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    v[i] = __ldg(sp + i);
                    one = one && v[i].x == 1.f && v[i].y == 1.f && v[i].z == 1.f && v[i].w == 1.f;
                }
                if (!one) {
                    const int at = atomicAdd(n_cached, 1);
                    tag = kTUncached;
                    if (at < kTCacheUnits) {
                        tag = at + 1;
#pragma unroll
                        for (int i = 0; i < 4; ++i) reinterpret_cast<float4*>(s_cache + at * 16)[i] = v[i];
                    }
                }
            }
            ones_sm[g] = (uint8_t)tag;
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    // "my barriers are ready for your copies": waited for before the first copy into a peer
    if (CK > 1) cluster_arrive();
    const uint32_t tmem = (r > 0) ? *tmem_slot : 0u;

    if (warp == kTWarpProd) {
        // ================= TMA producer =================
        const int early = (2 * nst < nst + NS) ? 2 * nst : nst + NS;
        bool ok = true;
        if (lane == 0) {
            for (int i = NS; i < early && ok; ++i) ok = load_use(i);
        }
        if (lane == 0) {
            for (int i = (early > NS ? early : NS); i < 2 * nst && ok; ++i) ok = load_use(i);
        }
        __syncwarp();
        if (CK > 1) cluster_wait();
    } else if (warp == kTWarpMma) {
        // ================= MMA issuer, then store issuer =================
        bool ok = true;
        if (lane == 0) {
            // M = 128 rows of L_A (r of them real), N = 64 tokens
            const uint32_t idesc = make_idesc(1u, 0u, 128u, (uint32_t)kTTok);
            for (int i = 0; i < nst; ++i) {
                const int st = i % NS;
                ok = qa_wait(bar_ready(st), (uint32_t)(i / NS) & 1u, abort_flag);
                if (!ok) break;
                if (r > 0) {
                    tc_fence_after();
#pragma unroll
                    for (int a = 0; a < 2; ++a) {
                        const uint64_t adesc = smem_desc_sw128(sb + L.region_b + st * L.la_stage_bytes + a * L.la_atom_bytes);
                        const uint64_t bdesc = smem_desc_sw128(sb + L.x_ring + st * kXStageBytes + a * kXAtomBytes);
#pragma unroll
                        for (int kk = 0; kk < kTAtom / 16; ++kk)
                            mma_f16_ss(tmem, adesc + 2 * kk, bdesc + 2 * kk, idesc, (i != 0 || a != 0 || kk != 0) ? 1u : 0u);
                    }
                    tc_commit(bar_free1(st));
                } else {
                    mbar_arrive(bar_free1(st));
                }
            }
            if (r > 0) tc_commit(bar_acc);      // arrives when every MMA above has completed
        }
        __syncwarp();
        if (CK > 1) cluster_wait();
        if (lane == 0) {
            // Sweep 2: one TMA store per output tile.  A tile goes back to the consumers once
            // the store has read it; the stores run two behind.
            for (int j = 0; j < nst && ok; ++j) {
                const int o = j % kTOut;
                ok = qa_wait(bar_out_full(o), (uint32_t)(j / kTOut) & 1u, abort_flag);
                if (!ok) break;
                tma_store_2d(&map_q, k0 + j * kTCols, m0, sb + L.region_b + o * kOutTileBytes);
                bulk_commit();
                if (j >= 2) {
                    bulk_wait_read<2>();
                    mbar_arrive(bar_out_free((j - 2) % kTOut));
                }
            }
            bulk_wait_read<0>();    // shared memory stays valid until the stores have read it
        }
        __syncwarp();
    } else {
        // ================= consumers =================
        // The 16 consumer warps form two groups that take alternate stages, so that two stages
        // are worked on at any time.  Inside its stage a warp owns one 16-column group for all 64
        // rows: lane = row and row + 32 (two 16-byte pieces each, of one swizzled tile; their
        // places differ in address bit 4).
        const int grp = warp >> 3, cg = warp & 7;
        const int row = lane;                                   // and row + 32
        const uint32_t x_off = (uint32_t)(cg >> 2) * kXAtomBytes + (uint32_t)row * 128u +
                               (uint32_t)(((2 * (cg & 3)) ^ (row & 7)) << 4);
        constexpr uint32_t kRow32 = 32u * 128u;                 // 32 rows further down the tile
        // ---- sweep 1: row maxima; units with divisors get x~ written back as fp16 ----
        float amax0 = 0.f, amax1 = 0.f;
        __half2 hamax0 = __float2half2_rn(0.f), hamax1 = hamax0;
        bool ok = true;
        for (int i = all_observe ? 0 : grp; i < nst; i += all_observe ? 1 : 2) {
            const int st = i % NS;
            ok = qa_warp_wait(bar_full(st), (uint32_t)(i / NS) & 1u, abort_flag, lane);
            if (!ok) break;
            if ((i & 1) != grp) {           // the other group's use: observed, handed on
                if (lane == 0) mbar_arrive(bar_ready(st));
                continue;
            }
            const uint32_t a0 = sb + L.x_ring + st * kXStageBytes + x_off, a1 = a0 ^ 16u;
            const uint4 v0 = lds128(a0), v1 = lds128(a1);
            const uint4 w0 = lds128(a0 + kRow32), w1 = lds128(a1 + kRow32);
            const int tag1 = ones_sm[i * 8 + cg];
            if (tag1 == 0) {
                const __half2* h0 = reinterpret_cast<const __half2*>(&v0);
                const __half2* h1 = reinterpret_cast<const __half2*>(&v1);
                const __half2* g0 = reinterpret_cast<const __half2*>(&w0);
                const __half2* g1 = reinterpret_cast<const __half2*>(&w1);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    hamax0 = __hmax2(hamax0, __habs2(h0[e]));
                    hamax1 = __hmax2(hamax1, __habs2(g0[e]));
                    hamax0 = __hmax2(hamax0, __habs2(h1[e]));
                    hamax1 = __hmax2(hamax1, __habs2(g1[e]));
                }
            } else {
                const float4* sp = (tag1 != kTUncached) ? reinterpret_cast<const float4*>(s_cache + (tag1 - 1) * 16)
                                                        : reinterpret_cast<const float4*>(s + k0 + i * kTCols + cg * 16);
                const float4 s0 = sp[0], s1 = sp[1], s2 = sp[2], s3 = sp[3];
                // Only the columns with a divisor (the same for every lane: lanes are rows) take
                // the fp32 division and maximum and are written back as fp16(x~); the others go
                // through the half-precision maximum like an untagged unit, with the divided
                // columns blanked out of that maximum.  Pieces: 0 and 1 are this lane's first row
                // (columns 0..7 and 8..15 of the unit), 2 and 3 the row 32 further down.
                const float sv[16] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w,
                                      s2.x, s2.y, s2.z, s2.w, s3.x, s3.y, s3.z, s3.w};
                uint32_t wd[4][4] = {{v0.x, v0.y, v0.z, v0.w}, {v1.x, v1.y, v1.z, v1.w},
                                     {w0.x, w0.y, w0.z, w0.w}, {w1.x, w1.y, w1.z, w1.w}};
                uint32_t zd[4][4];
#pragma unroll
                for (int pc = 0; pc < 4; ++pc)
#pragma unroll
                    for (int i = 0; i < 4; ++i) zd[pc][i] = wd[pc][i];
#pragma unroll
                for (int e = 0; e < 16; ++e) {
                    if (sv[e] != 1.f) {
                        const int wi = (e & 7) >> 1;
#pragma unroll
                        for (int rr = 0; rr < 2; ++rr) {
                            const int pc = 2 * rr + (e >> 3);
                            const uint32_t word = wd[pc][wi];
                            const __half hv = __ushort_as_half((unsigned short)((e & 1) ? (word >> 16) : (word & 0xffffu)));
                            const float f = __fdiv_rn(__half2float(hv), sv[e]);
                            if (rr == 0) amax0 = fmaxf(amax0, fabsf(f));
                            else amax1 = fmaxf(amax1, fabsf(f));
                            const uint32_t hb = (uint32_t)__half_as_ushort(__float2half_rn(f));
                            wd[pc][wi] = (e & 1) ? ((word & 0x0000ffffu) | (hb << 16)) : ((word & 0xffff0000u) | hb);
                            zd[pc][wi] &= (e & 1) ? 0x0000ffffu : 0xffff0000u;
                        }
                    }
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    hamax0 = __hmax2(hamax0, __habs2(*reinterpret_cast<const __half2*>(&zd[0][i])));
                    hamax0 = __hmax2(hamax0, __habs2(*reinterpret_cast<const __half2*>(&zd[1][i])));
                    hamax1 = __hmax2(hamax1, __habs2(*reinterpret_cast<const __half2*>(&zd[2][i])));
                    hamax1 = __hmax2(hamax1, __habs2(*reinterpret_cast<const __half2*>(&zd[3][i])));
                }
                sts128(a0, make_uint4(wd[0][0], wd[0][1], wd[0][2], wd[0][3]));
                sts128(a1, make_uint4(wd[1][0], wd[1][1], wd[1][2], wd[1][3]));
                sts128(a0 + kRow32, make_uint4(wd[2][0], wd[2][1], wd[2][2], wd[2][3]));
                sts128(a1 + kRow32, make_uint4(wd[3][0], wd[3][1], wd[3][2], wd[3][3]));
                fence_proxy_async_smem();       // the MMA reads these through the async proxy
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_ready(st));
        }
        amax0 = fmaxf(amax0, fmaxf(__low2float(hamax0), __high2float(hamax0)));
        amax1 = fmaxf(amax1, fmaxf(__low2float(hamax1), __high2float(hamax1)));
        amax_cg[warp * kTTok + row] = amax0;
        amax_cg[warp * kTTok + row + 32] = amax1;
        if (CK > 1) cluster_wait();     // every CTA of the cluster has its barriers set up
        named_bar_sync(1, kTConsumers);
        // ---- row maxima of this slice; copied into every CTA of the cluster (each needs all
        // row scales) ----
        if (tid < kTTok) {
            float a = amax_cg[tid];
#pragma unroll
            for (int g = 1; g < 16; ++g) a = fmaxf(a, amax_cg[g * kTTok + tid]);
            amax_stage[tid] = a;
            fence_proxy_async_smem();
        }
        if (CK > 1) {
            if (warp < 2) named_bar_sync(2, 64);        // the 64 values are written (warps 0 and 1)
            if (tid < CK)       // one lane per destination
                dsmem_bulk_copy(dsmem_addr(sb + L.amax_slots + rank * (kTTok * 4), (uint32_t)tid),
                                sb + L.amax_stage, kTTok * 4, dsmem_addr(bar_amax, (uint32_t)tid));
        }
        // ---- partial T: tensor memory -> shared memory -> the CTAs that own the tokens ----
        if (r > 0) {
            if (ok) ok = qa_warp_wait(bar_acc, 0u, abort_flag, lane);
            tc_fence_after();
            // A warp reaches the 32 lanes (rows j of L_A) of its quarter, warp % 4; the four warps
            // of a quarter take 16 tokens each.
            const int q = warp & 3, t0 = (warp >> 2) * 16;
            const int j = q * 32 + lane;
            if (q * 32 < r) {
                uint32_t v[16];
                tmem_ld16(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)t0, v);
                tmem_wait_ld(v);
                if (j < r) {
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        const int t = t0 + e;
                        if (CK > 1) t_stage[t * r + j] = __uint_as_float(v[e]);
                        else if (m0 + t < M) store_t(T + (size_t)(m0 + t) * ldt, j, __uint_as_float(v[e]), lo_off);
                    }
                }
            }
            tc_fence_before();
            if (CK > 1) {
                fence_proxy_async_smem();
                named_bar_sync(1, kTConsumers);
                if (tid < CK) {
                    const uint32_t bytes = (uint32_t)(rows_owned * r * 4);
                    dsmem_bulk_copy(dsmem_addr(sb + L.t_slots + rank * bytes, (uint32_t)tid),
                                    sb + L.t_stage + (uint32_t)tid * bytes, bytes, dsmem_addr(bar_t, (uint32_t)tid));
                }
            }
        }

        // ---- row scales of this thread's two rows; the owner of a row writes its scale out ----
        float sc0, sc1;
        if (CK > 1) {
            if (ok) ok = qa_warp_wait(bar_amax, 0u, abort_flag, lane);     // all row maxima have landed
            float a = 0.f, b = 0.f;
            for (int qq = 0; qq < CK; ++qq) {
                a = fmaxf(a, amax_slots[qq * kTTok + row]);
                b = fmaxf(b, amax_slots[qq * kTTok + row + 32]);
            }
            sc0 = __fdiv_rn(a, qmax);
            sc1 = __fdiv_rn(b, qmax);
        } else {
            named_bar_sync(1, kTConsumers);
            sc0 = __fdiv_rn(amax_stage[row], qmax);
            sc1 = __fdiv_rn(amax_stage[row + 32], qmax);
        }
        if (warp == 0) {
            if ((int)rank == row / rows_owned && m0 + row < M) a_scale[m0 + row] = sc0;
            if ((int)rank == (row + 32) / rows_owned && m0 + row + 32 < M) a_scale[m0 + row + 32] = sc1;
        }

        // ---- sweep 2: int8 codes into the output tiles (they take the place of the L_A ring;
        // the wait on the accumulator above says the MMAs are done reading it) ----
        const float rcp0 = (sc0 > 0.f) ? __frcp_rn(sc0) : 0.f;
        const float rcp1 = (sc1 > 0.f) ? __frcp_rn(sc1) : 0.f;
        for (int jj = all_observe ? 0 : grp; jj < nst && ok; jj += all_observe ? 1 : 2) {
            const int i = nst + jj, st = i % NS, o = jj % kTOut;
            ok = qa_warp_wait(bar_full(st), (uint32_t)(i / NS) & 1u, abort_flag, lane);
            if (!ok) break;
            if ((jj & 1) != grp) {          // the other group's use: observed, handed on
                if (lane == 0) mbar_arrive(bar_free2(st));
                continue;
            }
            const uint32_t a0 = sb + L.x_ring + st * kXStageBytes + x_off, a1 = a0 ^ 16u;
            const uint4 v0 = lds128(a0), v1 = lds128(a1);
            const uint4 w0 = lds128(a0 + kRow32), w1 = lds128(a1 + kRow32);
            // x~ of the two units (all loaded words are consumed here) ...
            float f0[8], f1[8], g0[8], g1[8];
            const int tag2 = ones_sm[jj * 8 + cg];
            if (tag2 == 0) {
                cvt8(v0, f0);
                cvt8(v1, f1);
                cvt8(w0, g0);
                cvt8(w1, g1);
            } else {
                const float4* sp = (tag2 != kTUncached) ? reinterpret_cast<const float4*>(s_cache + (tag2 - 1) * 16)
                                                        : reinterpret_cast<const float4*>(s + k0 + jj * kTCols + cg * 16);
                const float4 s0 = sp[0], s1 = sp[1], s2 = sp[2], s3 = sp[3];
                div8(v0, s0, s1, f0);
                div8(v1, s2, s3, f1);
                div8(w0, s0, s1, g0);
                div8(w1, s2, s3, g1);
            }
            // ... so the stage can be released now.  An arrival issued straight after the loads,
            // before anything used their results, let the next TMA write overtake them.
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_free2(st));
            const uint2 lo0 = quant8_pairs(f0, sc0, rcp0, qmax);
            const uint2 hi0 = quant8_pairs(f1, sc0, rcp0, qmax);
            const uint2 lo1 = quant8_pairs(g0, sc1, rcp1, qmax);
            const uint2 hi1 = quant8_pairs(g1, sc1, rcp1, qmax);
            if (jj >= kTOut) {      // the store that last read this tile is done with it
                ok = qa_warp_wait(bar_out_free(o), (uint32_t)(jj / kTOut - 1) & 1u, abort_flag, lane);
                if (!ok) break;
            }
            // output tile: rows of 128 bytes, 16-byte piece cg at its swizzled place
            const uint32_t od = sb + L.region_b + o * kOutTileBytes + (uint32_t)row * 128u + (uint32_t)((cg ^ (row & 7)) << 4);
            sts128(od, make_uint4(lo0.x, lo0.y, hi0.x, hi0.y));
            sts128(od + kRow32, make_uint4(lo1.x, lo1.y, hi1.x, hi1.y));
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_out_full(o));
        }

        // ---- T of the tokens this CTA owns: sum of the CK partials -> bf16 ----
        if (CK > 1 && r > 0) {
            if (ok) ok = qa_warp_wait(bar_t, 0u, abort_flag, lane);        // all partials have landed
            const int pairs = r >> 1;
            for (int e = tid; e < rows_owned * pairs; e += kTConsumers) {
                const int tl = e / pairs, col = (e - tl * pairs) * 2;
                const int t = (int)rank * rows_owned + tl;
                float s0 = 0.f, s1 = 0.f;
                for (int qq = 0; qq < CK; ++qq) {
                    const float2 pv = *reinterpret_cast<const float2*>(t_slots + (qq * rows_owned + tl) * r + col);
                    s0 += pv.x; s1 += pv.y;
                }
                if (m0 + t < M) store_t2(T + (size_t)(m0 + t) * ldt, col, s0, s1, lo_off);
            }
        }
        if (*abort_flag && warp == 0) {     // a wait gave up: poison the rows
            if (m0 + row < M) a_scale[m0 + row] = __int_as_float(0x7fc00000);
            if (m0 + row + 32 < M) a_scale[m0 + row + 32] = __int_as_float(0x7fc00000);
        }
    }
    // Nobody leaves while a peer may still copy from or into this CTA's shared memory.
    if (CK > 1) {
        cluster_arrive();
        cluster_wait();
    }
    tc_fence_before();
    __syncthreads();
    if (warp == kTWarpMma && r > 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

// Opts the kernel in to `smem` bytes of dynamic shared memory (the one place that does it, so
// that the value last set is known).
int tma_set_smem(size_t smem) {
    static size_t current[kMaxDevices] = {0};
    int dev = 0;
    const int rc = current_device(&dev);
    if (rc != ASER_OK) return rc;
    if (smem == current[dev]) return ASER_OK;
    cudaError_t e = cudaFuncSetAttribute(quant_act_tma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) {
        current[dev] = 0;
        return record_cuda_error(e, "quant_act_tma smem attribute");
    }
    current[dev] = smem;
    return ASER_OK;
}

// Clusters of `ck` CTAs of this kernel that the device keeps resident at once (0 if it cannot
// schedule that size).  Queried once per (size, shared memory) pair.  The query counts with
// the kernel's opted-in maximum of dynamic shared memory, so that is set to the size asked for.
int tma_active_clusters(int ck, size_t smem) {
    static int cached_all[kMaxDevices][17];
    static size_t cached_smem_all[kMaxDevices][17];
    int dev = 0;
    if (current_device(&dev) != ASER_OK) return 0;
    int* cached = cached_all[dev];
    size_t* cached_smem = cached_smem_all[dev];
    if (cached_smem[ck] == smem && smem != 0) return cached[ck];
    if (tma_set_smem(smem) != ASER_OK) {
        (void)cudaGetLastError();
        return 0;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(ck, 1, 1);
    cfg.blockDim = dim3(kTThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = ck;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, quant_act_tma_kernel, &cfg) != cudaSuccess) {
        (void)cudaGetLastError();
        n = 0;
    }
    cached[ck] = n;
    cached_smem[ck] = smem;
    return n;
}

// Cluster size for the TMA kernel: a power of two (the CTAs split the 64 tokens' T) that
// divides the K / 128 stages.  Larger clusters shorten a CTA's two sweeps but fewer of
// them are resident at once; the estimate is waves x (fixed cost + stages of both sweeps), in
// stage units.  The second sweep finds its slice in L2 only if the slices of all resident
// clusters fit there together; otherwise it streams from HBM again, behind the first sweep's
// traffic, and its stages count double.
int pick_tma_cluster(int M, int K, int r, int max_ck) {
    const int tiles = (M + kTTok - 1) / kTTok, blocks = K / kTCols;      // 128-column stages
    int best = 0;
    long long best_cost = 0;
    for (int ck = 1; ck <= max_ck; ck *= 2) {
        if (blocks % ck) continue;
        const size_t smem = (size_t)tma_smem(K / ck, r, ck).total;
        if (smem > 227 * 1024) continue;
        const int active = tma_active_clusters(ck, smem);
        if (active < 1) continue;
        const long long waves = (tiles + active - 1) / active;
        const long long resident = (tiles < active) ? tiles : active;
        const bool in_l2 = resident * kTTok * (long long)K * 2 <= kTL2Budget;
        const long long cost = waves * (6 + (blocks / ck) * (in_l2 ? 2 : 3));
        if (best == 0 || cost < best_cost) { best = ck; best_cost = cost; }
    }
    return best;
}

int launch_tma(const __half* X, const float* s, const __half* LA, int M, int K, int r,
               int8_t* Xq, float* a_scale, __nv_bfloat16* T, int ldt, int lo_off, float qmax,
               cudaStream_t st, bool* unsupported) {
    *unsupported = false;
    static int max_ck_all[kMaxDevices] = {0};   // 16 where the device allows clusters beyond the portable 8
    int dev = 0;
    {
        const int rc = current_device(&dev);
        if (rc != ASER_OK) return rc;
    }
    if (max_ck_all[dev] == 0) {
        cudaError_t e = cudaFuncSetAttribute(quant_act_tma_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
        max_ck_all[dev] = (e == cudaSuccess) ? 16 : 8;
        if (e != cudaSuccess) (void)cudaGetLastError();
    }
    const int max_ck = max_ck_all[dev];
    if ((M + kTTok - 1) / kTTok > 65535 || r > kTMaxRank) { *unsupported = true; return ASER_OK; }
    const int ck = pick_tma_cluster(M, K, r, max_ck);
    if (ck == 0) { *unsupported = true; return ASER_OK; }
    const int kc = K / ck;
    const size_t smem = (size_t)tma_smem(kc, r, ck).total;
    {
        const int rc = tma_set_smem(smem);
        if (rc != ASER_OK) return rc;
    }
    CUtensorMap mx, mla, mq;
    int rc = encode_map_blocks(&mx, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, X, M, K, kTTok, 2);
    if (rc != ASER_OK) return rc;
    if (r > 0) {
        rc = encode_map_blocks(&mla, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, LA, r, K, r, 2);
        if (rc != ASER_OK) return rc;
    } else {
        mla = mx;
    }
    rc = encode_map_2d(&mq, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, Xq, M, K, kTTok, kTCols, CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc != ASER_OK) return rc;

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(ck, (M + kTTok - 1) / kTTok, 1);
    cfg.blockDim = dim3(kTThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = ck;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, quant_act_tma_kernel, mx, mla, mq, s, M, K, kc, r, ck, a_scale, T, ldt, lo_off, qmax);
    if (e != cudaSuccess) return record_cuda_error(e, "quant_act_tma_kernel");
    return check_launch("quant_act_tma_kernel");
}

template <int MAXT>
int launch_large(const __half* X, const float* s, const __half* LA, int M, int K, int r,
                 int8_t* Xq, float* a_scale, __nv_bfloat16* T, int ldt, int lo_off, float qmax,
                 cudaStream_t st) {
    size_t smem = 2 * (size_t)(kTileM + r) * kRowBytes;
    static size_t configured[kMaxDevices] = {0};   // largest dynamic shared memory size opted into so far
    int dev = 0;
    const int drc = current_device(&dev);
    if (drc != ASER_OK) return drc;
    if (smem > configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(quant_act_large_kernel<MAXT>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return record_cuda_error(e, "quant_act_large smem attribute");
        configured[dev] = smem;
    }
    int grid = (M + kTileM - 1) / kTileM;
    quant_act_large_kernel<MAXT><<<grid, kLargeThreads, smem, st>>>(X, s, LA, M, K, r, Xq, a_scale, T, ldt, lo_off, qmax);
    return check_launch("quant_act_large_kernel");
}

}  // namespace

int launch_quant_act(const __half* X, const float* s, const __half* LA, int M, int K, int r,
                     int8_t* Xq, float* a_scale, __nv_bfloat16* T, cudaStream_t st, int act_bits,
                     bool t_pair) {
    // symmetric codes of act_bits bits in the int8 container: +-127 for 8 bits, +-31 for 6
    const float qmax = (float)((1 << (act_bits - 1)) - 1);
    if (M == 0) return ASER_OK;
    const int ldt = t_pair ? 2 * r : r, lo_off = t_pair ? r : 0;
    if (M <= 32) {
        size_t smem = (size_t)K * sizeof(float);
        static size_t configured[kMaxDevices] = {0};   // beyond the 48 KiB every kernel may use
        int dev = 0;
        const int drc = current_device(&dev);
        if (drc != ASER_OK) return drc;
        if (smem > 48 * 1024 && smem > configured[dev]) {
            cudaError_t e = cudaFuncSetAttribute(quant_act_small_kernel,
                                                 cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return record_cuda_error(e, "quant_act_small smem attribute");
            configured[dev] = smem;
        }
        dim3 grid(1 + (r + kRowsPerCta - 1) / kRowsPerCta, M);
        quant_act_small_kernel<<<grid, kSmallThreads, smem, st>>>(X, s, LA, M, K, r, Xq, a_scale, T, ldt, lo_off, qmax);
        return check_launch("quant_act_small_kernel");
    }
    bool unsupported = false;
    if (r > kTMaxRank && r <= 2 * kTMaxRank) {
        // Two launches of the cluster kernel, each for one half of L_A's rows and the matching
        // columns of T.  Both write the same codes and scales (the arithmetic is deterministic),
        // which costs one extra sweep over X but keeps the projection on the tensor cores.
        const int r1 = r - kTMaxRank;
        int rc = launch_tma(X, s, LA, M, K, kTMaxRank, Xq, a_scale, T, ldt, lo_off, qmax, st, &unsupported);
        if (!unsupported) {
            if (rc != ASER_OK) return rc;
            rc = launch_tma(X, s, LA + (size_t)kTMaxRank * K, M, K, r1, Xq, a_scale, T + kTMaxRank, ldt, lo_off,
                            qmax, st, &unsupported);
            // the shape test is the same for both halves, so the second cannot be refused alone
            if (!unsupported) return rc;
            return record_cuda_error(cudaErrorUnknown, "quant_act: second half refused");
        }
        return launch_large<4>(X, s, LA, M, K, r, Xq, a_scale, T, ldt, lo_off, qmax, st);
    }
    const int rc = launch_tma(X, s, LA, M, K, r, Xq, a_scale, T, ldt, lo_off, qmax, st, &unsupported);
    if (!unsupported) return rc;
    if (r <= 64) return launch_large<1>(X, s, LA, M, K, r, Xq, a_scale, T, ldt, lo_off, qmax, st);
    if (r <= 128) return launch_large<2>(X, s, LA, M, K, r, Xq, a_scale, T, ldt, lo_off, qmax, st);
    return launch_large<4>(X, s, LA, M, K, r, Xq, a_scale, T, ldt, lo_off, qmax, st);
}

}  // namespace aser
