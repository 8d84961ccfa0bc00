// Activation path for many tokens when the caller provides scratch memory: two kernels.
//
//   act_proj_kernel    reads X once from HBM.  A CTA owns 128 tokens and one slice of K; TMA
//                      streams the slice through a shared-memory ring together with the matching
//                      columns of L_A.  The consumer warps take the row maxima of |x / s| (and
//                      write x / s back as fp16 where s != 1), one thread issues tcgen05.mma
//                      (kind::f16) with L_A on the M side (up to four groups of 128 rows, so the
//                      down projections of several layers that share X are computed in one pass)
//                      and the 128 tokens on the N side; the partial T of the slice goes to the
//                      scratch as fp32 and the partial row maxima beside it.
//   act_quant_kernel   per token row: the scale from the slices' maxima, the int8 codes (X comes
//                      from L2 as far as it is still there), and T as the sum of the slices'
//                      partials in a fixed order, rounded to bf16.
//
// (Sec. 4.2 smoothing M^-1 X of Eq. 10, Sec. 5.1 per-token round-to-nearest, Sec. 4.1 projection
// V_r^T S^-1 of the reconstruction branch.)  Both kernels are deterministic: no atomics.
// Every mbarrier wait is bounded; a CTA that gives up poisons its row maxima with NaN.
#include "act_math.cuh"
#include "aser_common.cuh"
#include "sm100_ptx.cuh"

namespace aser {

namespace {

constexpr int kPTok = 128;                  // tokens per CTA (the MMA's N)
constexpr int kPCols = 64;                  // columns per stage: one 128-byte swizzled tile row
constexpr int kPConsumerWarps = 8;
constexpr int kPWarpLa = 2 + kPConsumerWarps;           // producer of the L_A tiles
constexpr int kPThreads = (3 + kPConsumerWarps) * 32;   // X producer, MMA issuer, consumers, L_A producer
constexpr int kPTileBytes = kPTok * 128;    // 128 rows x 64 fp16 (an X tile or one L_A group tile)
constexpr int kPMaxGroups = 4;              // 128-row groups of L_A: r <= 512
constexpr int kProjPlanSms = 148;           // chunks and slices are planned for this many SMs (the
                                            // scratch size must not depend on the device)
constexpr long long kPWaitLimitClocks = 400000000ll;   // about 0.2 s of SM clocks per wait
constexpr int kPCacheUnits = 254;           // 8-column units with a divisor whose divisors are kept in shared memory
constexpr int kPUncached = 255;             // tag of such a unit beyond the cache: its divisors are read from global memory

__host__ __device__ constexpr int proj_stages(int groups) {
    const int per_stage = kPTileBytes * (1 + groups);
    const int ns = (220 * 1024) / per_stage;
    return ns > 8 ? 8 : ns;                 // 8, 6, 4, 3, 2 stages for 0..4 groups
}

__device__ __noinline__ bool pj_wait_slow(uint32_t bar, uint32_t parity, volatile int* flag) {
    uint32_t spins = 0;
    long long t0 = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 255u) == 0) {
            if (*flag) return false;
            if (t0 == 0) {
                t0 = clock64();
            } else if (clock64() - t0 > kPWaitLimitClocks) {
                *flag = 1;
                return false;
            }
        }
    }
    return true;
}
__device__ __forceinline__ bool pj_wait(uint32_t bar, uint32_t parity, volatile int* flag) {
    if (mbar_try_wait(bar, parity)) return true;
    return pj_wait_slow(bar, parity, flag);
}
__device__ __forceinline__ bool pj_warp_wait(uint32_t bar, uint32_t parity, volatile int* flag, int lane) {
    int ok = 1;
    if (lane == 0) ok = pj_wait(bar, parity, flag) ? 1 : 0;
    return __shfl_sync(0xffffffffu, ok, 0) != 0;
}
__device__ __forceinline__ uint4 pj_lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void pj_sts128(uint32_t addr, uint4 v) {
    asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// grid = (KS slices, token tiles of the chunk).  Scratch of the chunk:
//   amax_part [KS][Mc]      fp32   row maxima of |x~| over the slice (NaN: the CTA gave up)
//   t_part    [KS][groups][Mc][128]  fp32   partial T, by 128-row group of L_A (rows past r: unspecified)
// map_x: X as fp16 [K / 64 blocks][M][64], box 1 block x 128 rows, 128-byte swizzle (rows past
// M read as zero).  map_la: L_A as fp16 [K / 64 blocks][r][64], box 1 block x r rows (r / 2 rows
// above 256).
__global__ void __launch_bounds__(kPThreads, 1)
act_proj_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_la,
                const float* __restrict__ s, int m_first, int Mc, int K, int Kc, int r,
                float* __restrict__ amax_part, float* __restrict__ t_part) {
    // The r rows of L_A arrive as one box (r <= 256, the largest box) or as two boxes of r / 2
    // rows; in shared memory the rows follow one another, 128 bytes each, so group g is the 16 KB
    // at g * 16 KB whatever the boxes.  Where r is not a multiple of 128 the last group's MMA also
    // reads the stale rows behind row r; their accumulator rows are never read.
    const int la_boxes = r <= 256 ? 1 : 2;
    const int la_box_rows = r / la_boxes;
    const uint32_t la_stage_bytes = (uint32_t)r * 128u;
    extern __shared__ uint8_t smem_raw[];
    grid_dep_launch();
    const uint32_t sraw = smem_u32(smem_raw);
    const uint32_t sb = (sraw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (sb - sraw);
    const int groups = (r + 127) / 128;
    const int NS = proj_stages(groups);
    const int stage_bytes = kPTileBytes * (1 + groups);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int ks = blockIdx.x, tile = blockIdx.y;
    const int k0 = ks * Kc;
    const int nst = Kc / kPCols;
    const int row0 = tile * kPTok;                  // first token of the tile inside the chunk
    // after the ring: barriers, flags, the per-warp row maxima
    uint8_t* tail = smem + NS * stage_bytes;
    const uint32_t bars = sb + NS * stage_bytes;
    auto bar_full = [&](int st) { return bars + st * 8; };
    auto bar_ready = [&](int st) { return bars + (8 + st) * 8; };
    auto bar_free = [&](int st) { return bars + (16 + st) * 8; };
    const uint32_t bar_acc = bars + 24 * 8;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail + 25 * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 25 * 8 + 8);
    volatile int* never_flag = abort_flag + 1;                      // stays 0: waits of the wind-down
    // per 8 columns of the slice: 0 = all divisors are 1, else 1 + the unit's place in s_cache (or kPUncached)
    uint8_t* unit_tag = tail + 256;
    float* amax_w = reinterpret_cast<float*>(tail + 256 + ((Kc / 8 + 15) & ~15));   // [8 warps][128 rows]
    float* s_cache = amax_w + kPConsumerWarps * kPTok;              // [kPCacheUnits][8] divisors
    int* n_cached = reinterpret_cast<int*>(tail + 25 * 8 + 16);
    const uint32_t tmem_cols = groups <= 1 ? 128u : groups == 2 ? 256u : 512u;

    if (warp == 0) {
        if (lane == 0) {
            for (int st = 0; st < 8; ++st) {
                mbar_init(bar_full(st), r > 0 ? 2 : 1);      // the X producer and the L_A producer
                mbar_init(bar_ready(st), kPConsumerWarps);
                mbar_init(bar_free(st), 1);
            }
            mbar_init(bar_acc, 1);
            *abort_flag = 0;
            *never_flag = 0;
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
            fence_proxy_async_smem();
            prefetch_tensormap(&map_x);
            if (r > 0) prefetch_tensormap(&map_la);
            // The first round of the ring is requested before the other warps are ready: it needs
            // only the barriers set up above.  X may come from the kernel before this one.
            grid_dep_wait();
            for (int i = 0; i < NS && i < nst; ++i) {
                mbar_arrive_expect_tx(bar_full(i), (uint32_t)kPTileBytes);
                tma_load_3d(sb + i * stage_bytes, &map_x, 0, m_first + row0, (k0 + i * kPCols) / kPCols, bar_full(i));
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (r > 0) {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32(tmem_slot)), "r"(tmem_cols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    } else if (warp < kPWarpLa) {
        // The smoothing divisors are 1 on all but the few outlier channels.  A unit that has one
        // keeps its eight divisors in shared memory, so that the streaming loop below never waits
        // for global memory.
        if (tid == 64) *n_cached = 0;
        named_bar_sync(1, kPConsumerWarps * 32);
        for (int g = tid - 64; g < Kc / 8; g += kPConsumerWarps * 32) {
            int tag = 0;
            if (s) {
                const float4 a = __ldg(reinterpret_cast<const float4*>(s + k0 + g * 8));
                const float4 b = __ldg(reinterpret_cast<const float4*>(s + k0 + g * 8) + 1);
                const bool one = a.x == 1.f && a.y == 1.f && a.z == 1.f && a.w == 1.f &&
                                 b.x == 1.f && b.y == 1.f && b.z == 1.f && b.w == 1.f;
                if (!one) {
                    const int at = atomicAdd(n_cached, 1);
                    tag = kPUncached;
                    if (at < kPCacheUnits) {
                        tag = at + 1;
                        *reinterpret_cast<float4*>(s_cache + at * 8) = a;
                        *reinterpret_cast<float4*>(s_cache + at * 8 + 4) = b;
                    }
                }
            }
            unit_tag[g] = (uint8_t)tag;
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = (r > 0) ? *tmem_slot : 0u;

    if (warp == 0) {
        // ================= TMA producer =================
        if (lane == 0) {
            bool ok = true;
            int issued = (NS < nst) ? NS : nst;
            for (int i = issued; i < nst && ok; ++i) {
                const int st = i % NS;
                ok = pj_wait(bar_free(st), (uint32_t)(i / NS - 1) & 1u, abort_flag);
                if (!ok) break;
                const uint32_t dst = sb + st * stage_bytes;
                const int kblk = (k0 + i * kPCols) / kPCols;
                mbar_arrive_expect_tx(bar_full(st), (uint32_t)kPTileBytes);
                tma_load_3d(dst, &map_x, 0, m_first + row0, kblk, bar_full(st));
                ++issued;
            }
            if (*abort_flag) {      // let copies already issued land before the shared memory goes away
                for (int i = (issued > NS ? issued - NS : 0); i < issued; ++i)
                    pj_wait(bar_full(i % NS), (uint32_t)(i / NS) & 1u, never_flag);
            }
        }
    } else if (warp == kPWarpLa) {
        // ================= L_A producer: one box of up to 256 rows (two groups) per copy =================
        if (lane == 0 && r > 0) {
            bool ok = true;
            int issued = 0;
            for (int i = 0; i < nst && ok; ++i) {
                const int st = i % NS;
                if (i >= NS) ok = pj_wait(bar_free(st), (uint32_t)(i / NS - 1) & 1u, abort_flag);
                if (!ok) break;
                const uint32_t dst = sb + st * stage_bytes + kPTileBytes;
                const int kblk = (k0 + i * kPCols) / kPCols;
                mbar_arrive_expect_tx(bar_full(st), la_stage_bytes);
                for (int b = 0; b < la_boxes; ++b)
                    tma_load_3d(dst + b * la_box_rows * 128, &map_la, 0, b * la_box_rows, kblk, bar_full(st));
                ++issued;
            }
            if (*abort_flag) {
                for (int i = (issued > NS ? issued - NS : 0); i < issued; ++i)
                    pj_wait(bar_full(i % NS), (uint32_t)(i / NS) & 1u, never_flag);
            }
        }
    } else if (warp == 1) {
        // ================= MMA issuer =================
        if (lane == 0) {
            const uint32_t idesc = make_idesc(1u, 0u, 128u, (uint32_t)kPTok);
            bool ok = true;
            for (int i = 0; i < nst && ok; ++i) {
                const int st = i % NS;
                ok = pj_wait(bar_ready(st), (uint32_t)(i / NS) & 1u, abort_flag);
                if (!ok) break;
                if (r > 0) {
                    tc_fence_after();
                    const uint64_t bdesc = smem_desc_sw128(sb + st * stage_bytes);
                    for (int g = 0; g < groups; ++g) {
                        const uint64_t adesc = smem_desc_sw128(sb + st * stage_bytes + (1 + g) * kPTileBytes);
#pragma unroll
                        for (int kk = 0; kk < kPCols / 16; ++kk)
                            mma_f16_ss(tmem + g * 128, adesc + 2 * kk, bdesc + 2 * kk, idesc, (i != 0 || kk != 0) ? 1u : 0u);
                    }
                    tc_commit(bar_free(st));
                } else {
                    mbar_arrive(bar_free(st));
                }
            }
            if (r > 0) {
                tc_commit(bar_acc);     // arrives when every MMA issued above has completed
                if (!ok) pj_wait(bar_acc, 0u, never_flag);      // giving up: let them finish before leaving
            }
        }
    } else if (warp < kPWarpLa) {
        // ================= consumers =================
        // Warp cw owns the 16-byte piece cw (8 columns) of every row; lane = rows lane, +32, +64, +96.
        const int cw = warp - 2;
        float amax[4] = {0.f, 0.f, 0.f, 0.f};
        __half2 hmax[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) hmax[q] = __float2half2_rn(0.f);
        bool ok = true;
        for (int i = 0; i < nst; ++i) {
            const int st = i % NS;
            ok = pj_warp_wait(bar_full(st), (uint32_t)(i / NS) & 1u, abort_flag, lane);
            if (!ok) break;
            const uint32_t base = sb + st * stage_bytes;
            uint32_t addr[4];
            uint4 v[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int row = lane + 32 * q;
                addr[q] = base + (uint32_t)row * 128u + (uint32_t)((cw ^ (row & 7)) << 4);
                v[q] = pj_lds128(addr[q]);
            }
            const int tag = unit_tag[i * 8 + cw];
            if (tag == 0) {
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const __half2* h = reinterpret_cast<const __half2*>(&v[q]);
#pragma unroll
                    for (int e = 0; e < 4; ++e) hmax[q] = __hmax2(hmax[q], __habs2(h[e]));
                }
            } else {
                const float4* sp = (tag != kPUncached) ? reinterpret_cast<const float4*>(s_cache + (tag - 1) * 8)
                                                       : reinterpret_cast<const float4*>(s + k0 + i * kPCols + cw * 8);
                const float4 s0 = sp[0], s1 = sp[1];
                const float sv[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
                // Only the columns with a divisor (the same for every lane: lanes are rows) take
                // the fp32 division and maximum and are written back as fp16(x~); the others go
                // through the half-precision maximum like an untagged unit, with the divided
                // columns blanked out of that maximum.
                uint32_t wd[4][4], zd[4][4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    wd[q][0] = v[q].x; wd[q][1] = v[q].y; wd[q][2] = v[q].z; wd[q][3] = v[q].w;
#pragma unroll
                    for (int i = 0; i < 4; ++i) zd[q][i] = wd[q][i];
                }
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    if (sv[e] != 1.f) {
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const uint32_t word = wd[q][e >> 1];
                            const __half hv = __ushort_as_half((unsigned short)((e & 1) ? (word >> 16) : (word & 0xffffu)));
                            const float f = __fdiv_rn(__half2float(hv), sv[e]);
                            amax[q] = fmaxf(amax[q], fabsf(f));
                            const uint32_t hb = (uint32_t)__half_as_ushort(__float2half_rn(f));
                            wd[q][e >> 1] = (e & 1) ? ((word & 0x0000ffffu) | (hb << 16)) : ((word & 0xffff0000u) | hb);
                            zd[q][e >> 1] &= (e & 1) ? 0x0000ffffu : 0xffff0000u;
                        }
                    }
                }
#pragma unroll
                for (int q = 0; q < 4; ++q) {
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        hmax[q] = __hmax2(hmax[q], __habs2(*reinterpret_cast<const __half2*>(&zd[q][i])));
                    pj_sts128(addr[q], make_uint4(wd[q][0], wd[q][1], wd[q][2], wd[q][3]));
                }
                fence_proxy_async_smem();       // the MMA reads these through the async proxy
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_ready(st));
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const float a = fmaxf(amax[q], fmaxf(__low2float(hmax[q]), __high2float(hmax[q])));
            amax_w[cw * kPTok + lane + 32 * q] = a;
        }
        named_bar_sync(1, kPConsumerWarps * 32);
        if (tid - 64 < kPTok) {
            const int row = tid - 64;
            float a = amax_w[row];
#pragma unroll
            for (int w = 1; w < kPConsumerWarps; ++w) a = fmaxf(a, amax_w[w * kPTok + row]);
            if (*abort_flag) a = __int_as_float(0x7fc00000);
            if (row0 + row < Mc) amax_part[(size_t)ks * Mc + row0 + row] = a;
        }
        // ---- partial T: tensor memory -> shared memory as [token][128 rows of the group] -> one
        // bulk copy per group into the scratch, where a group's tile is contiguous.  A warp
        // reaches the 32 lanes (rows j of a group) of its quarter, warp % 4; the two warps of a
        // quarter take 64 tokens each.  The ring is idle by now (every MMA has completed) and
        // serves as two 64 KB staging buffers. ----
        if (r > 0) {
            if (ok) ok = pj_warp_wait(bar_acc, 0u, abort_flag, lane);
            tc_fence_after();
            const int q = warp & 3, half = cw >> 2;
            const int rows_valid = (Mc - row0 < kPTok) ? (Mc - row0) : kPTok;
            for (int g = 0; g < groups; ++g) {
                const uint32_t buf = sb + (uint32_t)(g & 1) * 65536u;
                if (g >= 2) {               // the copy that last read this buffer must be done with it
                    if (tid == 64) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                    named_bar_sync(1, kPConsumerWarps * 32);
                }
#pragma unroll 1
                for (int c0 = half * 64; c0 < half * 64 + 64; c0 += 16) {
                    uint32_t v[16];
                    tmem_ld16(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(g * 128 + c0), v);
                    tmem_wait_ld(v);
#pragma unroll
                    for (int e = 0; e < 16; ++e)
                        asm volatile("st.shared.b32 [%0], %1;" ::"r"(buf + (uint32_t)(c0 + e) * 512u + (uint32_t)(q * 32 + lane) * 4u), "r"(v[e]) : "memory");
                }
                fence_proxy_async_smem();
                named_bar_sync(1, kPConsumerWarps * 32);
                if (tid == 64 && !*abort_flag) {
                    float* dst = t_part + (((size_t)ks * groups + g) * Mc + row0) * 128;
                    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                                 ::"l"(dst), "r"(buf), "r"((uint32_t)rows_valid * 512u) : "memory");
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                }
            }
            if (tid == 64) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
            tc_fence_before();
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1 && r > 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(tmem_cols) : "memory");
    }
}

// Eight codes of a row whose divisors are all 1: fp16 pairs widened by the conversion unit, then on
// packed fp32 pairs su = x * (1 / sc) + 1.5 * 2^23 (one rounding: the low byte of su is the code),
// -w = 1.5 * 2^23 - su (exact) and d = x * (1 / sc) - w, the distance of the product to its integer.
// rne(x / sc) can differ from that integer only where the product is within 1e-4 of a tie (the
// quotient and the product differ by less than 3.1e-5): such a group takes the exact division.
__device__ __forceinline__ uint2 codes8_unit(const uint4& x, float sc, float rcp, float qmax) {
    const float kMagic = 12582912.0f;
    const float2 m2 = make_float2(kMagic, kMagic), neg1 = make_float2(-1.f, -1.f), r2 = make_float2(rcp, rcp);
    const uint32_t xw[4] = {x.x, x.y, x.z, x.w};
    float2 f[4];
    uint32_t u[8];
    float far = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[i] = __half22float2(*reinterpret_cast<const __half2*>(&xw[i]));
        const float2 su = __ffma2_rn(f[i], r2, m2);
        const float2 nw = __ffma2_rn(su, neg1, m2);
        const float2 d = __ffma2_rn(f[i], r2, nw);
        u[2 * i] = __float_as_uint(su.x);
        u[2 * i + 1] = __float_as_uint(su.y);
        far = fmaxf(far, fmaxf(fabsf(d.x), fabsf(d.y)));
    }
    if (far > 0.4999f)
        return quant8_exact(f[0].x, f[0].y, f[1].x, f[1].y, f[2].x, f[2].y, f[3].x, f[3].y, sc, qmax);
    const uint32_t a01 = __byte_perm(u[0], u[1], 0x0040), a23 = __byte_perm(u[2], u[3], 0x0040);
    const uint32_t a45 = __byte_perm(u[4], u[5], 0x0040), a67 = __byte_perm(u[6], u[7], 0x0040);
    return make_uint2(__byte_perm(a01, a23, 0x5410), __byte_perm(a45, a67, 0x5410));
}

// grid = ceil(rows of the chunk / kQRows), 256 threads; a CTA takes kQRows token rows, several
// 16-byte loads per thread are in flight, and the per-row scales are computed once per CTA (one
// warp per row).  The kernel is bound by instruction issue, not by bytes, so the common case is
// kept free of per-column work: the CTA first lists the columns whose divisor is not 1 (the few
// outlier channels); the main loop then treats every column as undivided, and the listed columns
// are redone afterwards, one (row, column) per thread, with both IEEE divisions.  A smoothing
// vector with more such columns than the list holds takes the general loop, which tests every
// group of eight divisors.
// Launched as a programmatic dependent of act_proj_kernel: the list and the first loads of X
// (inputs of the whole step, not products of that kernel) are done before the dependency wait.
constexpr int kQRows = 4;
constexpr int kQList = 512;             // columns with a divisor the fix-up pass can take
__global__ void __launch_bounds__(256, 4)
act_quant_kernel(const __half* __restrict__ X, const float* __restrict__ s, int m_first, int Mc, int K,
                 int r, int KS, const float* amax_part, const float* t_part,
                 int8_t* __restrict__ Xq, float* __restrict__ a_scale, __nv_bfloat16* __restrict__ T,
                 int ldt, int lo_off, float qmax) {
    __shared__ float sc_sm[kQRows], rcp_sm[kQRows];
    __shared__ int n_list;
    __shared__ int list_col[kQList];
    grid_dep_launch();      // a dependent linear kernel may start streaming its weights
    const int row0 = blockIdx.x * kQRows;
    const int nrows = (Mc - row0 < kQRows) ? (Mc - row0) : kQRows;
    const int chunks = K / 8;
    const int groups = (r + 127) / 128;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const __half* xbase = X + (size_t)(m_first + row0) * K;
    uint4 x[kQRows];
    int c = threadIdx.x;
    auto load_x = [&](int cc) {
#pragma unroll
        for (int rr = 0; rr < kQRows; ++rr)
            x[rr] = (rr < nrows && cc < chunks) ? *reinterpret_cast<const uint4*>(xbase + (size_t)rr * K + cc * 8)
                                                : make_uint4(0, 0, 0, 0);
    };
    load_x(c);
    // ---- columns with a divisor (any order; entries past the capacity are only counted) ----
    if (threadIdx.x == 0) n_list = 0;
    __syncthreads();
    if (s) {
        for (int g = threadIdx.x; g < K / 4; g += 256) {
            const float4 v = __ldg(reinterpret_cast<const float4*>(s) + g);
            const float sv[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                if (sv[e] != 1.f) {
                    const int at = atomicAdd(&n_list, 1);
                    if (at < kQList) list_col[at] = g * 4 + e;
                }
            }
        }
    }
    grid_dep_wait();        // the partial maxima and the partial T come from act_proj_kernel
    // ---- scales: warp w takes row w ----
    if (warp < nrows) {
        float v = (lane < KS) ? amax_part[(size_t)lane * Mc + row0 + warp] : 0.f;
        for (int ks = lane + 32; ks < KS; ks += 32) {
            const float u = amax_part[(size_t)ks * Mc + row0 + warp];
            v = (u != u || v != v) ? __int_as_float(0x7fc00000) : fmaxf(v, u);
        }
        const bool bad = __any_sync(0xffffffffu, v != v);
        float a = warp_max(v);
        if (bad) a = __int_as_float(0x7fc00000);
        if (lane == 0) {
            const float sc = __fdiv_rn(a, qmax);
            sc_sm[warp] = sc;
            rcp_sm[warp] = (sc > 0.f) ? __frcp_rn(sc) : 0.f;
            a_scale[m_first + row0 + warp] = sc;
        }
    } else if (warp < kQRows && lane == 0) {
        sc_sm[warp] = 0.f;
        rcp_sm[warp] = 0.f;
    }
    // ---- T of these rows: the slices' partials summed in slice order ----
    for (int e = threadIdx.x; e < nrows * r; e += 256) {
        const int rr = e / r, j = e - rr * r;
        const float* tp = t_part + ((size_t)(j >> 7) * Mc + row0 + rr) * 128 + (j & 127);
        const size_t slice = (size_t)groups * Mc * 128;
        float t = 0.f;
        int ks = 0;
        for (; ks + 4 <= KS; ks += 4) {         // four loads in flight, summed in slice order
            const float a0 = tp[ks * slice], a1 = tp[(ks + 1) * slice];
            const float a2 = tp[(ks + 2) * slice], a3 = tp[(ks + 3) * slice];
            t += a0; t += a1; t += a2; t += a3;
        }
        for (; ks < KS; ++ks) t += tp[ks * slice];
        store_t(T + (size_t)(m_first + row0 + rr) * ldt, j, t, lo_off);
    }
    __syncthreads();
    const int listed = n_list;
    float scr[kQRows], rc1[kQRows];
#pragma unroll
    for (int rr = 0; rr < kQRows; ++rr) {
        scr[rr] = sc_sm[rr];
        rc1[rr] = rcp_sm[rr];
    }
    if (listed <= kQList) {
        // ---- codes, every column taken as undivided ----
        for (; c < chunks; c += 256) {
            uint2 q[kQRows];
#pragma unroll
            for (int rr = 0; rr < kQRows; ++rr) {
                q[rr] = codes8_unit(x[rr], scr[rr], rc1[rr], qmax);
                if (!(scr[rr] > 0.f)) q[rr] = make_uint2(0u, 0u);      // zero row, or a poisoned scale
            }
            load_x(c + 256);        // the next iteration's loads are in flight during the stores
#pragma unroll
            for (int rr = 0; rr < kQRows; ++rr)
                if (rr < nrows) *reinterpret_cast<uint2*>(Xq + (size_t)(m_first + row0 + rr) * K + c * 8) = q[rr];
        }
        // ---- the listed columns again, with their divisors ----
        __syncthreads();            // orders the stores above before the single bytes below
        for (int e = threadIdx.x; e < listed * kQRows; e += 256) {
            const int rr = e & (kQRows - 1), col = list_col[e / kQRows];
            if (rr >= nrows) continue;
            const float sc = sc_sm[rr];
            int code = 0;
            if (sc > 0.f) {
                const float xt = __fdiv_rn(__half2float(xbase[(size_t)rr * K + col]), __ldg(s + col));
                code = rne_clamp(__fdiv_rn(xt, sc), -qmax, qmax);
            }
            Xq[(size_t)(m_first + row0 + rr) * K + col] = (int8_t)code;
        }
        return;
    }
    // ---- general loop: many columns have a divisor ----
    for (; c < chunks; c += 256) {
        const float4 s0 = __ldg(reinterpret_cast<const float4*>(s + c * 8));
        const float4 s1 = __ldg(reinterpret_cast<const float4*>(s + c * 8) + 1);
        const float sv[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
        uint2 q[kQRows];
#pragma unroll
        for (int rr = 0; rr < kQRows; ++rr) {
            const __half* h = reinterpret_cast<const __half*>(&x[rr]);
            float f[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {       // x~ = x / s, IEEE division, only where the divisor is not 1
                f[e] = __half2float(h[e]);
                if (sv[e] != 1.f) f[e] = __fdiv_rn(f[e], sv[e]);
            }
            q[rr] = (scr[rr] > 0.f) ? quant8_pairs(f, scr[rr], rc1[rr], qmax) : make_uint2(0u, 0u);
        }
        load_x(c + 256);
#pragma unroll
        for (int rr = 0; rr < kQRows; ++rr)
            if (rr < nrows) *reinterpret_cast<uint2*>(Xq + (size_t)(m_first + row0 + rr) * K + c * 8) = q[rr];
    }
}

struct ProjPlan {
    int Mc;         // tokens per chunk (a multiple of 128 unless it is all of M)
    int KS;         // slices of K
};

// Slice count: as many slices of K as keep the grid within one wave (a slice has at least four
// 64-column stages).  The whole input is one chunk: splitting long inputs into chunks of tokens
// whose X stays in L2 for the second kernel cost more in fixed time per launch pair than the L2
// hits saved (4096 x 14336 at rank 128: 140 us in three chunks, 95 us in one; 8192 x 8192: 140
// against 107 us), so the chunk loop below runs once.
ProjPlan proj_plan(int M, int K, int num_sms) {
    const int blocks = K / kPCols;
    const int tiles = (M + kPTok - 1) / kPTok;
    int ks_best = 1;
    for (int ks = 1; ks <= blocks / 4 && tiles * ks <= num_sms; ++ks)
        if (blocks % ks == 0) ks_best = ks;
    return ProjPlan{M, ks_best};
}

// Floats of the row-maxima part of the scratch, padded so that the partial T behind it starts on
// a 128-byte boundary (it is written by bulk copies, which need 16-byte alignment).
size_t proj_amax_floats(const ProjPlan& p) { return ((size_t)p.KS * p.Mc + 31) & ~(size_t)31; }

size_t proj_scratch_bytes(int M, int K, int r, int num_sms) {
    const ProjPlan p = proj_plan(M, K, num_sms);
    const int groups = (r + 127) / 128;
    return (proj_amax_floats(p) + (size_t)p.KS * p.Mc * groups * 128) * sizeof(float);
}

}  // namespace

size_t quant_act_ws_scratch_bytes(int M, int K, int r) {
    if (M <= 32) return 0;
    return proj_scratch_bytes(M, K, r, kProjPlanSms);
}

int quant_act_ws_launches(int M, int K) {
    if (M <= 32) return 1;
    const ProjPlan plan = proj_plan(M, K, kProjPlanSms);
    return 2 * ((M + plan.Mc - 1) / plan.Mc);
}

int launch_quant_act_ws(const __half* X, const float* s, const __half* LA, int M, int K, int r,
                        int8_t* Xq, float* a_scale, __nv_bfloat16* T, void* scratch, size_t scratch_bytes,
                        cudaStream_t st, int act_bits, bool t_pair) {
    const float qmax = (float)((1 << (act_bits - 1)) - 1);
    const int ldt = t_pair ? 2 * r : r, lo_off = t_pair ? r : 0;
    const int groups = (r + 127) / 128;
    if (groups > kPMaxGroups) return record_error(ASER_ERR_SHAPE, "quant_act: r beyond 512");
    const ProjPlan plan = proj_plan(M, K, kProjPlanSms);
    if (scratch == nullptr || misaligned16(scratch) ||
        scratch_bytes < (proj_amax_floats(plan) + (size_t)plan.KS * plan.Mc * groups * 128) * sizeof(float))
        return record_error(ASER_ERR_WORKSPACE, "quant_act: scratch missing or too small");
    float* amax_part = static_cast<float*>(scratch);
    float* t_part = amax_part + proj_amax_floats(plan);
    const int Kc = K / plan.KS;
    const int NS = proj_stages(groups);
    // the ring (at least 128 KB with a projection: it later stages the partial T) and the tail
    const size_t smem = (size_t)NS * kPTileBytes * (1 + groups) + 256 + ((Kc / 8 + 15) & ~15) +
                        kPConsumerWarps * kPTok * sizeof(float) + kPCacheUnits * 8 * sizeof(float) + 1024;
    static size_t configured[kMaxDevices] = {0};
    int dev = 0;
    {
        const int rc = current_device(&dev);
        if (rc != ASER_OK) return rc;
    }
    if (smem > configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(act_proj_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return record_cuda_error(e, "act_proj smem attribute");
        configured[dev] = smem;
    }
    CUtensorMap mx, mla;
    int rc = encode_map_blocks(&mx, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, X, M, K, kPTok, 1);
    if (rc != ASER_OK) return rc;
    if (r > 0) {
        rc = encode_map_blocks(&mla, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, LA, r, K, r <= 256 ? r : r / 2, 1);
        if (rc != ASER_OK) return rc;
    } else {
        mla = mx;
    }
    for (int m_first = 0; m_first < M; m_first += plan.Mc) {
        const int Mc = (M - m_first < plan.Mc) ? (M - m_first) : plan.Mc;
        const int tiles = (Mc + kPTok - 1) / kPTok;
        act_proj_kernel<<<dim3(plan.KS, tiles, 1), kPThreads, smem, st>>>(mx, mla, s, m_first, Mc, K, Kc, r,
                                                                          amax_part, t_part);
        rc = check_launch("act_proj_kernel");
        if (rc != ASER_OK) return rc;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((Mc + kQRows - 1) / kQRows, 1, 1);
        cfg.blockDim = dim3(256, 1, 1);
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        cudaError_t e = cudaLaunchKernelEx(&cfg, act_quant_kernel, X, s, m_first, Mc, K, r, plan.KS,
                                           (const float*)amax_part, (const float*)t_part, Xq, a_scale, T, ldt,
                                           lo_off, qmax);
        if (e != cudaSuccess) return record_cuda_error(e, "act_quant_kernel");
    }
    return ASER_OK;
}

}  // namespace aser
