// Arithmetic shared by the activation kernels: the smoothing divide, the int8 codes and the
// storage of T (Sec. 4.2 smoothing, Sec. 5.1 per-token round-to-nearest, Sec. 4.1 projection).
#pragma once
#include "aser_common.cuh"

namespace aser {

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

// T element(s) -> memory.  `lo_off` == 0: T[j] = bf16(t).  Otherwise T is stored as a PAIR of
// bf16 numbers, T[j] = bf16(t) and T[j + lo_off] = bf16(t - T[j]), whose sum carries 16
// significant bits; a linear kernel given the up projection twice, [L_B | L_B], then adds both.
__device__ __forceinline__ void store_t(__nv_bfloat16* row, int j, float t, int lo_off) {
    const __nv_bfloat16 hi = __float2bfloat16_rn(t);
    row[j] = hi;
    if (lo_off) row[j + lo_off] = __float2bfloat16_rn(t - __bfloat162float(hi));
}
__device__ __forceinline__ void store_t2(__nv_bfloat16* row, int j, float t0, float t1, int lo_off) {
    const __nv_bfloat162 hi = __floats2bfloat162_rn(t0, t1);
    *reinterpret_cast<__nv_bfloat162*>(row + j) = hi;
    if (lo_off)
        *reinterpret_cast<__nv_bfloat162*>(row + j + lo_off) =
            __floats2bfloat162_rn(t0 - __low2float(hi), t1 - __high2float(hi));
}

// Exact codes for eight values (the definition: IEEE quotient, round half to even, clamp).
static __device__ __noinline__ uint2 quant8_exact(float v0, float v1, float v2, float v3, float v4, float v5,
                                           float v6, float v7, float sc, float qmax) {
    const float v[8] = {v0, v1, v2, v3, v4, v5, v6, v7};
    uint32_t w[2] = {0, 0};
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int q = rne_clamp(__fdiv_rn(v[i], sc), -qmax, qmax);
        w[i >> 2] |= (uint32_t)(q & 0xFF) << (8 * (i & 3));
    }
    return make_uint2(w[0], w[1]);
}
// Same codes as quant8 for sc > 0, on packed fp32 pairs: t = x~ * (1 / sc), rounded by adding
// 1.5 * 2^23 (the low byte of the sum is the code); the distance of t to that integer tells the
// near-ties, and a group with one takes the exact path as a whole.
__device__ __forceinline__ uint2 quant8_pairs(const float (&v)[8], float sc, float rcp, float qmax) {
    const float kMagic = 12582912.0f;
    const float2 r2 = make_float2(rcp, rcp), m2 = make_float2(kMagic, kMagic);
    const float2 nm2 = make_float2(-kMagic, -kMagic), neg1 = make_float2(-1.f, -1.f);
    uint32_t q[8];
    float far = 0.f;        // largest distance of a product to its rounded integer (branch-free)
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 t = __fmul2_rn(make_float2(v[2 * i], v[2 * i + 1]), r2);
        const float2 u = __fadd2_rn(t, m2);
        const float2 w = __fadd2_rn(u, nm2);            // the rounded integer
        const float2 d = __ffma2_rn(w, neg1, t);        // t - w, exact
        q[2 * i] = __float_as_uint(u.x);
        q[2 * i + 1] = __float_as_uint(u.y);
        far = fmaxf(far, fmaxf(fabsf(d.x), fabsf(d.y)));
    }
    if (far > 0.4999f) return quant8_exact(v[0], v[1], v[2], v[3], v[4], v[5], v[6], v[7], sc, qmax);
    const uint32_t a01 = __byte_perm(q[0], q[1], 0x0040), a23 = __byte_perm(q[2], q[3], 0x0040);
    const uint32_t a45 = __byte_perm(q[4], q[5], 0x0040), a67 = __byte_perm(q[6], q[7], 0x0040);
    return make_uint2(__byte_perm(a01, a23, 0x5410), __byte_perm(a45, a67, 0x5410));
}

}  // namespace aser
