/*
 * CPU oracle for the forward pass of an ASER-quantized linear layer
 * (Activation Smoothing + Error Reconstruction, arXiv 2411.07762).
 *
 * THIS IS TEST INFRASTRUCTURE.  It is a deliberately plain, slow restatement of
 * what the method computes, one loop per definition, so that it can be checked
 * against the paper by eye.  It shares no code with the CUDA library and is
 * only ever called from the test-suite, the smoke check and the benchmark's
 * CPU-baseline leg.
 *
 * Naming: the library is token-major.  X is [M tokens, K], W is [N, K],
 * Y = X W^T is [M, N].  `s` is the diagonal of the paper's smoothing matrix M
 * (Sec. 4.2).  L_A is the rank-r DOWN projection [r, K] (the paper's
 * V_r^T S^-1) and L_B the UP projection [N, r] (the paper's U_r Sigma_r); the
 * paper uses the two letters the other way round (Sec. 4.1, text below Eq. 8).
 *
 * Arithmetic conventions (the paper only says "RTN", "per-channel weights",
 * "per-token activations", Sec. 5.1; everything finer is this build's reading):
 *   - smoothing, scales and rounding are single IEEE fp32 operations
 *     (one multiply or one divide, round-to-nearest-even, no fused
 *     multiply-add, no reciprocal);
 *   - rounding to integer codes is round-half-to-even;
 *   - the integer product is exact;
 *   - dequantisation and the low-rank branch are evaluated in fp64.
 *
 * Build: gcc -O2 -ffp-contract=off -fno-fast-math -fopenmp -shared -fPIC
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static int g_threads = 1;

/* Number of OpenMP threads used for the row loops (1 = plain serial loops). */
void aser_oracle_set_threads(int n) { g_threads = n < 1 ? 1 : n; }
int aser_oracle_get_threads(void) { return g_threads; }
int aser_oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* IEEE binary16 -> binary32, exact. */
static float f16_to_f32(uint16_t h)
{
    uint32_t sign = (uint32_t)(h & 0x8000u) << 16;
    uint32_t exp = (h >> 10) & 0x1Fu;
    uint32_t man = h & 0x3FFu;
    union { uint32_t u; float f; } v;
    if (exp == 0) {
        /* zero or subnormal: man * 2^-24 */
        float m = (float)man * (1.0f / 16777216.0f);
        v.f = m;
        v.u |= sign;
        return v.f;
    }
    if (exp == 31) {
        v.u = sign | 0x7F800000u | (man << 13);
        return v.f;
    }
    v.u = sign | ((exp + 112u) << 23) | (man << 13);
    return v.f;
}

/* ---------------------------------------------------------------------------
 * Activation smoothing (Sec. 4.2, Eq. 10: W X = (W M)(M^-1 X)).
 * x~[m,k] = fp32(X[m,k]) / s[k], one fp32 division.  s == NULL means all ones.
 * ------------------------------------------------------------------------- */
void aser_oracle_smooth_act(const uint16_t* X, const float* s, long M, long K, float* xs)
{
#pragma omp parallel for num_threads(g_threads) schedule(static)
    for (long m = 0; m < M; ++m)
        for (long k = 0; k < K; ++k) {
            float x = f16_to_f32(X[m * K + k]);
            xs[m * K + k] = s ? x / s[k] : x;
        }
}

/* ---------------------------------------------------------------------------
 * Per-token symmetric round-to-nearest of the activations to `bits`-bit codes
 * (Sec. 5.1 "per-token for activations"; 8 bits in the W4A8 setting, 6 in the
 * W4A6 setting of Sec. 5.2).  qmax = 2^(bits-1) - 1; a_scale[m] = max_k |x~| / qmax;
 * code = rne(x~ / a_scale) clamped to [-qmax, qmax], stored in an int8.  An
 * all-zero token gets scale 0 and codes 0.
 * ------------------------------------------------------------------------- */
void aser_oracle_quant_act_bits(const float* xs, long M, long K, int bits, int8_t* Xq, float* a_scale)
{
    const float qmax = (float)((1 << (bits - 1)) - 1);
#pragma omp parallel for num_threads(g_threads) schedule(static)
    for (long m = 0; m < M; ++m) {
        float amax = 0.0f;
        for (long k = 0; k < K; ++k) {
            float a = fabsf(xs[m * K + k]);
            if (a > amax) amax = a;
        }
        float sc = amax / qmax;
        a_scale[m] = sc;
        for (long k = 0; k < K; ++k) {
            float c = 0.0f;
            if (amax > 0.0f) {
                c = rintf(xs[m * K + k] / sc);
                if (c > qmax) c = qmax;
                if (c < -qmax) c = -qmax;
            }
            Xq[m * K + k] = (int8_t)c;
        }
    }
}

/* The W4A8 setting: 8-bit codes, a_scale[m] = max_k |x~| / 127, codes in [-127, 127]. */
void aser_oracle_quant_act(const float* xs, long M, long K, int8_t* Xq, float* a_scale)
{
    aser_oracle_quant_act_bits(xs, M, K, 8, Xq, a_scale);
}

/* ---------------------------------------------------------------------------
 * Per-output-channel symmetric int4 round-to-nearest of the smoothed weight
 * W diag(s) (Sec. 4.2 Eq. 10 and Eq. 12, Q(W_s); Sec. 5.1 "per-channel for
 * weights").  ws = fp32(W) * s (one fp32 multiply); w_scale[n] = max_k|ws|/7;
 * code = rne(ws / w_scale) clamped to [-8, 7].  A zero row: scale 0, codes 0.
 * `ws_out` (optional) receives the smoothed fp32 weights.
 * ------------------------------------------------------------------------- */
void aser_oracle_quant_w4(const uint16_t* W, const float* s, long N, long K,
                          int8_t* q, float* w_scale, float* ws_out)
{
#pragma omp parallel for num_threads(g_threads) schedule(static)
    for (long n = 0; n < N; ++n) {
        float amax = 0.0f;
        for (long k = 0; k < K; ++k) {
            float w = f16_to_f32(W[n * K + k]);
            float v = s ? w * s[k] : w;
            if (ws_out) ws_out[n * K + k] = v;
            float a = fabsf(v);
            if (a > amax) amax = a;
        }
        float sc = amax / 7.0f;
        w_scale[n] = sc;
        for (long k = 0; k < K; ++k) {
            float c = 0.0f;
            if (amax > 0.0f) {
                float w = f16_to_f32(W[n * K + k]);
                float v = s ? w * s[k] : w;
                c = rintf(v / sc);
                if (c > 7.0f) c = 7.0f;
                if (c < -8.0f) c = -8.0f;
            }
            q[n * K + k] = (int8_t)c;
        }
    }
}

/* Canonical nibble packing: byte j of row n = (q[n,2j] & 0xF) | (q[n,2j+1] << 4). */
void aser_oracle_pack_w4(const int8_t* q, long N, long K, uint8_t* packed)
{
    for (long n = 0; n < N; ++n)
        for (long j = 0; j < K / 2; ++j) {
            uint8_t lo = (uint8_t)q[n * K + 2 * j] & 0xFu;
            uint8_t hi = (uint8_t)q[n * K + 2 * j + 1] & 0xFu;
            packed[n * (K / 2) + j] = (uint8_t)(lo | (hi << 4));
        }
}

void aser_oracle_unpack_w4(const uint8_t* packed, long N, long K, int8_t* q)
{
    for (long n = 0; n < N; ++n)
        for (long j = 0; j < K / 2; ++j) {
            uint8_t b = packed[n * (K / 2) + j];
            int lo = b & 0xF, hi = b >> 4;
            q[n * K + 2 * j] = (int8_t)(lo >= 8 ? lo - 16 : lo);
            q[n * K + 2 * j + 1] = (int8_t)(hi >= 8 ? hi - 16 : hi);
        }
}

/* ---------------------------------------------------------------------------
 * Integer product of the quantized operands, the W_q X term of the inference
 * pass (Sec. 4.2, last paragraph): acc[m,n] = sum_k Xq[m,k] * q[n,k], exact
 * in int32.  `rows` (optional, n_rows entries) restricts m to a subset; the
 * output then has n_rows rows in that order.
 * ------------------------------------------------------------------------- */
void aser_oracle_int_matmul(const int8_t* Xq, const int8_t* q, long M, long N, long K,
                            const long* rows, long n_rows, int32_t* acc)
{
    long R = rows ? n_rows : M;
#pragma omp parallel for num_threads(g_threads) schedule(static)
    for (long i = 0; i < R; ++i) {
        long m = rows ? rows[i] : i;
        for (long n = 0; n < N; ++n) {
            int32_t sum = 0;
            for (long k = 0; k < K; ++k)
                sum += (int32_t)Xq[m * K + k] * (int32_t)q[n * K + k];
            acc[i * N + n] = sum;
        }
    }
}

/* ---------------------------------------------------------------------------
 * Down projection of the error-reconstruction branch (the paper's L_B X with
 * its L_B = V_r^T S^-1, Sec. 4.1): T[m,j] = sum_k L_A[j,k] * x~[m,k] in fp64,
 * fed by the smoothed full-precision activation.
 * ------------------------------------------------------------------------- */
void aser_oracle_down_proj(const float* xs, const uint16_t* LA, long M, long K, long r,
                           const long* rows, long n_rows, double* T)
{
    long R = rows ? n_rows : M;
#pragma omp parallel for num_threads(g_threads) schedule(static)
    for (long i = 0; i < R; ++i) {
        long m = rows ? rows[i] : i;
        for (long j = 0; j < r; ++j) {
            double sum = 0.0;
            for (long k = 0; k < K; ++k)
                sum += (double)f16_to_f32(LA[j * K + k]) * (double)xs[m * K + k];
            T[i * r + j] = sum;
        }
    }
}

/* ---------------------------------------------------------------------------
 * Dequantisation plus up projection (W_q X + L_A L_B X in the paper's letters,
 * Sec. 4.2): y[i,n] = acc[i,n] * a_scale[m_i] * w_scale[n] + sum_j L_B[n,j] T[i,j],
 * all in fp64.  acc and T hold only the selected rows (see above); a_scale is
 * indexed by the original row number.  r == 0 leaves the plain W4A8 product.
 * ------------------------------------------------------------------------- */
void aser_oracle_dequant_add(const int32_t* acc, const float* a_scale, const float* w_scale,
                             const double* T, const uint16_t* LB, long M, long N, long r,
                             const long* rows, long n_rows, double* y)
{
    long R = rows ? n_rows : M;
#pragma omp parallel for num_threads(g_threads) schedule(static)
    for (long i = 0; i < R; ++i) {
        long m = rows ? rows[i] : i;
        for (long n = 0; n < N; ++n) {
            double v = (double)acc[i * N + n] * (double)a_scale[m] * (double)w_scale[n];
            double lr = 0.0;
            for (long j = 0; j < r; ++j)
                lr += (double)f16_to_f32(LB[n * r + j]) * T[i * r + j];
            y[i * N + n] = v + lr;
        }
    }
}
