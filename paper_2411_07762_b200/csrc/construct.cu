// Device-side construction of the error-reconstruction factors of one layer (Algorithm 1 body;
// Sec. 4.1 Eq. 5-6 and the factor split below Eq. 8; Sec. 4.2 Eq. 10 for the smoothed operands):
//   E   = W diag(s) - dequant(Q4(W diag(s)))                     [N, K]
//   G   = X~^T X~ + lambda I,  X~ = X_cal diag(s)^-1,  lambda = damping * trace / K   (the paper's X X^T)
//   S   = lower Cholesky factor of G                              (whitening, Eq. 5)
//   A   = E S,  A ~ U_r Sigma_r V_r^T                             (truncated SVD, Eq. 6)
//   L_B = U_r Sigma_r  [N, r],   L_A = V_r^T S^-1  [r, K]
// All in fp64 on CUDA cores (an offline step: a few hundred GFLOP at the largest shapes).
//
// The top-r singular triplets come from subspace iteration on A^T A with p = r + oversampling
// vectors kept as ROWS (Qt [p, K]): Yt = Qt A^T, Zt = Yt A, Qt = orthonormalised Zt (Cholesky of
// Zt Zt^T and a forward substitution, done twice), then Rayleigh-Ritz by one-sided Jacobi
// rotations applied to the rows of Bt = Qt A^T and of Qt together: when the rows of Bt are
// orthogonal their norms are the singular values, the r longest rows of Bt are (U_r Sigma_r)^T
// and the matching rows of Qt are V_r^T.  The whitened spectrum of a quantization error decays,
// so a few dozen iterations reach the singular subspace to near machine precision.
#include "aser_common.cuh"

namespace aser {

namespace {

// ---------------------------------------------------------------------------
// C[i,j] = beta * C[i,j] + alpha * sum_k A(i,k) B(k,j), all fp64, element (i,k) of A at
// A[i * ai + k * ak] (so a transposed operand is a pair of swapped strides), C row-major with
// leading dimension ldc.  64 x 64 x 16 tiles, 256 threads, 4 x 4 results per thread.
// ---------------------------------------------------------------------------
constexpr int kGT = 64, kGK = 16;

__global__ void __launch_bounds__(256)
dgemm_kernel(int m, int n, int k, double alpha, const double* __restrict__ A, long long ai, long long ak,
             const double* __restrict__ B, long long bk, long long bj, double beta, double* __restrict__ C,
             long long ldc) {
    __shared__ double As[kGK][kGT + 1];
    __shared__ double Bs[kGK][kGT + 1];
    const int tid = threadIdx.x;
    const int i0 = blockIdx.y * kGT, j0 = blockIdx.x * kGT;
    const int ti = (tid / 16) * 4, tj = (tid % 16) * 4;
    double acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = 0.0;
    for (int k0 = 0; k0 < k; k0 += kGK) {
#pragma unroll
        for (int l = 0; l < 4; ++l) {
            const int t = tid + l * 256;
            int ii, kk;
            if (ak == 1) { kk = t % kGK; ii = t / kGK; } else { ii = t % kGT; kk = t / kGT; }
            As[kk][ii] = (i0 + ii < m && k0 + kk < k) ? A[(long long)(i0 + ii) * ai + (long long)(k0 + kk) * ak] : 0.0;
            int jj, kb;
            if (bj == 1) { jj = t % kGT; kb = t / kGT; } else { kb = t % kGK; jj = t / kGK; }
            Bs[kb][jj] = (j0 + jj < n && k0 + kb < k) ? B[(long long)(k0 + kb) * bk + (long long)(j0 + jj) * bj] : 0.0;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < kGK; ++kk) {
            double a[4], b[4];
#pragma unroll
            for (int x = 0; x < 4; ++x) { a[x] = As[kk][ti + x]; b[x] = Bs[kk][tj + x]; }
#pragma unroll
            for (int x = 0; x < 4; ++x)
#pragma unroll
                for (int y = 0; y < 4; ++y) acc[x][y] = fma(a[x], b[y], acc[x][y]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int x = 0; x < 4; ++x)
#pragma unroll
        for (int y = 0; y < 4; ++y) {
            const int i = i0 + ti + x, j = j0 + tj + y;
            if (i < m && j < n) {
                double* c = C + (long long)i * ldc + j;
                *c = (beta == 0.0 ? 0.0 : beta * *c) + alpha * acc[x][y];
            }
        }
}

int dgemm(cudaStream_t st, int m, int n, int k, double alpha, const double* A, long long ai, long long ak,
          const double* B, long long bk, long long bj, double beta, double* C, long long ldc) {
    if (m <= 0 || n <= 0) return ASER_OK;
    dim3 grid((n + kGT - 1) / kGT, (m + kGT - 1) / kGT);
    dgemm_kernel<<<grid, 256, 0, st>>>(m, n, k, alpha, A, ai, ak, B, bk, bj, beta, C, ldc);
    return check_launch("dgemm_kernel");
}

// ---------------------------------------------------------------------------
// Cholesky, lower, in place, blocked by 64 columns: factor the diagonal block (one CTA), solve
// the panel below it row by row against that block, update the trailing matrix with a GEMM.
// A non-positive pivot sets *fail (the factor is then unusable).
// ---------------------------------------------------------------------------
constexpr int kCB = 64;

__global__ void __launch_bounds__(kCB)
potrf_diag_kernel(double* __restrict__ A, long long lda, int nb, int* __restrict__ fail) {
    __shared__ double T[kCB][kCB + 1];
    const int t = threadIdx.x;
    for (int i = 0; i < nb; ++i) T[i][t] = (t < nb) ? A[(long long)i * lda + t] : 0.0;
    __syncthreads();
    for (int j = 0; j < nb; ++j) {
        if (t == j) {
            double d = T[j][j];
            if (!(d > 0.0)) { *fail = 1; d = 1.0; }
            T[j][j] = sqrt(d);
        }
        __syncthreads();
        if (t > j && t < nb) T[t][j] /= T[j][j];
        __syncthreads();
        if (t > j && t < nb)
            for (int c = j + 1; c <= t; ++c) T[t][c] -= T[t][j] * T[c][j];
        __syncthreads();
    }
    for (int i = 0; i < nb; ++i)
        if (t < nb) A[(long long)i * lda + t] = (t <= i) ? T[i][t] : 0.0;    // the strict upper part is zeroed
}

// Rows of the panel P [rows, nb] (leading dimension ld): P <- P L^-T with L the nb x nb lower
// block; one thread per row (forward substitution along the row).
__global__ void __launch_bounds__(128)
panel_solve_kernel(double* __restrict__ P, long long ld, int rows, const double* __restrict__ L, long long ldl, int nb) {
    __shared__ double Ls[kCB][kCB + 1];
    for (int e = threadIdx.x; e < nb * nb; e += blockDim.x) Ls[e / nb][e % nb] = L[(long long)(e / nb) * ldl + e % nb];
    __syncthreads();
    const int row = blockIdx.x * blockDim.x + threadIdx.x;
    if (row >= rows) return;
    double x[kCB];
    double* p = P + (long long)row * ld;
#pragma unroll 1
    for (int j = 0; j < nb; ++j) {
        double v = p[j];
        for (int i = 0; i < j; ++i) v -= x[i] * Ls[j][i];
        x[j] = v / Ls[j][j];
        p[j] = x[j];
    }
}

int potrf_lower(cudaStream_t st, double* A, long long lda, int n, int* fail) {
    for (int j = 0; j < n; j += kCB) {
        const int nb = (n - j < kCB) ? (n - j) : kCB;
        double* Ajj = A + (long long)j * lda + j;
        potrf_diag_kernel<<<1, kCB, 0, st>>>(Ajj, lda, nb, fail);
        const int rest = n - j - nb;
        if (rest > 0) {
            double* P = A + (long long)(j + nb) * lda + j;
            panel_solve_kernel<<<(rest + 127) / 128, 128, 0, st>>>(P, lda, rest, Ajj, lda, nb);
            // trailing update: A22 -= P P^T
            int rc = dgemm(st, rest, rest, nb, -1.0, P, lda, 1, P, 1, lda, 1.0, A + (long long)(j + nb) * lda + (j + nb), lda);
            if (rc != ASER_OK) return rc;
        }
    }
    return check_launch("potrf");
}

// Zero the strict upper triangle (the blocked factorisation leaves the original entries there).
__global__ void zero_upper_kernel(double* __restrict__ A, long long lda, int n) {
    const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= (long long)n * n) return;
    const int i = (int)(e / n), j = (int)(e % n);
    if (j > i) A[(long long)i * lda + j] = 0.0;
}

// ---------------------------------------------------------------------------
// Z [p, ncols] <- L^-1 Z with L lower p x p: thread per column, forward substitution down the rows.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(128)
left_solve_lower_kernel(const double* __restrict__ L, long long ldl, int p, double* __restrict__ Z, long long ldz, int ncols) {
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= ncols) return;
    for (int i = 0; i < p; ++i) {
        double v = Z[(long long)i * ldz + c];
        const double* Li = L + (long long)i * ldl;
        for (int j = 0; j < i; ++j) v -= Li[j] * Z[(long long)j * ldz + c];
        Z[(long long)i * ldz + c] = v / Li[i];
    }
}

// Rows of X [rows, nb] (leading dimension ld): X <- X L^-1 with L the nb x nb lower block, i.e.
// solve x L = b backwards along the row; one thread per row.
__global__ void __launch_bounds__(128)
right_solve_lower_kernel(double* __restrict__ X, long long ld, int rows, const double* __restrict__ L, long long ldl, int nb) {
    __shared__ double Ls[kCB][kCB + 1];
    for (int e = threadIdx.x; e < nb * nb; e += blockDim.x) Ls[e / nb][e % nb] = L[(long long)(e / nb) * ldl + e % nb];
    __syncthreads();
    const int row = blockIdx.x * blockDim.x + threadIdx.x;
    if (row >= rows) return;
    double x[kCB];
    double* p = X + (long long)row * ld;
#pragma unroll 1
    for (int c = nb - 1; c >= 0; --c) {
        double v = p[c];
        for (int k = c + 1; k < nb; ++k) v -= x[k] * Ls[k][c];
        x[c] = v / Ls[c][c];
        p[c] = x[c];
    }
}

// ---------------------------------------------------------------------------
// operands
// ---------------------------------------------------------------------------
// E = fp32(W) * s (one fp32 multiply, as the quantizer sees it) - q * w_scale, in fp64.
__global__ void build_error_kernel(const __half* __restrict__ W, const float* __restrict__ s,
                                   const uint8_t* __restrict__ Wq, const float* __restrict__ w_scale,
                                   int N, int K, double* __restrict__ E) {
    const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= (long long)N * K) return;
    const int n = (int)(e / K), k = (int)(e % K);
    const float ws = __fmul_rn(__half2float(W[e]), s ? s[k] : 1.f);
    const uint8_t byte = Wq[(long long)n * (K / 2) + k / 2];
    int q = (k & 1) ? (byte >> 4) : (byte & 0xF);
    q = (q ^ 8) - 8;                                    // sign-extend the nibble
    E[e] = (double)ws - (double)q * (double)w_scale[n];
}

// Copy of W with the columns of the outlier set zeroed: what the quantizer sees under the outlier
// split of Sec. 4.2 (Eq. 12), where those columns are carried by the factors alone.
__global__ void mask_columns_kernel(const __half* __restrict__ W, int N, int K, const int* __restrict__ idx,
                                    int n_idx, __half* __restrict__ Wm) {
    const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= (long long)N * K) return;
    const int k = (int)(e % K);
    bool out = false;
    for (int i = 0; i < n_idx; ++i) out = out || (idx[i] == k);
    Wm[e] = out ? __float2half(0.f) : W[e];
}

// X~ = fp32(X) / s (one fp32 division), in fp64.
__global__ void build_xs_kernel(const __half* __restrict__ X, const float* __restrict__ s, int T, int K,
                                double* __restrict__ Xs) {
    const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= (long long)T * K) return;
    const float x = __half2float(X[e]);
    Xs[e] = (double)(s ? __fdiv_rn(x, s[e % K]) : x);
}

// G += lambda I with lambda = damping * trace(G) / K; one CTA (the trace is summed in a fixed order).
__global__ void __launch_bounds__(256) damp_kernel(double* __restrict__ G, int K, double damping, double* __restrict__ lambda_out) {
    __shared__ double red[256];
    double t = 0.0;
    for (int i = threadIdx.x; i < K; i += 256) t += G[(long long)i * K + i];
    red[threadIdx.x] = t;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if ((int)threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    const double lam = damping * red[0] / K;
    for (int i = threadIdx.x; i < K; i += 256) G[(long long)i * K + i] += lam;
    if (threadIdx.x == 0 && lambda_out) *lambda_out = lam;
}

// Start vectors: a fixed hash of the index mapped to (-1, 1) (any full-rank start works).
__global__ void init_basis_kernel(double* __restrict__ Qt, long long n) {
    const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= n) return;
    unsigned long long z = (unsigned long long)e * 0x9E3779B97F4A7C15ull + 0x243F6A8885A308D3ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    z ^= z >> 31;
    Qt[e] = (double)(z >> 11) * (2.0 / 9007199254740992.0) - 1.0;
}

// ---------------------------------------------------------------------------
// One round of one-sided Jacobi: CTA b rotates rows (i, j) = pairs[b] of Bt [p, N] so that they
// become orthogonal, and applies the same rotation to rows i, j of Qt [p, K].
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
jacobi_round_kernel(double* __restrict__ Bt, int N, double* __restrict__ Qt, int K, int p, int round) {
    // round-robin tournament over p (even) players: player p-1 stays, the others rotate
    const int b = blockIdx.x, m = p - 1;
    int i = (b == 0) ? m : (round + b) % m;
    int j = (round + m - b) % m;
    if (b == 0) { i = round % m; j = m; }
    if (i > j) { const int t = i; i = j; j = t; }
    double* bi = Bt + (long long)i * N;
    double* bj = Bt + (long long)j * N;
    __shared__ double red[3][256];
    double a = 0.0, bb = 0.0, g = 0.0;
    for (int k = threadIdx.x; k < N; k += 256) {
        const double x = bi[k], y = bj[k];
        a = fma(x, x, a); bb = fma(y, y, bb); g = fma(x, y, g);
    }
    red[0][threadIdx.x] = a; red[1][threadIdx.x] = bb; red[2][threadIdx.x] = g;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if ((int)threadIdx.x < o) {
            red[0][threadIdx.x] += red[0][threadIdx.x + o];
            red[1][threadIdx.x] += red[1][threadIdx.x + o];
            red[2][threadIdx.x] += red[2][threadIdx.x + o];
        }
        __syncthreads();
    }
    a = red[0][0]; bb = red[1][0]; g = red[2][0];
    if (fabs(g) <= 1e-300 || fabs(g) <= 1e-17 * sqrt(a * bb)) return;      // already orthogonal
    const double zeta = (bb - a) / (2.0 * g);
    const double t = (zeta >= 0.0 ? 1.0 : -1.0) / (fabs(zeta) + sqrt(1.0 + zeta * zeta));
    const double c = 1.0 / sqrt(1.0 + t * t), s = c * t;
    for (int k = threadIdx.x; k < N; k += 256) {
        const double x = bi[k], y = bj[k];
        bi[k] = c * x - s * y;
        bj[k] = s * x + c * y;
    }
    double* qi = Qt + (long long)i * K;
    double* qj = Qt + (long long)j * K;
    for (int k = threadIdx.x; k < K; k += 256) {
        const double x = qi[k], y = qj[k];
        qi[k] = c * x - s * y;
        qj[k] = s * x + c * y;
    }
}

// Squared norms of the rows of Bt, then (one thread) the indices of the r largest in descending
// order: order[0..r).  p <= 1024.
__global__ void __launch_bounds__(256) row_norms_kernel(const double* __restrict__ Bt, int N, double* __restrict__ norms) {
    __shared__ double red[256];
    const double* b = Bt + (long long)blockIdx.x * N;
    double a = 0.0;
    for (int k = threadIdx.x; k < N; k += 256) a = fma(b[k], b[k], a);
    red[threadIdx.x] = a;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if ((int)threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) norms[blockIdx.x] = red[0];
}
__global__ void select_top_kernel(double* __restrict__ norms, int p, int r, int* __restrict__ order, double* __restrict__ sigma_out) {
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    for (int t = 0; t < r; ++t) {
        int best = 0;
        for (int i = 1; i < p; ++i) if (norms[i] > norms[best]) best = i;
        order[t] = best;
        if (sigma_out) sigma_out[t] = sqrt(norms[best]);
        norms[best] = -1.0;
    }
}

// L_B[n, t] = fp16(Bt[order[t], n]);  Vt[t, k] = Qt[order[t], k] (fp64, input of the last solve).
__global__ void gather_kernel(const double* __restrict__ Bt, int N, const double* __restrict__ Qt, int K,
                              const int* __restrict__ order, int r, __half* __restrict__ LB, double* __restrict__ Vt) {
    const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (e < (long long)N * r) {
        const int n = (int)(e / r), t = (int)(e % r);
        LB[e] = __double2half(Bt[(long long)order[t] * N + n]);
    }
    if (e < (long long)r * K) {
        const int t = (int)(e / K), k = (int)(e % K);
        Vt[e] = Qt[(long long)order[t] * K + k];
    }
}
__global__ void to_half_kernel(const double* __restrict__ src, long long n, __half* __restrict__ dst) {
    const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (e < n) dst[e] = __double2half(src[e]);
}

struct ConstructLayout {
    int p;
    size_t E, A, G, Xs, Qt, Zt, Yt, C, Vt, norms, lambda, order, fail, Wm, total;     // byte offsets
};

ConstructLayout construct_layout(int N, int K, int Tcal, int r, int n_split) {
    ConstructLayout L;
    int p = r + (r / 2 > 32 ? r / 2 : 32);
    p += p & 1;
    const int lim = (N < K ? N : K) & ~1;
    if (p > lim) p = lim;
    L.p = p;
    size_t off = 0;
    auto take = [&](size_t bytes) { const size_t o = off; off += (bytes + 255) / 256 * 256; return o; };
    L.E = take((size_t)N * K * 8);
    L.A = take((size_t)N * K * 8);
    L.G = take((size_t)K * K * 8);
    L.Xs = take((size_t)Tcal * K * 8);
    L.Qt = take((size_t)p * K * 8);
    L.Zt = take((size_t)p * K * 8);
    L.Yt = take((size_t)p * N * 8);
    L.C = take((size_t)p * p * 8);
    L.Vt = take((size_t)(r > 0 ? r : 1) * K * 8);
    L.norms = take((size_t)p * 8);
    L.lambda = take(8);
    L.order = take((size_t)(r > 0 ? r : 1) * 4);
    L.fail = take(4);
    L.Wm = take(n_split > 0 ? (size_t)N * K * 2 : 0);
    L.total = off;
    return L;
}

inline int blocks_for(long long n, int threads) { return (int)((n + threads - 1) / threads); }

// Rows of Z [p, K] made orthonormal: C = Z Z^T = L L^T, Z <- L^-1 Z, twice (the second pass
// removes what rounding left of the first).
int orthonormalize_rows(cudaStream_t st, double* Z, int p, int K, double* C, int* fail) {
    for (int pass = 0; pass < 2; ++pass) {
        int rc = dgemm(st, p, p, K, 1.0, Z, K, 1, Z, 1, K, 0.0, C, p);
        if (rc != ASER_OK) return rc;
        rc = potrf_lower(st, C, p, p, fail);
        if (rc != ASER_OK) return rc;
        left_solve_lower_kernel<<<blocks_for(K, 128), 128, 0, st>>>(C, p, p, Z, K, K);
    }
    return check_launch("orthonormalize_rows");
}

}  // namespace

size_t construct_workspace_bytes(int N, int K, int Tcal, int r, int n_split) {
    return construct_layout(N, K, Tcal, r, n_split).total;
}

int launch_construct(const __half* W, const float* s, const __half* Xcal, int N, int K, int Tcal, int r,
                     double damping, int iters, uint8_t* Wq, float* w_scale, __half* LA, __half* LB,
                     double* sigma_out, double* S_out, const int* split_idx, int n_split, void* workspace,
                     cudaStream_t st) {
    const ConstructLayout L = construct_layout(N, K, Tcal, r, n_split);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    double* E = reinterpret_cast<double*>(ws + L.E);
    double* A = reinterpret_cast<double*>(ws + L.A);
    double* G = reinterpret_cast<double*>(ws + L.G);
    double* Xs = reinterpret_cast<double*>(ws + L.Xs);
    double* Qt = reinterpret_cast<double*>(ws + L.Qt);
    double* Zt = reinterpret_cast<double*>(ws + L.Zt);
    double* Yt = reinterpret_cast<double*>(ws + L.Yt);
    double* C = reinterpret_cast<double*>(ws + L.C);
    double* Vt = reinterpret_cast<double*>(ws + L.Vt);
    double* norms = reinterpret_cast<double*>(ws + L.norms);
    double* lambda = reinterpret_cast<double*>(ws + L.lambda);
    int* order = reinterpret_cast<int*>(ws + L.order);
    int* fail = reinterpret_cast<int*>(ws + L.fail);
    const int p = L.p;

    const __half* Wquant = W;
    if (n_split > 0) {      // the quantizer sees W without the outlier columns; E below keeps them
        __half* Wm = reinterpret_cast<__half*>(ws + L.Wm);
        mask_columns_kernel<<<blocks_for((long long)N * K, 256), 256, 0, st>>>(W, N, K, split_idx, n_split, Wm);
        Wquant = Wm;
    }
    int rc = launch_pack_w4(Wquant, s, N, K, Wq, w_scale, st);
    if (rc != ASER_OK) return rc;
    if (r == 0) return ASER_OK;
    cudaError_t e = cudaMemsetAsync(fail, 0, sizeof(int), st);
    if (e != cudaSuccess) return record_cuda_error(e, "construct: memset");
    build_error_kernel<<<blocks_for((long long)N * K, 256), 256, 0, st>>>(W, s, Wq, w_scale, N, K, E);
    build_xs_kernel<<<blocks_for((long long)Tcal * K, 256), 256, 0, st>>>(Xcal, s, Tcal, K, Xs);
    // G = X~^T X~ (the paper's X X^T), damped, then its Cholesky factor in place
    rc = dgemm(st, K, K, Tcal, 1.0, Xs, 1, K, Xs, K, 1, 0.0, G, K);
    if (rc != ASER_OK) return rc;
    damp_kernel<<<1, 256, 0, st>>>(G, K, damping, lambda);
    rc = potrf_lower(st, G, K, K, fail);
    if (rc != ASER_OK) return rc;
    zero_upper_kernel<<<blocks_for((long long)K * K, 256), 256, 0, st>>>(G, K, K);
    if (S_out) {
        e = cudaMemcpyAsync(S_out, G, (size_t)K * K * 8, cudaMemcpyDeviceToDevice, st);
        if (e != cudaSuccess) return record_cuda_error(e, "construct: copy S");
    }
    // A = E S
    rc = dgemm(st, N, K, K, 1.0, E, K, 1, G, K, 1, 0.0, A, K);
    if (rc != ASER_OK) return rc;
    // subspace iteration on A^T A with the basis as rows
    init_basis_kernel<<<blocks_for((long long)p * K, 256), 256, 0, st>>>(Qt, (long long)p * K);
    rc = orthonormalize_rows(st, Qt, p, K, C, fail);
    if (rc != ASER_OK) return rc;
    for (int it = 0; it < iters; ++it) {
        rc = dgemm(st, p, N, K, 1.0, Qt, K, 1, A, 1, K, 0.0, Yt, N);          // Yt = Qt A^T
        if (rc != ASER_OK) return rc;
        rc = dgemm(st, p, K, N, 1.0, Yt, N, 1, A, K, 1, 0.0, Zt, K);          // Zt = Yt A
        if (rc != ASER_OK) return rc;
        double* t = Qt; Qt = Zt; Zt = t;
        rc = orthonormalize_rows(st, Qt, p, K, C, fail);
        if (rc != ASER_OK) return rc;
    }
    // Rayleigh-Ritz: rotate the rows of Bt = Qt A^T (and of Qt with them) until they are orthogonal
    rc = dgemm(st, p, N, K, 1.0, Qt, K, 1, A, 1, K, 0.0, Yt, N);
    if (rc != ASER_OK) return rc;
    for (int sweep = 0; sweep < 12; ++sweep)
        for (int round = 0; round < p - 1; ++round)
            jacobi_round_kernel<<<p / 2, 256, 0, st>>>(Yt, N, Qt, K, p, round);
    row_norms_kernel<<<p, 256, 0, st>>>(Yt, N, norms);
    select_top_kernel<<<1, 32, 0, st>>>(norms, p, r, order, sigma_out);
    const long long ge = (long long)(N > K ? N : K) * r;
    gather_kernel<<<blocks_for(ge, 256), 256, 0, st>>>(Yt, N, Qt, K, order, r, LB, Vt);
    // L_A S = V_r^T: solve backwards over 64-column blocks, in place in Vt
    for (int c0 = ((K - 1) / kCB) * kCB; c0 >= 0; c0 -= kCB) {
        const int nb = (K - c0 < kCB) ? (K - c0) : kCB;
        const int done = K - c0 - nb;           // columns behind the block, already solved
        if (done > 0) {
            rc = dgemm(st, r, nb, done, -1.0, Vt + c0 + nb, K, 1, G + (long long)(c0 + nb) * K + c0, K, 1, 1.0,
                       Vt + c0, K);
            if (rc != ASER_OK) return rc;
        }
        right_solve_lower_kernel<<<blocks_for(r, 128), 128, 0, st>>>(Vt + c0, K, r, G + (long long)c0 * K + c0, K, nb);
    }
    to_half_kernel<<<blocks_for((long long)r * K, 256), 256, 0, st>>>(Vt, (long long)r * K, LA);
    rc = check_launch("construct");
    if (rc != ASER_OK) return rc;
    // an offline step: wait for it and report a failed factorisation
    int host_fail = 0;
    e = cudaMemcpyAsync(&host_fail, fail, sizeof(int), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return record_cuda_error(e, "construct");
    if (host_fail) return record_error(ASER_ERR_SHAPE, "construct: the damped Gram matrix is not positive definite");
    return ASER_OK;
}

}  // namespace aser
