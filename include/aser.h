/*
 * aser.h -- C ABI of the B200 (sm_100a) library for the forward pass of an
 * ASER-quantized linear layer (Activation Smoothing + Error Reconstruction,
 * arXiv 2411.07762):
 *
 *     Y = dequant( Q4(W diag(s)) . Q8(diag(s)^-1 X) ) + L_B (L_A X~),   X~ = diag(s)^-1 X
 *
 * which is the paper's inference pass "W_q X + L_A L_B X" on the smoothed
 * activation M^-1 X (Sec. 4.2, last paragraph before Algorithm 1).
 *
 * NAMES.  Token-major storage: X [M tokens, K], W [N, K], Y = X W^T [M, N].
 *   s    [K]   fp32  diagonal of the paper's smoothing matrix M (Sec. 4.2, Eq. 10)
 *   L_A  [r,K] fp16  DOWN projection  V_r^T S^-1   (the paper calls this one L_B)
 *   L_B  [N,r] fp16  UP projection    U_r Sigma_r  (the paper calls this one L_A)
 *   T    [M,r] bf16  T = X~ L_A^T, the intermediate between the two kernels
 *
 * CONVENTIONS.  Every function returns 0 (ASER_OK) or a negative ASER_ERR_*;
 * on error nothing has been launched unless stated.  Every data pointer is a
 * DEVICE pointer owned by the caller unless its name ends in _host; arrays are
 * row-major and contiguous; pointers must be 16-byte aligned.  The library
 * allocates no memory, never synchronises (except aser_check_status), and
 * enqueues all work on the cudaStream_t passed as `stream` (NULL = the legacy
 * default stream).  A process may use the library on several devices (the one current at the
 * call is used; per-device set-up is done on first use).  NaN/Inf inputs give unspecified
 * values but never a fault.
 * Shapes: M >= 0, K % 128 == 0, N % 8 == 0, r % 16 == 0, 0 <= r <= 256.
 * M == 0 is a no-op that returns ASER_OK.
 */
#ifndef ASER_H_
#define ASER_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ASER_OK                  0
#define ASER_ERR_NULL           -1  /* a required pointer is NULL */
#define ASER_ERR_ALIGN          -2  /* a pointer is not 16-byte aligned */
#define ASER_ERR_SHAPE          -3  /* unsupported M, N, K or r */
#define ASER_ERR_WORKSPACE      -4  /* workspace NULL or smaller than aser_workspace_bytes() */
#define ASER_ERR_LAUNCH         -5  /* CUDA reported an error; text in aser_last_error() */
#define ASER_ERR_DEVICE_TIMEOUT -6  /* a bounded in-kernel wait gave up (see aser_check_status) */
#define ASER_ERR_DEVICE         -7  /* current device is not compute capability 10.x */

/*
 * aser_pack_w4 -- offline weight quantization (Sec. 4.2 Eq. 10/12: Q(W_s) of the
 * smoothed weight W M; Sec. 5.1: per-channel round-to-nearest).
 *   ws = fp32(W[n,k]) * s[k]            (one fp32 multiply; s == NULL means ones)
 *   w_scale[n] = max_k |ws| / 7         (fp32 division)
 *   q = clamp(rne(ws / w_scale[n]), -8, 7)   (fp32 division, half-to-even)
 * A zero row gets scale 0 and codes 0.
 * Output Wq [N, K/2] is the CANONICAL packed form: byte j of row n holds
 * (q[n,2j] & 0xF) | (q[n,2j+1] << 4).  Bit-exact with the definition above.
 */
int aser_pack_w4(const void* W_f16, const float* s, int N, int K,
                 uint8_t* Wq, float* w_scale, void* stream);

/*
 * aser_repack_w4 / aser_unrepack_w4 -- pure permutation between the canonical
 * packed form and the layout the tensor-core kernel streams ("Wk").  Wk has
 * aser_repacked_bytes(N, K) bytes: N is padded to a multiple of 128 with zero
 * codes; each (128-row, 128-column) block is stored contiguously.  The paper
 * has no counterpart (it fixes no storage format).  unrepack is the exact
 * inverse on the first N rows.
 */
size_t aser_repacked_bytes(int N, int K);
int aser_repack_w4(const uint8_t* Wq, int N, int K, void* Wk, void* stream);
int aser_unrepack_w4(const void* Wk, int N, int K, uint8_t* Wq, void* stream);

/*
 * aser_quant_act -- fused activation kernel: smoothing (Sec. 4.2, the M^-1 X
 * factor of Eq. 10), per-token int8 round-to-nearest (Sec. 5.1) and the down
 * projection of the reconstruction branch (Sec. 4.1, V_r^T S^-1 applied to X~).
 *   x~ = fp32(X[m,k]) / s[k]                       (fp32 division; s == NULL means ones)
 *   a_scale[m] = max_k |x~| / 127                  (fp32 division; zero row -> 0, codes 0)
 *   Xq[m,k] = clamp(rne(x~ / a_scale[m]), -127, 127)
 *   T[m,j]  = bf16( sum_k L_A[j,k] * x~[m,k] )     (fp32 accumulation; x~ may be rounded to
 *                                                   fp16 first when tensor cores are used)
 * Xq and a_scale are bit-exact with the definition.  r == 0: LA_f16 and T_bf16 are ignored.
 */
int aser_quant_act(const void* X_f16, const float* s, const void* LA_f16,
                   int M, int K, int r,
                   int8_t* Xq, float* a_scale, void* T_bf16, void* stream);

/*
 * aser_quant_act_bits -- aser_quant_act with activation codes of act_bits bits (2..8), the
 * paper's W4A6 setting being act_bits = 6 (Sec. 5.2, the W4A6 rows of the main results):
 *   qmax = 2^(act_bits-1) - 1;  a_scale[m] = max_k |x~| / qmax;
 *   Xq[m,k] = clamp(rne(x~ / a_scale[m]), -qmax, qmax)
 * The codes are stored in the same int8 array, so the linear kernels need no change: the scale
 * carries the coarser step.  act_bits = 8 is aser_quant_act.  Everything else (arguments,
 * layouts, T, bit-exactness of Xq and a_scale) as there; other widths return ASER_ERR_SHAPE.
 */
int aser_quant_act_bits(const void* X_f16, const float* s, const void* LA_f16,
                        int M, int K, int r, int act_bits,
                        int8_t* Xq, float* a_scale, void* T_bf16, void* stream);

/*
 * aser_quant_act_ex -- aser_quant_act_bits with a choice of how T is stored (the paper fixes no
 * storage precision for the intermediate of its low-rank branch, Sec. 4.1):
 *   t_pair == 0: T [M, r] bf16, as above.
 *   t_pair == 1: T [M, 2r] bf16 holds every entry as a pair, T[m,j] = bf16(t) and
 *                T[m,r+j] = bf16(t - T[m,j]), i.e. 16 significant bits instead of 8.  The linear
 *                kernels need no change: call them with rank 2r and the up projection written
 *                twice, LB2 [N, 2r] = [L_B | L_B], so that L_B T_hi + L_B T_lo is what they add.
 *                Needs 2r <= 256.  Meant for layers whose low-rank term is as large as the
 *                output itself (the paper's outlier split of Sec. 4.2, Eq. 12, where whole
 *                weight columns ride on the factors): there the 2^-9 rounding of a single bf16
 *                is not small against the output tolerance.
 * Everything else as aser_quant_act_bits.
 */
int aser_quant_act_ex(const void* X_f16, const float* s, const void* LA_f16,
                      int M, int K, int r, int act_bits, int t_pair,
                      int8_t* Xq, float* a_scale, void* T_bf16, void* stream);

/*
 * aser_quant_act_ws -- aser_quant_act_ex for callers that can spare scratch memory (same
 * passages of the paper; the scratch is an implementation matter).  With more than 32 tokens it
 * runs two kernels instead of one: the first reads X once, takes the row maxima and the
 * projection T on the tensor cores and leaves per-slice partial results in the scratch; the
 * second writes the scales, the codes and T.  Results are those of aser_quant_act_ex (Xq and
 * a_scale bit-exact; T may differ in its last bf16 bit because the fp32 sums are formed in a
 * different order), at several times the throughput.  Two extensions:
 *   - r may go up to 512 (a multiple of 16): L_A may be the STACKED down projections of
 *     several layers that read the same X and share s (query/key/value, gate/up), so that X is
 *     read and quantized once; T [M, r] then holds the layers' T side by side and each layer's
 *     linear kernel is given its column range (aser_linear_w4a8_lr_ld);
 *   - with t_pair, 2 r <= 512.
 * workspace: aser_quant_workspace_bytes(M, K, r) bytes, 16-byte aligned, contents irrelevant
 * (the first 1024 bytes are not touched, so a linear kernel's workspace may be lent).  Work on
 * `stream` that still uses the workspace when the call is made must precede it on `stream`.
 */
size_t aser_quant_workspace_bytes(int M, int K, int r);
/* Number of kernels one aser_quant_act_ws call enqueues (two per chunk of tokens; 0 for bad shapes). */
int aser_quant_act_ws_launches(int M, int K);
int aser_quant_act_ws(const void* X_f16, const float* s, const void* LA_f16,
                      int M, int K, int r, int act_bits, int t_pair,
                      int8_t* Xq, float* a_scale, void* T_bf16,
                      void* workspace, size_t workspace_bytes, void* stream);

/*
 * aser_linear_w4a8_lr -- integer GEMM, dequantisation and up projection
 * (Sec. 4.2: W_q X + L_A L_B X in the paper's letters):
 *   acc[m,n] = sum_k Xq[m,k] * q[n,k]                               (exact int32)
 *   Y[m,n]   = fp16( acc * a_scale[m] * w_scale[n] + sum_j L_B[n,j] * T[m,j] )   (fp32)
 * Wk is the repacked weight (aser_repack_w4).  acc_debug, when not NULL, receives the
 * int32 accumulators [M,N] (bit-exact); pass NULL in timed runs.  workspace must hold
 * aser_workspace_bytes(M,N,K,r) bytes, must have been zeroed once with
 * aser_workspace_init, and may be reused by later calls on the same stream, of the same or of
 * any other shape it is large enough for (the status word and the tile counters sit at fixed
 * offsets and every launch leaves the counters at zero); two calls that overlap in time need
 * separate workspaces.  Both kernels feed T to the tensor cores as fp16: finite entries of
 * magnitude 65504 or more become infinite there, so |T| must stay below that.  With at most 16 tokens and at most 64 MB of
 * packed weights the call runs a streaming kernel that leaves the workspace untouched; the
 * argument is validated all the same, so callers need not know which kernel serves a shape.
 * aser_linear_w4a8 is the same without the low-rank term (the plain W4A8 control).
 */
int aser_linear_w4a8_lr(const int8_t* Xq, const float* a_scale, const void* Wk,
                        const float* w_scale, const void* T_bf16, const void* LB_f16,
                        int M, int N, int K, int r, void* Y_f16, int32_t* acc_debug,
                        void* workspace, size_t workspace_bytes, void* stream);
int aser_linear_w4a8(const int8_t* Xq, const float* a_scale, const void* Wk,
                     const float* w_scale, int M, int N, int K, void* Y_f16,
                     int32_t* acc_debug, void* workspace, size_t workspace_bytes, void* stream);
/*
 * aser_linear_w4a8_lr_ld -- aser_linear_w4a8_lr with T given as a column range of a wider
 * matrix: T_bf16 points at the layer's first column and consecutive rows are ldt elements apart
 * (ldt >= r, a multiple of 8; 0 means r).  This is how the layers of a shared-input group read
 * their part of a stacked T.
 */
int aser_linear_w4a8_lr_ld(const int8_t* Xq, const float* a_scale, const void* Wk,
                           const float* w_scale, const void* T_bf16, int ldt, const void* LB_f16,
                           int M, int N, int K, int r, void* Y_f16, int32_t* acc_debug,
                           void* workspace, size_t workspace_bytes, void* stream);

/*
 * aser_linear_w4a8_lr_simt -- the same operation on CUDA cores (dp4a) from the
 * CANONICAL packed weights; slow, used as an on-device cross-check.  r == 0 (with
 * NULL T/LB) gives the plain product.  Needs no workspace.
 */
int aser_linear_w4a8_lr_simt(const int8_t* Xq, const float* a_scale, const uint8_t* Wq,
                             const float* w_scale, const void* T_bf16, const void* LB_f16,
                             int M, int N, int K, int r, void* Y_f16, int32_t* acc_debug,
                             void* stream);

/*
 * aser_linear_w4a8_lr_static -- the tensor-core kernel of aser_linear_w4a8_lr (the one that needs
 * scratch memory, at every shape this entry accepts) for callers that must not allocate device
 * memory and therefore have no workspace to hand over: code running inside a memory budget
 * that was fixed at start-up (a serving process that gave every free byte to its own pool, so
 * cudaMalloc would fail), or at a point where allocating is not allowed because it would
 * synchronise the device (inside a latency-critical loop, between the kernels of a step).  The
 * paper has no counterpart; this is a deployment convenience of the library.
 * The scratch is a fixed 8 MiB array inside the library image; every GPU that loads the library
 * holds one copy until the process exits.  Limits and rules:
 *   - only problems with aser_workspace_bytes(M,N,K,r) <= 8 MiB are accepted, i.e. at most 32
 *     tokens per call (any N, K, r the library supports); larger ones return ASER_ERR_WORKSPACE
 *     and launch nothing;
 *   - the first call on each device looks the array's device address up (with that device
 *     current); make that first call before starting any stream capture;
 *   - no cudaMalloc/cudaFree or other allocating routine is called; each call enqueues a small
 *     memset (status word and tile counters) and the kernel on `stream`;
 *   - all calls on a device share the one array, so two calls that may overlap in time on the
 *     GPU (different streams, no dependency) corrupt each other: order them;
 *   - the status word is not readable by the caller: a timed-out wait (see aser_check_status)
 *     cannot be detected through this entry point.
 * Arguments and results are those of aser_linear_w4a8_lr; pass r = 0 with NULL T/LB for the
 * plain product.
 */
int aser_linear_w4a8_lr_static(const int8_t* Xq, const float* a_scale, const void* Wk,
                               const float* w_scale, const void* T_bf16, const void* LB_f16,
                               int M, int N, int K, int r, void* Y_f16, int32_t* acc_debug,
                               void* stream);

/* Workspace: split-K partial sums, tile counters and a status word. */
size_t aser_workspace_bytes(int M, int N, int K, int r);
int aser_workspace_init(void* workspace, size_t workspace_bytes, void* stream);
/*
 * aser_check_status -- synchronises `stream`, reads the status word and returns
 * ASER_OK or ASER_ERR_DEVICE_TIMEOUT (a kernel's bounded wait, about 0.2 s, gave up; its output
 * is invalid).  Clears the word and the tile counters that such a launch may have left
 * behind, so the workspace is usable again.  Debugging aid, not part of the hot path.
 */
int aser_check_status(void* workspace, void* stream);

/*
 * aser_forward -- one whole forward pass of the layer (Sec. 4.2, Eq. 10 with the low-rank term
 * of Sec. 4.1) from DEVICE buffers: aser_quant_act followed by aser_linear_w4a8_lr (the plain
 * kernel when r == 0), enqueued on `stream`, no synchronisation.
 * Because the library knows that the quantization kernel is what precedes the linear kernel,
 * it launches the latter as a programmatic dependent: the linear kernel starts while the
 * quantization still runs, streams the weights (which that kernel does not write) and waits
 * for its completion before it reads Xq, a_scale or T.  The activation step is whichever of
 * aser_quant_act's kernels and aser_quant_act_ws's (on the same workspace) is faster at the
 * shape: the latter from 1024 tokens on and for every rank above 128;
 * aser_forward_act_launches tells how many kernels that is.  Results are those of the separate
 * calls.
 * X_f16 [M,K], s [K] or NULL, LA_f16 [r,K] / LB_f16 [N,r] (NULL when r == 0), Wk and w_scale as
 * for aser_linear_w4a8_lr.  Xq [M,K], a_scale [M], T_bf16 [M,r] (NULL when r == 0) are the
 * caller's intermediates (written), Y_f16 [M,N] the result.  Wk, w_scale and LB_f16 must not
 * be written by work still in flight on `stream` when the call is made.
 * Errors: as the two calls; every argument of both launches is checked first, so nothing is
 * enqueued when one is rejected.
 */
int aser_forward_act_launches(int M, int K, int r);
int aser_forward(const void* X_f16, const float* s, const void* LA_f16, const void* Wk,
                 const float* w_scale, const void* LB_f16, int M, int N, int K, int r,
                 int8_t* Xq, float* a_scale, void* T_bf16, void* Y_f16,
                 void* workspace, size_t workspace_bytes, void* stream);

/*
 * aser_forward_shared -- the forward pass of n_layers layers that read the SAME activation X
 * and share the smoothing vector s (Algorithm 1 builds each layer's factors on its own; where
 * the layers' inputs and s coincide their activation work is identical): X is smoothed and
 * quantized once, one pass computes every layer's T from the stacked down projections
 * LA_stacked [sum r, K] (layer l's rows follow layer l-1's), then each layer's linear kernel runs
 * on the shared codes.  Per layer l: Wk[l], w_scale[l], LB_f16[l] [N[l], r[l]], Y_f16[l] [M, N[l]].
 * Xq [M, K], a_scale [M], T_bf16 [M, sum r] are the caller's intermediates.  sum r <= 512.
 * workspace: aser_forward_shared_workspace_bytes(...) bytes, zeroed once with
 * aser_workspace_init.  Each layer's output equals that of aser_forward on that layer alone up
 * to the last bf16 bit of T.  Errors: every argument is checked before anything is enqueued.
 */
size_t aser_forward_shared_workspace_bytes(int n_layers, const int* N, const int* r, int M, int K);
int aser_forward_shared(const void* X_f16, const float* s, const void* LA_stacked_f16, int n_layers,
                        const void* const* Wk, const float* const* w_scale,
                        const void* const* LB_f16, const int* N, const int* r, int M, int K,
                        int8_t* Xq, float* a_scale, void* T_bf16, void* const* Y_f16,
                        void* workspace, size_t workspace_bytes, void* stream);

/*
 * aser_linear_w4a8_lr_cat / aser_forward_shared_cat -- a shared-input group whose layers are STORED
 * one after the other along N, as a fused q/k/v or gate/up projection is: Wk_cat is the layers'
 * blocked weights concatenated (aser_pack_w4 of each layer, layer l's bytes behind layer l-1's;
 * every N[l] a positive multiple of 128, at most four layers), w_scale_cat [sum N],
 * LB_cat_f16 [sum N, r] (all layers of one rank r, r * n_layers <= 512), Y_cat_f16 [M, sum N]
 * (layer l's output is the column range of its rows).  One linear launch then serves the whole
 * group: a weight tile multiplies the columns [l r, (l + 1) r) of T_bf16 [M, r * n_layers] of the
 * layer l it lies in.  The arithmetic per output element is that of aser_linear_w4a8_lr on the
 * layer alone (Sec. 4.1 Eq. 7 with the stacked operands of Algorithm 1's independent layers), so
 * the results are bit-identical to it.  aser_forward_shared_cat runs the activation pass first
 * (as aser_forward_shared).  workspace: aser_forward_shared_cat_workspace_bytes(...) bytes,
 * zeroed once with aser_workspace_init; for the linear step alone
 * aser_workspace_bytes(M, sum N, K, r) is enough.  Errors: every argument is checked before
 * anything is enqueued.
 */
int aser_linear_w4a8_lr_cat(const int8_t* Xq, const float* a_scale, const void* Wk_cat,
                            const float* w_scale_cat, const void* T_bf16, const void* LB_cat_f16,
                            int n_layers, const int* N, int r, int M, int K, void* Y_cat_f16,
                            void* workspace, size_t workspace_bytes, void* stream);
size_t aser_forward_shared_cat_workspace_bytes(int n_layers, const int* N, int r, int M, int K);
int aser_forward_shared_cat(const void* X_f16, const float* s, const void* LA_stacked_f16, int n_layers,
                            const void* Wk_cat, const float* w_scale_cat, const void* LB_cat_f16,
                            const int* N, int r, int M, int K, int8_t* Xq, float* a_scale,
                            void* T_bf16, void* Y_cat_f16, void* workspace, size_t workspace_bytes,
                            void* stream);

/*
 * aser_forward_host -- one whole forward pass from HOST buffers: copies X (fp16 [M,K],
 * ideally pinned) to the device staging buffer X_dev, runs aser_forward, and copies Y back to Y_host,
 * all enqueued on `stream`; returns without synchronising.  Device-side operands and
 * staging buffers are the caller's.  All arguments are checked before the first copy is
 * enqueued.
 */
int aser_forward_host(const void* X_host_f16, void* Y_host_f16,
                      void* X_dev, int8_t* Xq_dev, float* a_scale_dev, void* T_dev, void* Y_dev,
                      const float* s, const void* LA_f16, const void* Wk, const float* w_scale,
                      const void* LB_f16, int M, int N, int K, int r,
                      void* workspace, size_t workspace_bytes, void* stream);

/*
 * aser_construct -- the per-layer body of Algorithm 1 on the device: quantize W diag(s) to int4
 * (aser_pack_w4), form the error E = W diag(s) - dequant(W_q), whiten with the Cholesky factor S
 * of the calibration Gram matrix (Sec. 4.1 Eq. 5; the paper's X X^T is X~^T X~ here, X~ =
 * X_cal diag(s)^-1, damped by lambda I with lambda = damping * trace / K because the Gram matrix
 * is singular with fewer calibration tokens than channels), take the r leading singular triplets
 * of E S (Eq. 6) and split them into L_B = U_r Sigma_r [N, r] and L_A = V_r^T S^-1 [r, K] (the
 * paper's L_A and L_B, in that order).  fp64 throughout, factors rounded to fp16 at the end.
 *   W_f16 [N, K], s [K] or NULL, Xcal_f16 [n_cal, K] calibration tokens (NOT yet smoothed).
 *   iterations: subspace iterations for the singular subspace (<= 0: 48); p = r + max(32, r/2)
 *   vectors are iterated, so the r-th triplet converges like (sigma_{p+1} / sigma_r)^(2 iterations).
 *   Outputs: Wq [N, K/2] canonical, w_scale [N], LA_f16 [r, K], LB_f16 [N, r]; optional
 *   sigma_out [r] (fp64 singular values, descending) and S_out [K, K] (fp64, lower, row-major).
 *   split_idx [n_split] (device, int32; NULL with n_split = 0): the outlier columns of the
 *   paper's split W M = W_s + W_o (Sec. 4.2 Eq. 12).  They are zeroed before the int4 quantizer
 *   (Wq then holds W_s only) and stay in the error E, so the factors carry them.  A forward pass
 *   of such a layer wants T stored as bf16 pairs (aser_quant_act_ex).
 *   workspace: aser_construct_workspace_bytes(N, K, n_cal, r, n_split) bytes (several N*K and
 *   K*K fp64 matrices).
 * Singular vectors are determined up to sign (and up to rotation among equal singular values):
 * compare the product L_B L_A and the singular values, not the factors element by element.
 * An offline step: the call SYNCHRONISES `stream` before it returns, and returns ASER_ERR_SHAPE
 * if the damped Gram matrix turned out not to be positive definite.  r == 0 only packs.
 */
size_t aser_construct_workspace_bytes(int N, int K, int n_cal, int r, int n_split);
int aser_construct(const void* W_f16, const float* s, const void* Xcal_f16, int N, int K, int n_cal,
                   int r, double damping, int iterations, uint8_t* Wq, float* w_scale,
                   void* LA_f16, void* LB_f16, double* sigma_out, double* S_out,
                   const int32_t* split_idx, int n_split,
                   void* workspace, size_t workspace_bytes, void* stream);

/* Text of the last CUDA error seen by the calling thread ("" if none). */
const char* aser_last_error(void);
/* Library version: major * 1000 + minor. */
int aser_version(void);

#ifdef __cplusplus
}
#endif
#endif /* ASER_H_ */
