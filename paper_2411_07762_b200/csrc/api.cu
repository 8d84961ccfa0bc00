// extern "C" boundary of the ASER linear library: argument validation and dispatch.
// No kernel lives here.
#include <stdio.h>
#include <string.h>

#include "aser_common.cuh"

namespace aser {

static thread_local char g_last_error[512] = "";

int record_cuda_error(cudaError_t e, const char* where) {
    snprintf(g_last_error, sizeof(g_last_error), "%s: %s (%s)", where, cudaGetErrorString(e),
             cudaGetErrorName(e));
    return ASER_ERR_LAUNCH;
}

int record_error(int code, const char* msg) {
    snprintf(g_last_error, sizeof(g_last_error), "%s", msg);
    return code;
}

int check_launch(const char* where) {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return record_cuda_error(e, where);
    return ASER_OK;
}

int current_device(int* dev) {
    cudaError_t e = cudaGetDevice(dev);
    if (e != cudaSuccess) return record_cuda_error(e, "cudaGetDevice");
    if (*dev < 0 || *dev >= kMaxDevices)
        return record_error(ASER_ERR_DEVICE, "device ordinal beyond the per-device tables");
    return ASER_OK;
}

int device_sm_count(int* num_sms) {
    static int cached[kMaxDevices] = {0};
    int dev = 0;
    int rc = current_device(&dev);
    if (rc != ASER_OK) return rc;
    if (cached[dev] == 0) {
        int n = 0;
        cudaError_t e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess || n <= 0) return record_cuda_error(e, "query SM count");
        cached[dev] = n;
    }
    *num_sms = cached[dev];
    return ASER_OK;
}

namespace {

int fail(int code, const char* msg) {
    snprintf(g_last_error, sizeof(g_last_error), "%s", msg);
    return code;
}

bool shape_ok(int M, int N, int K, int r) {
    return M >= 0 && N >= 0 && K > 0 && K % 128 == 0 && K <= 32768 && N % 8 == 0 && r >= 0 &&
           r <= 256 && r % 16 == 0;
}

// The kernels are built for sm_100a only; refuse to launch anywhere else.
int check_device() {
    static thread_local int cached_dev = -1;
    static thread_local int cached_rc = ASER_OK;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return record_cuda_error(e, "cudaGetDevice");
    if (dev == cached_dev) return cached_rc;
    int major = 0;
    e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) return record_cuda_error(e, "cudaDeviceGetAttribute");
    cached_dev = dev;
    cached_rc = (major == 10) ? ASER_OK
                              : fail(ASER_ERR_DEVICE, "device is not compute capability 10.x");
    return cached_rc;
}

#define ASER_REQUIRE_PTR(p)                                                   \
    do {                                                                      \
        if ((p) == nullptr) return fail(ASER_ERR_NULL, #p " is NULL");        \
        if (misaligned16(p)) return fail(ASER_ERR_ALIGN, #p " is not 16-byte aligned"); \
    } while (0)
#define ASER_OPTIONAL_PTR(p)                                                  \
    do {                                                                      \
        if ((p) != nullptr && misaligned16(p))                                \
            return fail(ASER_ERR_ALIGN, #p " is not 16-byte aligned");        \
    } while (0)

int linear_common(const int8_t* Xq, const float* a_scale, const void* Wk, const float* w_scale,
                  const void* T_bf16, const void* LB_f16, int M, int N, int K, int r, void* Y_f16,
                  int32_t* acc_debug, void* workspace, size_t workspace_bytes, void* stream,
                  bool overlap_prev = false, int ldt = 0, CatSplit cat = CatSplit()) {
    if (!shape_ok(M, N, K, r)) return fail(ASER_ERR_SHAPE, "unsupported M, N, K or r");
    if (r > 0 && ldt != 0 && (ldt < r || ldt % 8 != 0))
        return fail(ASER_ERR_SHAPE, "ldt must be a multiple of 8 and at least r");
    if (M == 0 || N == 0) return ASER_OK;
    ASER_REQUIRE_PTR(Xq);
    ASER_REQUIRE_PTR(a_scale);
    ASER_REQUIRE_PTR(Wk);
    ASER_REQUIRE_PTR(w_scale);
    ASER_REQUIRE_PTR(Y_f16);
    ASER_OPTIONAL_PTR(acc_debug);
    if (r > 0) {
        ASER_REQUIRE_PTR(T_bf16);
        ASER_REQUIRE_PTR(LB_f16);
    }
    if (workspace == nullptr || misaligned16(workspace) ||
        workspace_bytes < kWsHeaderBytes + linear_tc_workspace_bytes(M, N, K, r))
        return fail(ASER_ERR_WORKSPACE, "workspace missing, misaligned or too small");
    int rc = check_device();
    if (rc != ASER_OK) return rc;
    if (linear_decode_prefers(M, N, K))   // few tokens: the streaming kernel (the workspace stays untouched)
        return launch_linear_decode(Xq, a_scale, static_cast<const uint8_t*>(Wk), w_scale,
                                    static_cast<const __nv_bfloat16*>(T_bf16),
                                    static_cast<const __half*>(LB_f16), M, N, K, r,
                                    static_cast<__half*>(Y_f16), acc_debug,
                                    static_cast<cudaStream_t>(stream), overlap_prev, ldt, cat);
    return launch_linear_tc(Xq, a_scale, static_cast<const uint8_t*>(Wk), w_scale,
                            static_cast<const __nv_bfloat16*>(T_bf16),
                            static_cast<const __half*>(LB_f16), M, N, K, r,
                            static_cast<__half*>(Y_f16), acc_debug, workspace, workspace_bytes,
                            static_cast<cudaStream_t>(stream), overlap_prev, ldt, cat);
}

// Stacked ranks (several layers' down projections in one pass) go up to 512.
bool act_shape_ok(int M, int K, int r) {
    return M >= 0 && K > 0 && K % 128 == 0 && K <= 32768 && r >= 0 && r <= 512 && r % 16 == 0;
}

// Which activation kernels a forward pass runs.  The two-kernel path with scratch reads X once
// from HBM whatever the rank; it is the only one above rank 128 (stacked down projections of a
// shared-input group) and the faster one from about a thousand tokens on (measured at rank 128,
// two-kernel against cluster kernel: 1024 x 4096 21 against 27 us, 4096 x 4096 34 against 42 us,
// 2048 x 14336 52 against 65 us, 4096 x 14336 95 against 134 us, 8192 x 8192 107 against 159 us).
// Below that the one-launch cluster kernel is faster (256 x 4096: 23 against 17 us), and up to 32
// tokens the few-token kernel serves every rank.
bool forward_act_uses_scratch(int M, int K, int r) {
    if (M <= 32) return false;
    if (r > 128) return true;
    (void)K;
    return M >= 1024;
}

// The activation step of a forward pass (the scratch of the two-kernel path sits behind the
// workspace's zeroed prefix, where the linear kernel later keeps its partial sums).
int quant_with_workspace(const void* X_f16, const float* s, const void* LA_f16, int M, int K, int r,
                         int act_bits, bool t_pair, int8_t* Xq, float* a_scale, void* T_bf16,
                         void* workspace, size_t workspace_bytes, void* stream) {
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!forward_act_uses_scratch(M, K, r))
        return launch_quant_act(static_cast<const __half*>(X_f16), s, static_cast<const __half*>(LA_f16), M, K, r,
                                Xq, a_scale, static_cast<__nv_bfloat16*>(T_bf16), st, act_bits, t_pair);
    return launch_quant_act_ws(static_cast<const __half*>(X_f16), s, static_cast<const __half*>(LA_f16), M, K, r,
                               Xq, a_scale, static_cast<__nv_bfloat16*>(T_bf16),
                               static_cast<uint8_t*>(workspace) + kWsZeroedBytes,
                               workspace_bytes - kWsZeroedBytes, st, act_bits, t_pair);
}

}  // namespace
}  // namespace aser

using namespace aser;

extern "C" {

int aser_version(void) { return 1000; }

const char* aser_last_error(void) { return g_last_error; }

int aser_pack_w4(const void* W_f16, const float* s, int N, int K, uint8_t* Wq, float* w_scale,
                 void* stream) {
    if (!shape_ok(0, N, K, 0)) return fail(ASER_ERR_SHAPE, "unsupported N or K");
    if (N == 0) return ASER_OK;
    ASER_REQUIRE_PTR(W_f16);
    ASER_OPTIONAL_PTR(s);
    ASER_REQUIRE_PTR(Wq);
    ASER_REQUIRE_PTR(w_scale);
    int rc = check_device();
    if (rc != ASER_OK) return rc;
    return launch_pack_w4(static_cast<const __half*>(W_f16), s, N, K, Wq, w_scale,
                          static_cast<cudaStream_t>(stream));
}

size_t aser_repacked_bytes(int N, int K) {
    if (N <= 0 || K <= 0) return 0;
    size_t nb = ((size_t)N + kWkRows - 1) / kWkRows, kb = ((size_t)K + kWkCols - 1) / kWkCols;
    return nb * kb * kWkBlockBytes;
}

int aser_repack_w4(const uint8_t* Wq, int N, int K, void* Wk, void* stream) {
    if (!shape_ok(0, N, K, 0)) return fail(ASER_ERR_SHAPE, "unsupported N or K");
    if (N == 0) return ASER_OK;
    ASER_REQUIRE_PTR(Wq);
    ASER_REQUIRE_PTR(Wk);
    int rc = check_device();
    if (rc != ASER_OK) return rc;
    return launch_repack_w4(Wq, N, K, static_cast<uint8_t*>(Wk), false,
                            static_cast<cudaStream_t>(stream));
}

int aser_unrepack_w4(const void* Wk, int N, int K, uint8_t* Wq, void* stream) {
    if (!shape_ok(0, N, K, 0)) return fail(ASER_ERR_SHAPE, "unsupported N or K");
    if (N == 0) return ASER_OK;
    ASER_REQUIRE_PTR(Wq);
    ASER_REQUIRE_PTR(Wk);
    int rc = check_device();
    if (rc != ASER_OK) return rc;
    return launch_repack_w4(Wq, N, K, static_cast<uint8_t*>(const_cast<void*>(Wk)), true,
                            static_cast<cudaStream_t>(stream));
}

int aser_quant_act(const void* X_f16, const float* s, const void* LA_f16, int M, int K, int r,
                   int8_t* Xq, float* a_scale, void* T_bf16, void* stream) {
    return aser_quant_act_bits(X_f16, s, LA_f16, M, K, r, 8, Xq, a_scale, T_bf16, stream);
}

int aser_quant_act_bits(const void* X_f16, const float* s, const void* LA_f16, int M, int K, int r,
                        int act_bits, int8_t* Xq, float* a_scale, void* T_bf16, void* stream) {
    return aser_quant_act_ex(X_f16, s, LA_f16, M, K, r, act_bits, 0, Xq, a_scale, T_bf16, stream);
}

int aser_quant_act_ex(const void* X_f16, const float* s, const void* LA_f16, int M, int K, int r,
                      int act_bits, int t_pair, int8_t* Xq, float* a_scale, void* T_bf16,
                      void* stream) {
    if (!shape_ok(M, 0, K, r)) return fail(ASER_ERR_SHAPE, "unsupported M, K or r");
    if (act_bits < 2 || act_bits > 8) return fail(ASER_ERR_SHAPE, "act_bits must be 2..8");
    if (t_pair != 0 && t_pair != 1) return fail(ASER_ERR_SHAPE, "t_pair must be 0 or 1");
    if (t_pair && 2 * r > 256) return fail(ASER_ERR_SHAPE, "t_pair needs 2 r <= 256");
    if (M == 0) return ASER_OK;
    ASER_REQUIRE_PTR(X_f16);
    ASER_OPTIONAL_PTR(s);
    ASER_REQUIRE_PTR(Xq);
    ASER_REQUIRE_PTR(a_scale);
    if (r > 0) {
        ASER_REQUIRE_PTR(LA_f16);
        ASER_REQUIRE_PTR(T_bf16);
    }
    int rc = check_device();
    if (rc != ASER_OK) return rc;
    return launch_quant_act(static_cast<const __half*>(X_f16), s, static_cast<const __half*>(LA_f16),
                            M, K, r, Xq, a_scale, static_cast<__nv_bfloat16*>(T_bf16),
                            static_cast<cudaStream_t>(stream), act_bits, t_pair != 0);
}

int aser_linear_w4a8_lr(const int8_t* Xq, const float* a_scale, const void* Wk,
                        const float* w_scale, const void* T_bf16, const void* LB_f16, int M, int N,
                        int K, int r, void* Y_f16, int32_t* acc_debug, void* workspace,
                        size_t workspace_bytes, void* stream) {
    return linear_common(Xq, a_scale, Wk, w_scale, T_bf16, LB_f16, M, N, K, r, Y_f16, acc_debug,
                         workspace, workspace_bytes, stream);
}

int aser_linear_w4a8(const int8_t* Xq, const float* a_scale, const void* Wk, const float* w_scale,
                     int M, int N, int K, void* Y_f16, int32_t* acc_debug, void* workspace,
                     size_t workspace_bytes, void* stream) {
    return linear_common(Xq, a_scale, Wk, w_scale, nullptr, nullptr, M, N, K, 0, Y_f16, acc_debug,
                         workspace, workspace_bytes, stream);
}

int aser_linear_w4a8_lr_simt(const int8_t* Xq, const float* a_scale, const uint8_t* Wq,
                             const float* w_scale, const void* T_bf16, const void* LB_f16, int M,
                             int N, int K, int r, void* Y_f16, int32_t* acc_debug, void* stream) {
    if (!shape_ok(M, N, K, r)) return fail(ASER_ERR_SHAPE, "unsupported M, N, K or r");
    if (M == 0 || N == 0) return ASER_OK;
    ASER_REQUIRE_PTR(Xq);
    ASER_REQUIRE_PTR(a_scale);
    ASER_REQUIRE_PTR(Wq);
    ASER_REQUIRE_PTR(w_scale);
    ASER_REQUIRE_PTR(Y_f16);
    ASER_OPTIONAL_PTR(acc_debug);
    if (r > 0) {
        ASER_REQUIRE_PTR(T_bf16);
        ASER_REQUIRE_PTR(LB_f16);
    }
    int rc = check_device();
    if (rc != ASER_OK) return rc;
    return launch_linear_simt(Xq, a_scale, Wq, w_scale, static_cast<const __nv_bfloat16*>(T_bf16),
                              static_cast<const __half*>(LB_f16), M, N, K, r,
                              static_cast<__half*>(Y_f16), acc_debug,
                              static_cast<cudaStream_t>(stream));
}

size_t aser_construct_workspace_bytes(int N, int K, int n_cal, int r, int n_split) {
    if (!shape_ok(0, N, K, r) || N <= 0 || n_cal <= 0 || n_split < 0) return 0;
    return construct_workspace_bytes(N, K, n_cal, r, n_split);
}

int aser_construct(const void* W_f16, const float* s, const void* Xcal_f16, int N, int K, int n_cal, int r,
                   double damping, int iterations, uint8_t* Wq, float* w_scale, void* LA_f16,
                   void* LB_f16, double* sigma_out, double* S_out, const int32_t* split_idx, int n_split,
                   void* workspace, size_t workspace_bytes, void* stream) {
    if (!shape_ok(0, N, K, r) || N <= 0 || n_cal <= 0 || r > (N < K ? N : K))
        return fail(ASER_ERR_SHAPE, "unsupported N, K, n_cal or r");
    if (!(damping > 0.0)) return fail(ASER_ERR_SHAPE, "damping must be positive");
    if (n_split < 0 || n_split > K) return fail(ASER_ERR_SHAPE, "n_split out of range");
    if (n_split > 0 && split_idx == nullptr) return fail(ASER_ERR_NULL, "split_idx is NULL");
    ASER_REQUIRE_PTR(W_f16);
    ASER_OPTIONAL_PTR(s);
    ASER_REQUIRE_PTR(Xcal_f16);
    ASER_REQUIRE_PTR(Wq);
    ASER_REQUIRE_PTR(w_scale);
    if (r > 0) {
        ASER_REQUIRE_PTR(LA_f16);
        ASER_REQUIRE_PTR(LB_f16);
    }
    ASER_OPTIONAL_PTR(sigma_out);
    ASER_OPTIONAL_PTR(S_out);
    if (workspace == nullptr || misaligned16(workspace) ||
        workspace_bytes < aser_construct_workspace_bytes(N, K, n_cal, r, n_split))
        return fail(ASER_ERR_WORKSPACE, "workspace missing, misaligned or too small");
    int rc = check_device();
    if (rc != ASER_OK) return rc;
    return launch_construct(static_cast<const __half*>(W_f16), s, static_cast<const __half*>(Xcal_f16), N, K,
                            n_cal, r, damping, iterations > 0 ? iterations : 48, Wq, w_scale,
                            static_cast<__half*>(LA_f16), static_cast<__half*>(LB_f16), sigma_out, S_out,
                            split_idx, n_split, workspace, static_cast<cudaStream_t>(stream));
}

size_t aser_workspace_bytes(int M, int N, int K, int r) {
    if (!shape_ok(M, N, K, r)) return 0;
    const size_t lin = kWsHeaderBytes + linear_tc_workspace_bytes(M, N, K, r);
    const size_t act = aser_quant_workspace_bytes(M, K, r);
    return lin > act ? lin : act;
}

size_t aser_quant_workspace_bytes(int M, int K, int r) {
    if (!act_shape_ok(M, K, r)) return 0;
    return kWsZeroedBytes + quant_act_ws_scratch_bytes(M, K, r);
}

int aser_quant_act_ws_launches(int M, int K) {
    if (!act_shape_ok(M, K, 0) || M == 0) return 0;
    return quant_act_ws_launches(M, K);
}

int aser_quant_act_ws(const void* X_f16, const float* s, const void* LA_f16, int M, int K, int r,
                      int act_bits, int t_pair, int8_t* Xq, float* a_scale, void* T_bf16,
                      void* workspace, size_t workspace_bytes, void* stream) {
    if (!act_shape_ok(M, K, r)) return fail(ASER_ERR_SHAPE, "unsupported M, K or r");
    if (act_bits < 2 || act_bits > 8) return fail(ASER_ERR_SHAPE, "act_bits must be 2..8");
    if (t_pair != 0 && t_pair != 1) return fail(ASER_ERR_SHAPE, "t_pair must be 0 or 1");
    if (t_pair && 2 * r > 512) return fail(ASER_ERR_SHAPE, "t_pair needs 2 r <= 512");
    if (M == 0) return ASER_OK;
    ASER_REQUIRE_PTR(X_f16);
    ASER_OPTIONAL_PTR(s);
    ASER_REQUIRE_PTR(Xq);
    ASER_REQUIRE_PTR(a_scale);
    if (r > 0) {
        ASER_REQUIRE_PTR(LA_f16);
        ASER_REQUIRE_PTR(T_bf16);
    }
    if (workspace == nullptr || misaligned16(workspace) ||
        workspace_bytes < aser_quant_workspace_bytes(M, K, r))
        return fail(ASER_ERR_WORKSPACE, "workspace missing, misaligned or too small");
    int rc = check_device();
    if (rc != ASER_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (M <= 32)
        return launch_quant_act(static_cast<const __half*>(X_f16), s, static_cast<const __half*>(LA_f16), M, K, r,
                                Xq, a_scale, static_cast<__nv_bfloat16*>(T_bf16), st, act_bits, t_pair != 0);
    return launch_quant_act_ws(static_cast<const __half*>(X_f16), s, static_cast<const __half*>(LA_f16), M, K, r,
                               Xq, a_scale, static_cast<__nv_bfloat16*>(T_bf16),
                               static_cast<uint8_t*>(workspace) + kWsZeroedBytes,
                               workspace_bytes - kWsZeroedBytes, st, act_bits, t_pair != 0);
}

int aser_forward_act_launches(int M, int K, int r) {
    if (!act_shape_ok(M, K, r) || M == 0) return 0;
    return forward_act_uses_scratch(M, K, r) ? quant_act_ws_launches(M, K) : 1;
}

int aser_linear_w4a8_lr_ld(const int8_t* Xq, const float* a_scale, const void* Wk,
                           const float* w_scale, const void* T_bf16, int ldt, const void* LB_f16,
                           int M, int N, int K, int r, void* Y_f16, int32_t* acc_debug,
                           void* workspace, size_t workspace_bytes, void* stream) {
    return linear_common(Xq, a_scale, Wk, w_scale, T_bf16, LB_f16, M, N, K, r, Y_f16, acc_debug,
                         workspace, workspace_bytes, stream, false, ldt);
}

size_t aser_forward_shared_workspace_bytes(int n_layers, const int* N, const int* r, int M, int K) {
    if (n_layers < 1 || N == nullptr || r == nullptr) return 0;
    int r_total = 0;
    size_t need = 0;
    for (int l = 0; l < n_layers; ++l) {
        if (!shape_ok(M, N[l], K, r[l])) return 0;
        r_total += r[l];
        const size_t lin = kWsHeaderBytes + linear_tc_workspace_bytes(M, N[l], K, r[l]);
        if (lin > need) need = lin;
    }
    const size_t act = aser_quant_workspace_bytes(M, K, r_total);
    if (act == 0) return 0;
    return act > need ? act : need;
}

int aser_forward_shared(const void* X_f16, const float* s, const void* LA_stacked_f16, int n_layers,
                        const void* const* Wk, const float* const* w_scale, const void* const* LB_f16,
                        const int* N, const int* r, int M, int K, int8_t* Xq, float* a_scale,
                        void* T_bf16, void* const* Y_f16, void* workspace, size_t workspace_bytes,
                        void* stream) {
    if (n_layers < 1 || n_layers > 16) return fail(ASER_ERR_SHAPE, "n_layers must be 1..16");
    if (Wk == nullptr || w_scale == nullptr || LB_f16 == nullptr || N == nullptr || r == nullptr ||
        Y_f16 == nullptr)
        return fail(ASER_ERR_NULL, "a per-layer array is NULL");
    const size_t need = aser_forward_shared_workspace_bytes(n_layers, N, r, M, K);
    if (need == 0) return fail(ASER_ERR_SHAPE, "unsupported M, N, K or r (stacked ranks go up to 512)");
    if (M == 0) return ASER_OK;
    int r_total = 0;
    for (int l = 0; l < n_layers; ++l) r_total += r[l];
    // every argument of every launch is checked before the first one is enqueued
    ASER_REQUIRE_PTR(X_f16);
    ASER_OPTIONAL_PTR(s);
    ASER_REQUIRE_PTR(Xq);
    ASER_REQUIRE_PTR(a_scale);
    if (r_total > 0) {
        ASER_REQUIRE_PTR(LA_stacked_f16);
        ASER_REQUIRE_PTR(T_bf16);
    }
    for (int l = 0; l < n_layers; ++l) {
        if (N[l] == 0) continue;
        ASER_REQUIRE_PTR(Wk[l]);
        ASER_REQUIRE_PTR(w_scale[l]);
        ASER_REQUIRE_PTR(Y_f16[l]);
        if (r[l] > 0) ASER_REQUIRE_PTR(LB_f16[l]);
    }
    if (workspace == nullptr || misaligned16(workspace) || workspace_bytes < need)
        return fail(ASER_ERR_WORKSPACE, "workspace missing, misaligned or too small");
    int rc = check_device();
    if (rc != ASER_OK) return rc;
    for (int l = 0; l < n_layers; ++l)
        if (N[l] > 0 && !linear_decode_prefers(M, N[l], K)) {
            rc = linear_tc_check(M, N[l], K, r[l], workspace_bytes);
            if (rc != ASER_OK) return rc;
        }
    rc = quant_with_workspace(X_f16, s, LA_stacked_f16, M, K, r_total, 8, false, Xq, a_scale, T_bf16,
                              workspace, workspace_bytes, stream);
    if (rc != ASER_OK) return rc;
    int col = 0;
    for (int l = 0; l < n_layers; ++l) {
        const void* Tl = r[l] > 0 ? static_cast<const void*>(static_cast<const __nv_bfloat16*>(T_bf16) + col) : nullptr;
        rc = linear_common(Xq, a_scale, Wk[l], w_scale[l], Tl, r[l] > 0 ? LB_f16[l] : nullptr, M, N[l], K,
                           r[l], Y_f16[l], nullptr, workspace, workspace_bytes, stream,
                           /*overlap_prev=*/l == 0, r_total);
        if (rc != ASER_OK) return rc;
        col += r[l];
    }
    return ASER_OK;
}

// The layers of a shared-input group stored one after the other along N (weights, scales, L_B and
// the columns of Y), all of one rank: bounds for the kernels, or an error text.
static const char* cat_split_of(int n_layers, const int* N, int r, int* n_total, CatSplit* cat) {
    if (n_layers < 1 || n_layers > 4) return "n_layers must be 1..4";
    if (N == nullptr) return "N is NULL";
    long long total = 0;
    int bound[4] = {0x7fffffff, 0x7fffffff, 0x7fffffff, 0x7fffffff};
    for (int l = 0; l < n_layers; ++l) {
        if (N[l] <= 0 || N[l] % 128 != 0) return "every layer's N must be a positive multiple of 128";
        total += N[l];
        if (l + 1 < n_layers) bound[l] = (int)total;
    }
    if (total > 0x7fffffff || (long long)r * n_layers > 512) return "stacked sizes out of range";
    *n_total = (int)total;
    cat->layers = n_layers;
    cat->b1 = bound[0]; cat->b2 = bound[1]; cat->b3 = bound[2];
    return nullptr;
}

int aser_linear_w4a8_lr_cat(const int8_t* Xq, const float* a_scale, const void* Wk_cat, const float* w_scale_cat,
                            const void* T_bf16, const void* LB_cat_f16, int n_layers, const int* N, int r,
                            int M, int K, void* Y_cat_f16, void* workspace, size_t workspace_bytes,
                            void* stream) {
    int n_total = 0;
    CatSplit cat;
    const char* why = cat_split_of(n_layers, N, r, &n_total, &cat);
    if (why) return fail(ASER_ERR_SHAPE, why);
    return linear_common(Xq, a_scale, Wk_cat, w_scale_cat, T_bf16, LB_cat_f16, M, n_total, K, r, Y_cat_f16,
                         nullptr, workspace, workspace_bytes, stream, false, r * n_layers, cat);
}

size_t aser_forward_shared_cat_workspace_bytes(int n_layers, const int* N, int r, int M, int K) {
    int n_total = 0;
    CatSplit cat;
    if (cat_split_of(n_layers, N, r, &n_total, &cat)) return 0;
    if (!shape_ok(M, n_total, K, r)) return 0;
    const size_t lin = kWsHeaderBytes + linear_tc_workspace_bytes(M, n_total, K, r);
    const size_t act = aser_quant_workspace_bytes(M, K, r * n_layers);
    if (act == 0) return 0;
    return act > lin ? act : lin;
}

int aser_forward_shared_cat(const void* X_f16, const float* s, const void* LA_stacked_f16, int n_layers,
                            const void* Wk_cat, const float* w_scale_cat, const void* LB_cat_f16,
                            const int* N, int r, int M, int K, int8_t* Xq, float* a_scale, void* T_bf16,
                            void* Y_cat_f16, void* workspace, size_t workspace_bytes, void* stream) {
    int n_total = 0;
    CatSplit cat;
    const char* why = cat_split_of(n_layers, N, r, &n_total, &cat);
    if (why) return fail(ASER_ERR_SHAPE, why);
    const size_t need = aser_forward_shared_cat_workspace_bytes(n_layers, N, r, M, K);
    if (need == 0) return fail(ASER_ERR_SHAPE, "unsupported M, N, K or r (stacked ranks go up to 512)");
    if (M == 0) return ASER_OK;
    const int r_total = r * n_layers;
    // every argument of both launches is checked before the first one is enqueued
    ASER_REQUIRE_PTR(X_f16);
    ASER_OPTIONAL_PTR(s);
    ASER_REQUIRE_PTR(Xq);
    ASER_REQUIRE_PTR(a_scale);
    ASER_REQUIRE_PTR(Wk_cat);
    ASER_REQUIRE_PTR(w_scale_cat);
    ASER_REQUIRE_PTR(Y_cat_f16);
    if (r > 0) {
        ASER_REQUIRE_PTR(LA_stacked_f16);
        ASER_REQUIRE_PTR(T_bf16);
        ASER_REQUIRE_PTR(LB_cat_f16);
    }
    if (workspace == nullptr || misaligned16(workspace) || workspace_bytes < need)
        return fail(ASER_ERR_WORKSPACE, "workspace missing, misaligned or too small");
    int rc = check_device();
    if (rc != ASER_OK) return rc;
    if (!linear_decode_prefers(M, n_total, K)) {
        rc = linear_tc_check(M, n_total, K, r, workspace_bytes);
        if (rc != ASER_OK) return rc;
    }
    rc = quant_with_workspace(X_f16, s, LA_stacked_f16, M, K, r_total, 8, false, Xq, a_scale, T_bf16,
                              workspace, workspace_bytes, stream);
    if (rc != ASER_OK) return rc;
    return linear_common(Xq, a_scale, Wk_cat, w_scale_cat, r > 0 ? T_bf16 : nullptr, r > 0 ? LB_cat_f16 : nullptr,
                         M, n_total, K, r, Y_cat_f16, nullptr, workspace, workspace_bytes, stream,
                         /*overlap_prev=*/true, r_total, cat);
}

int aser_workspace_init(void* workspace, size_t workspace_bytes, void* stream) {
    if (workspace == nullptr || misaligned16(workspace) || workspace_bytes < kWsHeaderBytes)
        return fail(ASER_ERR_WORKSPACE, "workspace missing, misaligned or too small");
    cudaError_t e = cudaMemsetAsync(workspace, 0, workspace_bytes, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return record_cuda_error(e, "cudaMemsetAsync(workspace)");
    return ASER_OK;
}

int aser_check_status(void* workspace, void* stream) {
    if (workspace == nullptr) return fail(ASER_ERR_WORKSPACE, "workspace is NULL");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint32_t word = 0;
    cudaError_t e = cudaMemcpyAsync(&word, workspace, sizeof(word), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return record_cuda_error(e, "aser_check_status");
    if (word == 0) return ASER_OK;
    // a launch that gave up may also have left tile counters behind: clear them with the word
    e = cudaMemsetAsync(workspace, 0, kWsZeroedBytes, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return record_cuda_error(e, "aser_check_status clear");
    snprintf(g_last_error, sizeof(g_last_error),
             "a bounded device-side wait gave up (status word 0x%08x)", word);
    return ASER_ERR_DEVICE_TIMEOUT;
}

// Every check aser_forward makes, with nothing enqueued: the arguments of both launches and the
// linear kernel's own range checks.
static int forward_validate(const void* X_f16, const float* s, const void* LA_f16, const void* Wk,
                            const float* w_scale, const void* LB_f16, int M, int N, int K, int r,
                            const int8_t* Xq, const float* a_scale, const void* T_bf16,
                            const void* Y_f16, const void* workspace, size_t workspace_bytes) {
    ASER_REQUIRE_PTR(X_f16);
    ASER_OPTIONAL_PTR(s);
    ASER_REQUIRE_PTR(Xq);
    ASER_REQUIRE_PTR(a_scale);
    ASER_REQUIRE_PTR(Wk);
    ASER_REQUIRE_PTR(w_scale);
    ASER_REQUIRE_PTR(Y_f16);
    if (r > 0) {
        ASER_REQUIRE_PTR(LA_f16);
        ASER_REQUIRE_PTR(T_bf16);
        ASER_REQUIRE_PTR(LB_f16);
    }
    if (workspace == nullptr || misaligned16(workspace) ||
        workspace_bytes < aser_workspace_bytes(M, N, K, r))
        return fail(ASER_ERR_WORKSPACE, "workspace missing, misaligned or too small");
    int rc = check_device();
    if (rc != ASER_OK) return rc;
    if (!linear_decode_prefers(M, N, K)) rc = linear_tc_check(M, N, K, r, workspace_bytes);
    return rc;
}

int aser_forward(const void* X_f16, const float* s, const void* LA_f16, const void* Wk,
                 const float* w_scale, const void* LB_f16, int M, int N, int K, int r,
                 int8_t* Xq, float* a_scale, void* T_bf16, void* Y_f16, void* workspace,
                 size_t workspace_bytes, void* stream) {
    if (!shape_ok(M, N, K, r)) return fail(ASER_ERR_SHAPE, "unsupported M, N, K or r");
    if (M == 0 || N == 0) return ASER_OK;
    int rc = forward_validate(X_f16, s, LA_f16, Wk, w_scale, LB_f16, M, N, K, r, Xq, a_scale, T_bf16,
                              Y_f16, workspace, workspace_bytes);
    if (rc != ASER_OK) return rc;
    rc = quant_with_workspace(X_f16, s, LA_f16, M, K, r, 8, false, Xq, a_scale, T_bf16, workspace,
                              workspace_bytes, stream);
    if (rc != ASER_OK) return rc;
    return linear_common(Xq, a_scale, Wk, w_scale, r > 0 ? T_bf16 : nullptr, r > 0 ? LB_f16 : nullptr,
                         M, N, K, r, Y_f16, nullptr, workspace, workspace_bytes, stream,
                         /*overlap_prev=*/true);
}

int aser_forward_host(const void* X_host_f16, void* Y_host_f16, void* X_dev, int8_t* Xq_dev,
                      float* a_scale_dev, void* T_dev, void* Y_dev, const float* s,
                      const void* LA_f16, const void* Wk, const float* w_scale, const void* LB_f16,
                      int M, int N, int K, int r, void* workspace, size_t workspace_bytes,
                      void* stream) {
    if (!shape_ok(M, N, K, r)) return fail(ASER_ERR_SHAPE, "unsupported M, N, K or r");
    if (M == 0 || N == 0) return ASER_OK;
    if (X_host_f16 == nullptr || Y_host_f16 == nullptr)
        return fail(ASER_ERR_NULL, "host buffer is NULL");
    // everything is checked before the first copy is enqueued
    int rc = forward_validate(X_dev, s, LA_f16, Wk, w_scale, LB_f16, M, N, K, r, Xq_dev, a_scale_dev,
                              T_dev, Y_dev, workspace, workspace_bytes);
    if (rc != ASER_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(X_dev, X_host_f16, (size_t)M * K * 2, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return record_cuda_error(e, "copy X to device");
    rc = aser_forward(X_dev, s, LA_f16, Wk, w_scale, LB_f16, M, N, K, r, Xq_dev, a_scale_dev,
                      T_dev, Y_dev, workspace, workspace_bytes, stream);
    if (rc != ASER_OK) return rc;
    e = cudaMemcpyAsync(Y_host_f16, Y_dev, (size_t)M * N * 2, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return record_cuda_error(e, "copy Y to host");
    return ASER_OK;
}

}  // extern "C"
