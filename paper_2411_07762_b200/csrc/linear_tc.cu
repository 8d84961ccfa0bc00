// placeholder: replaced by the tcgen05 kernel
#include "aser_common.cuh"
namespace aser {
size_t linear_tc_workspace_bytes(int, int, int, int) { return 0; }
int launch_linear_tc(const int8_t*, const float*, const uint8_t*, const float*, const __nv_bfloat16*,
                     const __half*, int, int, int, int, __half*, int32_t*, void*, size_t, cudaStream_t) {
    return ASER_ERR_SHAPE;
}
}
