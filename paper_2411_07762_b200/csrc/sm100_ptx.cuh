// PTX wrappers for the sm_100a asynchronous machinery (mbarrier, bulk and tensor copies,
// tcgen05 tensor-core instructions and tensor memory) and the host-side tensor-map encoder.
// Shared by the kernels that use them; everything here is inline.
#pragma once
#include <cuda.h>
#include <string.h>

#include "aser_common.cuh"

namespace aser {

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void* src, uint32_t bytes,
                                              uint32_t bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y,
                                            uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z,
                                            uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}
// Programmatic dependent launch.  `grid_dep_wait` returns once the kernels this launch depends
// on have completed and their writes are visible (at once when the launch has no such
// dependency); `grid_dep_launch` lets a dependent kernel start its own preamble early.
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async_smem() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before() {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                 ::"r"(bar)
                 : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem desc], int8 x int8 -> int32
__device__ __forceinline__ void mma_i8_ts(uint32_t d, uint32_t a, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d), "r"(a), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// D[tmem] (+)= A[smem desc] * B[smem desc], fp16 x fp16 -> fp32
__device__ __forceinline__ void mma_f16_ss(uint32_t d, uint64_t adesc, uint64_t bdesc,
                                           uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
        "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]),
        "r"(v[7]), "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]),
        "r"(v[14]), "r"(v[15]), "r"(v[16]), "r"(v[17]), "r"(v[18]), "r"(v[19]), "r"(v[20]),
        "r"(v[21]), "r"(v[22]), "r"(v[23]), "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]),
        "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
        : "memory");
}
// Zero 16 consecutive columns of this warp's 32 lanes.
__device__ __forceinline__ void tmem_zero16(uint32_t taddr) {
    const uint32_t z = 0;
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1};"
        ::"r"(taddr), "r"(z)
        : "memory");
}
__device__ __forceinline__ void tmem_wait_st() {
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]),
          "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]),
          "=r"(v[14]), "=r"(v[15])
        : "r"(taddr)
        : "memory");
}
// Waits for the tensor-memory loads; the registers are listed as in/out operands so that no
// use of them can be scheduled ahead of the wait.
__device__ __forceinline__ void tmem_wait_ld(uint32_t (&v)[16]) {
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]),
                   "+r"(v[7]), "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]),
                   "+r"(v[13]), "+r"(v[14]), "+r"(v[15])
                 :
                 : "memory");
}
// Barrier over `count` threads that also ANDs a predicate across them.
__device__ __forceinline__ bool named_bar_all(int id, int count, bool pred) {
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.b32 p, %3, 0;\n\t"
        "barrier.cta.red.and.pred q, %1, %2, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(out)
        : "r"(id), "r"(count), "r"((uint32_t)pred)
        : "memory");
    return out != 0;
}
__device__ __forceinline__ void named_bar_sync(int id, int count) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of 128 bytes,
// groups of 8 rows 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);        // start address
    d |= (uint64_t)(1024u >> 4) << 32;              // stride between 8-row groups
    d |= 1ull << 46;                                // descriptor version of this architecture
    d |= 2ull << 61;                                // 128-byte swizzle
    return d;
}

// Instruction descriptor: dense, D format (1 = f32, 2 = s32), A/B format, K-major both, N, M.
__host__ __device__ constexpr uint32_t make_idesc(uint32_t dfmt, uint32_t abfmt, uint32_t M,
                                                  uint32_t N) {
    return (dfmt << 4) | (abfmt << 7) | (abfmt << 10) | ((N >> 3) << 17) | ((M >> 4) << 24);
}

// ---------------------------------------------------------------------------
// host side: tensor maps
// ---------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (fn) return fn;
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || ptr == nullptr) return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(ptr);
    return fn;
}

// A tensor map depends only on the address, shape, strides, box and modes it was encoded for,
// never on the tensor's contents, so a map encoded once can serve every later launch with the
// same arguments.  encode_tiled keeps the most recent maps of the calling thread in a small
// direct-mapped table (a layer's buffers come back call after call) and spares the hot path the
// driver's encoder.
struct MapKey {
    const void* base;
    uint64_t dims[3];
    uint64_t strides[2];
    uint32_t box[3];
    uint32_t dtype, rank, swizzle;
};

inline int encode_tiled(CUtensorMap* map, const MapKey& key, const char* what) {
    struct Entry { MapKey key; CUtensorMap map; bool used; };
    constexpr int kEntries = 256;
    static thread_local Entry table[kEntries];
    uint64_t h = 1469598103934665603ull;
    const unsigned char* kb = reinterpret_cast<const unsigned char*>(&key);
    for (size_t i = 0; i < sizeof(MapKey); ++i) h = (h ^ kb[i]) * 1099511628211ull;
    Entry& e = table[(h ^ (h >> 32)) % kEntries];
    if (e.used && memcmp(&e.key, &key, sizeof(MapKey)) == 0) { *map = e.map; return ASER_OK; }
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return record_cuda_error(cudaErrorUnknown, "cuTensorMapEncodeTiled unavailable");
    cuuint64_t dims[3] = {key.dims[0], key.dims[1], key.dims[2]};
    cuuint64_t strides[2] = {key.strides[0], key.strides[1]};
    cuuint32_t box[3] = {key.box[0], key.box[1], key.box[2]};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(map, (CUtensorMapDataType)key.dtype, key.rank, const_cast<void*>(key.base), dims,
                    strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, (CUtensorMapSwizzle)key.swizzle,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return record_cuda_error(cudaErrorInvalidValue, what);
    e.key = key; e.map = *map; e.used = true;
    return ASER_OK;
}

inline MapKey make_key(const void* base, CUtensorMapDataType dt, uint32_t rank, CUtensorMapSwizzle sw) {
    MapKey k;
    memset(&k, 0, sizeof(k));       // padding bytes take part in the comparison
    k.base = base; k.dtype = (uint32_t)dt; k.rank = rank; k.swizzle = (uint32_t)sw;
    return k;
}

// 2-D row-major tensor [rows, cols] of `esize`-byte elements whose rows are `ld` elements apart
// (a column range of a wider matrix), box = [box_rows, box_cols] with the given shared-memory
// swizzle; out-of-range elements read as zero and are not written.
inline int encode_map_2d_ld(CUtensorMap* map, CUtensorMapDataType dt, int esize, const void* base,
                            uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_rows,
                            uint32_t box_cols, CUtensorMapSwizzle swizzle) {
    MapKey k = make_key(base, dt, 2, swizzle);
    k.dims[0] = cols; k.dims[1] = rows;
    k.strides[0] = ld * (uint64_t)esize;
    k.box[0] = box_cols; k.box[1] = box_rows;
    return encode_tiled(map, k, "cuTensorMapEncodeTiled");
}

// The same with contiguous rows.
inline int encode_map_2d(CUtensorMap* map, CUtensorMapDataType dt, int esize, const void* base,
                         uint64_t rows, uint64_t cols, uint32_t box_rows, uint32_t box_cols,
                         CUtensorMapSwizzle swizzle) {
    return encode_map_2d_ld(map, dt, esize, base, rows, cols, cols, box_rows, box_cols, swizzle);
}

// Row-major tensor [rows, cols] of `esize`-byte elements viewed as 128-byte column blocks:
// [cols * esize / 128 blocks][rows][128 bytes].  A box takes `box_blocks` blocks x `box_rows` rows,
// 128-byte swizzle; in shared memory each block's rows are contiguous (the K-major operand layout
// of the MMA descriptors).  Coordinates: (0, row, block).
inline int encode_map_blocks(CUtensorMap* map, CUtensorMapDataType dt, int esize, const void* base,
                             uint64_t rows, uint64_t cols, uint32_t box_rows, uint32_t box_blocks) {
    const uint64_t per_block = 128 / (uint64_t)esize;
    MapKey k = make_key(base, dt, 3, CU_TENSOR_MAP_SWIZZLE_128B);
    k.dims[0] = per_block; k.dims[1] = rows; k.dims[2] = cols / per_block;
    k.strides[0] = cols * (uint64_t)esize; k.strides[1] = 128;
    k.box[0] = (uint32_t)per_block; k.box[1] = box_rows; k.box[2] = box_blocks;
    return encode_tiled(map, k, "cuTensorMapEncodeTiled (blocks)");
}

}  // namespace aser
