// Tensor-core kernel of the ASER linear (Sec. 4.2, "W_q X + L_A L_B X"):
//   acc = Xq Wq^T (int8 x int4 -> int32),  Y = fp16(acc * a_scale[m] * w_scale[n] + T L_B^T).
//
// Orientation: the output tile is computed transposed, D[n, token], so that the WEIGHTS sit on
// the MMA's M side.  Packed int4 weights are streamed from HBM with bulk copies into shared
// memory, turned into int8 (value 16*q) by two ALU operations per eight codes, and written
// straight into TENSOR MEMORY as the A operand of tcgen05.mma kind::i8; they never go back to
// shared memory.  The int8 activations arrive by TMA (128-byte swizzle) as the B operand, so the
// MMA N dimension is the token tile (16..128) and decode shapes use the same kernel.
// The low-rank term is a second accumulator fed by kind::f16 MMAs on L_B (TMA) and T (TMA, then
// bf16 -> fp16 in place).  Work is split stream-K style: the list of (tile, 128-column block)
// units is cut into equal contiguous ranges, one per CTA; tiles shared by several CTAs are
// summed through the workspace by whichever CTA arrives last.
//
// Warp roles (512 threads for token tiles of 16/32, 640 above): 0 = weight producer, 1 and the
// last warp = MMA issuers for even / odd stages (1 also owns the TMEM allocation and issues the
// low-rank MMAs), 2..5 and 6..9 = two groups of int4 -> int8 unpack warps that take alternate
// stages (group 0 also converts T), then 4 or 8 epilogue warps (two per tensor-memory lane
// quarter take alternate 16-column chunks), then the activation / low-rank operand producer.
// A single lane issues one tcgen05.mma per ~60-85 cycles, which bounds decode shapes (16 MMAs
// per 32 KiB of weights); the integer accumulation is order-independent, so two lanes share the
// issue work.  For that the accumulator is zeroed by the epilogue warps (tcgen05.st) when they
// hand it back, and every integer MMA accumulates.
// Every wait is bounded: on expiry the CTA sets the status word and winds down.
#include "aser_common.cuh"
#include "sm100_ptx.cuh"

namespace aser {

namespace {

constexpr int kMaxCtas = 160;     // upper bound on the persistent grid (workspace sizing)
constexpr uint32_t kStatusTimeout = 1u;
constexpr long long kWaitLimitClocks = 400000000ll;  // about 0.2 s of SM clocks per wait

// Per token-tile configuration.  A pipeline stage carries KS 128-column blocks: one bulk copy of
// KS x 8 KiB of packed weights, one TMA box of KS activation tiles, KS x 32 tensor-memory columns
// of unpacked A operand.  Under copy traffic every mbarrier operation costs a thread a few
// hundred cycles, so stages are made large (few waits, arrivals, copy issues and commits per
// byte) and the unpack work alternates between two groups of four warps.
template <int BT>
struct Cfg {
    // Epilogue warps: one per tensor-memory lane quarter, two where a tile has many columns.
    static constexpr int EW = (BT >= 64) ? 8 : 4;
    static constexpr int EpiThreads = EW * 32;
    static constexpr int WarpXProd = 10 + EW, WarpIssuer1 = 11 + EW;
    static constexpr int Threads = (12 + EW) * 32;
    static constexpr int KS = 2;
    static constexpr int NW = (BT == 128) ? 4 : (BT == 64 ? 6 : 8);     // weight ring depth (even)
    static constexpr int NX = 4;                                        // activation ring depth
    // A-operand ring (tensor memory).  All ring depths are even: stages alternate between two
    // unpack groups and two MMA issuers, and a parity wait is only sound if the waiter sees every
    // phase of the barrier, i.e. if a ring slot always belongs to the same group.
    // An A slot holds KA column blocks.  With 128 tokens only 128 tensor-memory columns are left
    // for A, so a slot is one block there: each group then still owns two slots and can unpack
    // one block while the MMAs of the other are in flight.
    static constexpr int KA = (BT == 128) ? 1 : KS;
    static constexpr int SPS = KS / KA;                                 // A slots per stage
    static constexpr int NA = 4;
    static_assert(NA % (2 * SPS) == 0 && NW % 2 == 0 && NX % 2 == 0, "ring ownership");
    // ring of low-rank chunks (64 columns of r each); one slot where shared memory is tight
    static constexpr int NL = (BT == 128) ? 1 : 2;
    static constexpr int WBytes = KS * kWkBlockBytes;
    static constexpr int XTile = BT * 128;                              // one 128-column block of Xq
    static constexpr int XBytes = KS * XTile;
    static constexpr int LbBytes = 128 * 128;          // 128 rows x 64 fp16
    static constexpr int TBytes = BT * 128;            // BT rows x 64 bf16/fp16
    static constexpr int OffW = 0;
    static constexpr int OffX = OffW + NW * WBytes;
    static constexpr int OffLb = OffX + NX * XBytes;
    static constexpr int OffT = OffLb + NL * LbBytes;
    static constexpr int OffBar = OffT + NL * TBytes;
    static constexpr int NumBars = 2 * NW + 2 * NX + 2 * NA + 3 * NL + 2 + 2 + 2;
    // Who issues the low-rank MMAs.  The two integer issuers spend nine tenths of their time
    // inside barrier and tensor-core instructions (a wait, MMA or commit costs its thread a few
    // hundred cycles under copy traffic), so every operation of a low-rank chunk on one of them
    // sets it back against the other and the whole pipeline with it.  A warp of its own for the
    // job costs every thread 16 registers (21 warps: six on one scheduler); a second lane of the
    // producer's warp as a third issuer measured the same as what is done here and leans on how the
    // hardware shares a warp between two diverged spinning lanes.  So, with the one-slot chunk
    // ring, the thread that loads the chunks also multiplies them: it runs a few stages ahead of
    // the MMAs, has slack, polls the chunk's barriers between its activation stages, and waits for
    // them only where nothing it still has to do is needed for them to complete (after the last
    // activation stage of the item).  For the same reason no other role waits for a chunk in
    // mid-tile: see the unpack warps.
    static constexpr bool ProducerLr = (NL == 1);
    static constexpr int SmemBytes = OffBar + NumBars * 8 + 128 + 1024;  // + slack for 1 KiB alignment
    static constexpr int ASlotCols = KA * 32;
    static constexpr int TmemColsUsed = 3 * BT + NA * ASlotCols;
    static constexpr int TmemCols = TmemColsUsed <= 256 ? 256 : 512;
    static_assert(TmemColsUsed <= 512, "tensor memory budget");
    static_assert(SmemBytes <= 227 * 1024, "shared memory budget");
};

// ---------------------------------------------------------------------------
// kernel parameters and work enumeration
// ---------------------------------------------------------------------------
struct Params {
    const uint8_t* Wk;
    const float* a_scale;
    const float* w_scale;
    __half* Y;
    int32_t* acc_debug;
    uint32_t* status;      // workspace word 0
    int* counters;         // one per CTA: a shared tile's counter is that of the CTA owning its first unit
    int32_t* part_int;     // [grid][2][BT][128]
    float* part_lr;        // [grid][BT][128]
    int M, N, K, r;
    int KB, TT, NT;        // 128-column blocks, token tiles, 128-row tiles
    int units;             // NT * TT * KB
    int tail_first;        // work order: 1 = both shared tiles first, 0 = range order
    int tt_outer;          // tile numbering: 1 = token tile outer (consecutive tiles share the activations)
    CatSplit cat;          // layers stacked along N: which columns of T a weight tile multiplies
};

struct Work {
    int tile, nt, tt, kb0, kb1;
    bool has_lr, whole;
};

// Units are numbered tile-major: unit = tile * KB + column block.  CTA c owns
// [range_begin(c), range_begin(c + 1)).  The unit count fits 31 bits (checked on the host).
__device__ __noinline__ int range_begin(int units, int c, int G) {
    return (int)((long long)units * c / G);
}
// CTA that owns unit x.
__device__ __noinline__ int unit_owner(int units, int x, int G) {
    return (int)((((long long)x + 1) * G - 1) / units);
}

// Cursor over a CTA's unit range.  The range is a tile cut off at its start (shared with the
// CTA before), whole tiles, and a tile cut off at its end (shared with the CTA after).  With
// Params::tail_first the two shared tiles come first: their cross-CTA reduction (atomic, and
// for the last arriver the sum over all contributors) then runs while the pipeline is busy with
// the whole tiles, instead of at the very end of the kernel where nothing hides it.  Otherwise
// the items come in range order.
struct Cursor {
    int first_tile, kb_b, last_tile, kb_e;   // range = [first_tile*KB + kb_b, last_tile*KB + kb_e)
    int phase;                               // 0: head part, 1: tail part, 2: whole tiles, 3: done
    int mid, mid_end;                        // whole tiles [mid, mid_end)
    __device__ __forceinline__ void init(int begin, int end, const Params& p) {
        if (begin >= end) { phase = 3; first_tile = last_tile = kb_b = kb_e = mid = mid_end = 0; return; }
        first_tile = begin / p.KB; kb_b = begin - first_tile * p.KB;
        last_tile = (end - 1) / p.KB; kb_e = end - last_tile * p.KB;
        phase = 0;
        mid = (kb_b != 0) ? first_tile + 1 : first_tile;
        mid_end = (kb_e != p.KB) ? last_tile : last_tile + 1;
    }
};

__device__ __forceinline__ void set_work(Work& w, const Params& p, int tile, int kb0, int kb1) {
    w.tile = tile; w.kb0 = kb0; w.kb1 = kb1;
    if (p.tt_outer) { w.tt = tile / p.NT; w.nt = tile - w.tt * p.NT; }
    else { w.nt = tile / p.TT; w.tt = tile - w.nt * p.TT; }
    w.has_lr = (kb0 == 0) && p.r > 0;
    w.whole = (kb0 == 0) && (kb1 == p.KB);
}

// Low-rank chunks inside a tile.  With a one-slot chunk ring (128-token tiles) and several chunks
// (r > 64), loading, converting and multiplying them one after the other at the END of a tile
// leaves the integer pipeline idle for a TMA round trip per chunk.  Where the tile is long enough
// all chunks but the last are therefore worked off in MID-TILE: chunk c is multiplied when stage
// lr_mma_stage(c) comes up (kLrSpacing stages per chunk, counted back from the end of the tile:
// a TMA round trip is three to four stages, conversion and MMAs one more) and converted two
// stages before; the slot is refilled as soon as those MMAs have retired, so the last chunk is
// in shared memory when the tile ends.  The first chunk can only be loaded once the previous
// tile's last chunk has been multiplied, i.e. around stage 4, hence the nine stages of head room.
// All three roles derive the schedule from the same numbers (stages of the work item, chunk
// count), so they agree without talking to each other.
constexpr int kLrSpacing = 5;
__device__ __forceinline__ bool lr_mid_tile(int ring_slots, bool has_lr, int chunks, int nst) {
    return ring_slots == 1 && has_lr && chunks >= 2 && nst >= 9 + kLrSpacing * (chunks - 1);
}
__device__ __forceinline__ int lr_mma_stage(int c, int chunks, int nst) {
    return nst - (chunks - 1 - c) * kLrSpacing;
}

// Next work item (the part of one tile inside this CTA's range).
__device__ __forceinline__ bool next_work(Cursor& c, const Params& p, Work& w) {
    if (c.phase == 0) {
        c.phase = 1;
        if (c.first_tile == c.last_tile) {          // the whole range lies inside one tile
            c.phase = 3;
            set_work(w, p, c.first_tile, c.kb_b, c.kb_e);
            return true;
        }
        if (c.kb_b != 0) { set_work(w, p, c.first_tile, c.kb_b, p.KB); return true; }
    }
    if (c.phase == 1) {
        c.phase = 2;
        if (p.tail_first && c.kb_e != p.KB) { set_work(w, p, c.last_tile, 0, c.kb_e); return true; }
    }
    if (c.phase == 2) {
        if (c.mid < c.mid_end) { set_work(w, p, c.mid, 0, p.KB); ++c.mid; return true; }
        c.phase = 3;
        if (!p.tail_first && c.kb_e != p.KB) { set_work(w, p, c.last_tile, 0, c.kb_e); return true; }
    }
    return false;
}

struct Abort {
    volatile int* flag;   // shared
    uint32_t* status;     // global
};

// Debugging aid: a role of the CTA whose wait gave up first leaves its progress counters in the
// workspace header (words 8 + 8 * role ...), read by the host after aser_check_status reports
// the time-out.
__device__ __noinline__ void dump_role(uint32_t* status, int role, uint32_t a, uint32_t b, uint32_t c,
                                       uint32_t d, uint32_t e) {
    for (int spin = 0; spin < 100000 && ((volatile uint32_t*)status)[5] == 0u; ++spin) {}
    if (((volatile uint32_t*)status)[2] != blockIdx.x) return;
    uint32_t* w = status + 8 + 6 * role;
    w[0] = 0xD0000000u | threadIdx.x; w[1] = a; w[2] = b; w[3] = c; w[4] = d; w[5] = e;
}

// Slow path of a bounded wait, kept out of line so that the role loops stay small (the kernel
// runs six different instruction streams per SM and lives or dies by its instruction cache).
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* flag,
                                            uint32_t* status) {
    uint32_t spins = 0;
    long long t0 = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 255u) == 0) {
            if (*flag) return false;
            if (t0 == 0) {
                t0 = clock64();
            } else if (clock64() - t0 > kWaitLimitClocks) {
                *flag = 1;
                atomicOr(status, kStatusTimeout);
                // where the first wait gave up (debugging aid): header words 1..5
                if (atomicCAS(status + 1, 0u, 0x80000000u | threadIdx.x) == 0u) {
                    status[2] = blockIdx.x;
                    status[3] = (bar & 1023u) >> 3;     // index of the barrier
                    status[4] = parity;
                    __threadfence();
                    status[5] = 1u;                     // record complete
                }
                return false;
            }
        }
    }
    return true;
}

// Bounded wait on an mbarrier phase.  Returns false after the time limit or when another role
// of this CTA has already given up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const Abort& ab) {
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, ab.flag, ab.status);
}

// Warp-collective form: lane 0 polls, the result is broadcast (which also re-converges the
// warp).  Keeps 31 of 32 lanes off the barrier unit, which every other role's waits share.
__device__ __forceinline__ bool warp_mbar_wait(uint32_t bar, uint32_t parity, const Abort& ab, int lane) {
    int ok = 1;
    if (lane == 0) ok = mbar_wait(bar, parity, ab) ? 1 : 0;
    return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

// Group-collective form for a 128-thread unpack group: a single lane polls the mbarrier and the
// outcome is spread by a hardware named barrier.  Keeps the mbarrier traffic of a group at one
// wait per event instead of four.
// The barrier numbers are literal (3 and 4) so that the kernel is known to use five hardware
// barriers, not all sixteen.
__device__ __forceinline__ bool group_bar_all(int group, bool pred) {
    return group == 0 ? named_bar_all(3, 128, pred) : named_bar_all(4, 128, pred);
}
__device__ __forceinline__ void group_bar_sync(int group) {
    if (group == 0) named_bar_sync(3, 128);
    else named_bar_sync(4, 128);
}
__device__ __forceinline__ bool group_mbar_wait(uint32_t bar, uint32_t parity, const Abort& ab,
                                                bool leader, int group) {
    bool ok = true;
    if (leader) ok = mbar_wait(bar, parity, ab);
    return group_bar_all(group, ok);
}

// ---------------------------------------------------------------------------
// the kernel
// ---------------------------------------------------------------------------
// MID: the mid-tile schedule for the low-rank chunks is compiled in (only useful, and only
// instantiated, for 128-token tiles with r > 64; the other variants keep their loops free of it).
template <int BT, bool MID>
__global__ void __launch_bounds__(Cfg<BT>::Threads, 1)
linear_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_lb,
                 const __grid_constant__ CUtensorMap map_t, const Params p) {
    using C = Cfg<BT>;
    constexpr int KS = C::KS;
    extern __shared__ uint8_t smem_raw[];
    // 1 KiB alignment for the swizzled tiles
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar0 = sbase + C::OffBar;
    auto bar = [&](int i) { return bar0 + 8u * i; };
    // barrier indices
    //   W_FULL[s]  weight bytes of stage landed (tx)          -> unpack warps
    //   W_FREE[s]  unpack warps have the weights in registers -> weight producer
    //   X_FULL[x]  activation bytes of stage landed (tx)      -> MMA issuer of the stage
    //   X_FREE[x]  MMAs of the stage retired (commit)         -> activation producer
    //   READY[a]   A operand of the stage written to tensor memory -> MMA issuer of the stage
    //   FREE[a]    MMAs of the stage retired (commit)         -> unpack warps
    //   FULL_LR / CONV_LR / EMPTY_LR[l]  low-rank chunk landed / converted / multiplied
    //   ACC_FULL / ACC_EMPTY[2]  integer accumulator complete / read and zeroed by the epilogue
    //   DLR_EMPTY  the epilogue has read the low-rank accumulator -> low-rank issuer
    //   LR_DONE    the item's low-rank MMAs retired (commit by the producer) -> epilogue
    constexpr int B_W_FULL = 0, B_W_FREE = B_W_FULL + C::NW, B_X_FULL = B_W_FREE + C::NW,
                  B_X_FREE = B_X_FULL + C::NX, B_READY = B_X_FREE + C::NX,
                  B_FREE = B_READY + C::NA, B_FULL_LR = B_FREE + C::NA,
                  B_CONV_LR = B_FULL_LR + C::NL, B_EMPTY_LR = B_CONV_LR + C::NL,
                  B_ACC_FULL = B_EMPTY_LR + C::NL, B_ACC_EMPTY = B_ACC_FULL + 2,
                  B_DLR_EMPTY = B_ACC_EMPTY + 2, B_LR_DONE = B_DLR_EMPTY + 1;
    static_assert(B_LR_DONE + 1 == C::NumBars, "barrier count");
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + C::OffBar + C::NumBars * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    int* last_flag = reinterpret_cast<int*>(tmem_slot + 2);
    volatile int* never_flag = reinterpret_cast<volatile int*>(tmem_slot + 3);  // stays 0
    constexpr int kMaxContrib = 12;
    int* contrib_slot = reinterpret_cast<int*>(tmem_slot + 4);                 // finalizer scratch

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = gridDim.x, cta = blockIdx.x;
    const int u_begin = range_begin(p.units, cta, G), u_end = range_begin(p.units, cta + 1, G);
    Abort ab{abort_flag, p.status};

    // Warp 0 initialises the barriers (one per lane and pass) and then only ARRIVES on the
    // start-up barrier, so that its lane 0 can begin streaming weights at once; every other warp
    // waits there until the barriers (and the tensor-memory allocation) are in place.
    if (warp == 0) {
        for (int i = lane; i < C::NumBars; i += 32) {
            const uint32_t count =
                (i == B_LR_DONE) ? 1u
                : (i >= B_ACC_EMPTY) ? (uint32_t)C::EW
                : (i >= B_ACC_FULL && i < B_ACC_EMPTY) ? 2u : 1u;
            mbar_init(bar(i), count);
        }
        if (lane == 0) {
            *abort_flag = 0;
            *last_flag = 0;
            *never_flag = 0;
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async_smem();
        __syncwarp();
        asm volatile("barrier.cta.arrive 2, %0;" ::"r"(C::Threads) : "memory");
    }
    // Weight producer state (thread 0).
    Cursor wcur;
    wcur.init(u_begin, u_end, p);
    Work ww{};
    int wkb = 0;
    bool w_have = false, w_ok = true;
    uint32_t wcw = 0;
    auto w_issue_one = [&]() -> bool {   // false: nothing left, or a wait gave up (w_ok)
        if (!w_have) {
            if (!next_work(wcur, p, ww)) return false;
            wkb = ww.kb0;
            w_have = true;
        }
        const int nkb = (ww.kb1 - wkb < KS) ? (ww.kb1 - wkb) : KS;
        const int s = wcw % C::NW;
        w_ok = mbar_wait(bar(B_W_FREE + s), ((wcw / C::NW) & 1) ^ 1, ab);
        if (!w_ok) return false;
        // the blocks of one row tile are adjacent in memory: one copy per stage
        mbar_arrive_expect_tx(bar(B_W_FULL + s), nkb * kWkBlockBytes);
        bulk_copy_g2s(sbase + C::OffW + s * C::WBytes,
                      p.Wk + ((size_t)ww.nt * p.KB + wkb) * kWkBlockBytes, nkb * kWkBlockBytes,
                      bar(B_W_FULL + s));
        ++wcw;
        wkb += KS;
        if (wkb >= ww.kb1) w_have = false;
        return true;
    };
    if (warp == C::WarpXProd && lane == 0) {
        prefetch_tensormap(&map_x);
        if (p.r > 0) { prefetch_tensormap(&map_lb); prefetch_tensormap(&map_t); }
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)C::TmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    uint32_t tmem = 0;
    if (warp != 0) {
        tc_fence_before();
        asm volatile("barrier.cta.sync 2, %0;" ::"r"(C::Threads) : "memory");
        tc_fence_after();
        tmem = *tmem_slot;
    }
    const uint32_t tm_dint0 = tmem, tm_dlr = tmem + 2 * BT, tm_a0 = tmem + 3 * BT;
    const int lr_chunks = (p.r + 63) / 64;

    if (warp == 0) {
        // =================== weight producer (one lane) ===================
        if (lane == 0) {
            while (w_ok && w_issue_one()) {}
            const uint32_t cw = wcw;
            const bool ok = w_ok;
            if (*abort_flag) dump_role(p.status, 0, cw, (uint32_t)wkb, (uint32_t)ww.tile, (uint32_t)ww.kb0, (uint32_t)ww.kb1);
            if (!ok || *abort_flag) {
                // let copies already issued land before the CTA's shared memory goes away
                for (uint32_t i = (cw > (uint32_t)C::NW ? cw - C::NW : 0); i < cw; ++i)
                    mbar_wait(bar(B_W_FULL + i % C::NW), (i / C::NW) & 1, Abort{never_flag, p.status});
            }
        }
    } else if (warp == C::WarpXProd) {
        // =================== activation + low-rank operand producer (one lane) ===================
        if (lane == 0) {
            grid_dep_wait();        // Xq and T come from the kernel launched before this one
            Cursor cur;
            cur.init(u_begin, u_end, p);
            Work w{};
            uint32_t cx = 0, cl = 0;
            bool ok = true;
            // ProducerLr: the chunk most recently loaded and not yet multiplied (one slot, so
            // there is never more than one), and the low-rank items multiplied so far.
            bool job = false, job_last = false, dlr_ok = false;
            int job_c = 0;
            uint32_t job_cl = 0, lr_items = 0;
            constexpr uint32_t idesc_lr = make_idesc(1, 0, 128, BT);
            auto run_job = [&]() {          // its conversion is complete: multiply, hand the slot back
                const int s = job_cl % C::NL;
                tc_fence_after();
                const uint64_t adesc = smem_desc_sw128(sbase + C::OffLb + s * C::LbBytes);
                const uint64_t bdesc = smem_desc_sw128(sbase + C::OffT + s * C::TBytes);
                int steps = (p.r - job_c * 64) / 16;
                if (steps > 4) steps = 4;
                for (int kk = 0; kk < steps; ++kk)
                    mma_f16_ss(tm_dlr, adesc + 2 * kk, bdesc + 2 * kk, idesc_lr, (job_c != 0 || kk != 0) ? 1u : 0u);
                tc_commit(bar(B_EMPTY_LR + s));
                if (job_last) {             // the item's low-rank term is complete when these retire
                    tc_commit(bar(B_LR_DONE));
                    ++lr_items;
                    dlr_ok = false;
                }
                job = false;
            };
            // without waiting: multiply the pending chunk if it is ready (the first chunk of an
            // item also needs the previous item's epilogue to have read the accumulator)
            auto poll_job = [&]() {
                if (!C::ProducerLr || !job) return;
                if (job_c == 0 && !dlr_ok) {
                    if (!mbar_try_wait(bar(B_DLR_EMPTY), (lr_items & 1) ^ 1)) return;
                    dlr_ok = true;
                }
                if (!mbar_try_wait(bar(B_CONV_LR + job_cl % C::NL), (job_cl / C::NL) & 1)) return;
                run_job();
            };
            // the same, waiting: before anything that waits for the slot (this thread frees it)
            auto finish_job = [&]() -> bool {
                if (!C::ProducerLr || !job) return true;
                if (job_c == 0 && !dlr_ok) {
                    if (!mbar_wait(bar(B_DLR_EMPTY), (lr_items & 1) ^ 1, ab)) return false;
                    dlr_ok = true;
                }
                if (!mbar_wait(bar(B_CONV_LR + job_cl % C::NL), (job_cl / C::NL) & 1, ab)) return false;
                run_job();
                return true;
            };
            auto load_lr = [&](int c) {
                const int s = cl % C::NL;
                mbar_arrive_expect_tx(bar(B_FULL_LR + s), C::LbBytes + C::TBytes);
                tma_load_2d(sbase + C::OffLb + s * C::LbBytes, &map_lb, c * 64, w.nt * 128, bar(B_FULL_LR + s));
                tma_load_2d(sbase + C::OffT + s * C::TBytes, &map_t, c * 64 + cat_layer(p.cat, w.nt * 128) * p.r, w.tt * BT,
                            bar(B_FULL_LR + s));
                if (C::ProducerLr) {
                    job = true;
                    job_c = c;
                    job_cl = cl;
                    job_last = (c == lr_chunks - 1);
                }
                ++cl;
            };
            auto issue_lr = [&](int c) {
                if (!finish_job()) return false;
                if (!mbar_wait(bar(B_EMPTY_LR + cl % C::NL), ((cl / C::NL) & 1) ^ 1, ab)) return false;
                load_lr(c);
                return true;
            };
            // the same without waiting: false when the slot is still in use
            auto try_issue_lr = [&](int c) {
                if (job) return false;
                if (!mbar_try_wait(bar(B_EMPTY_LR + cl % C::NL), ((cl / C::NL) & 1) ^ 1)) return false;
                load_lr(c);
                return true;
            };
            while (ok && next_work(cur, p, w)) {
                // low-rank chunks that fit the ring go first (they are needed last, so this only
                // prefetches); any further chunk follows the activation stages, which keeps every
                // ring's producer and consumer in the same order
                const int early = !w.has_lr ? 0 : (lr_chunks < C::NL ? lr_chunks : C::NL);
                // With a two-slot ring the chunks go out right after the first activation stage
                // (pure prefetch).  With one slot the previous tile's low-rank MMA has to retire
                // first, so they go out four stages before the end of the tile instead.
                const int nst = (w.kb1 - w.kb0 + KS - 1) / KS;
                const int lr_at = (C::NL == 1 && nst > 5) ? nst - 4 : 1;
                const bool mid = MID && lr_mid_tile(C::NL, w.has_lr, lr_chunks, nst);
                int mid_next = 0;          // mid-tile schedule: next chunk to load
                int st_idx = 0;
                for (int kb = w.kb0; kb < w.kb1 && ok; kb += KS, ++st_idx) {
                    if (!mid && st_idx == lr_at)
                        for (int c = 0; c < early && ok; ++c) ok = issue_lr(c);
                    if (!ok) break;
                    const int s = cx % C::NX;
                    ok = mbar_wait(bar(B_X_FREE + s), ((cx / C::NX) & 1) ^ 1, ab);
                    if (!ok) break;
                    // box = KS column blocks x BT tokens x 128 bytes (blocks past K read as zero)
                    mbar_arrive_expect_tx(bar(B_X_FULL + s), C::XBytes);
                    tma_load_3d(sbase + C::OffX + s * C::XBytes, &map_x, 0, w.tt * BT, kb, bar(B_X_FULL + s));
                    ++cx;
                    poll_job();
                    // mid-tile schedule: the next chunk goes out as soon as the slot is free; never
                    // wait here (the activation stages must keep flowing)
                    if (mid && mid_next < lr_chunks && try_issue_lr(mid_next)) ++mid_next;
                }
                if (mid) {
                    for (int c = mid_next; c < lr_chunks && ok; ++c) ok = issue_lr(c);
                } else if (w.has_lr) {
                    if (w.kb1 - w.kb0 <= KS)   // single-stage item: the early chunks are still due
                        for (int c = 0; c < early && ok; ++c) ok = issue_lr(c);
                    for (int c = early; c < lr_chunks && ok; ++c) ok = issue_lr(c);
                }
            }
            if (ok) ok = finish_job();      // the last item's last chunk
            if (*abort_flag) dump_role(p.status, 1, cx, cl, (uint32_t)w.tile, (uint32_t)w.kb0, (uint32_t)w.kb1);
            if (!ok || *abort_flag) {
                // let copies already issued land before the CTA's shared memory goes away
                for (uint32_t i = (cl > (uint32_t)C::NL ? cl - C::NL : 0); i < cl; ++i)
                    mbar_wait(bar(B_FULL_LR + i % C::NL), (i / C::NL) & 1, Abort{never_flag, p.status});
                for (uint32_t i = (cx > (uint32_t)C::NX ? cx - C::NX : 0); i < cx; ++i)
                    mbar_wait(bar(B_X_FULL + i % C::NX), (i / C::NX) & 1, Abort{never_flag, p.status});
            }
        }
    } else if (warp == 1 || warp == C::WarpIssuer1) {
        // =================== MMA issuers (one lane each; even / odd stages) ===================
        const int issuer = (warp == 1) ? 0 : 1;
        if (lane == 0) {
            constexpr uint32_t idesc_i8 = make_idesc(2, 1, 128, BT);
            constexpr uint32_t idesc_f16 = make_idesc(1, 0, 128, BT);
            Cursor cur;
            cur.init(u_begin, u_end, p);
            Work w;
            uint32_t ca = 0, cl = 0, ci = 0, clr_items = 0;
            bool ok = true;
            while (ok && next_work(cur, p, w)) {
                const int buf = ci & 1;
                const uint32_t d_int = tm_dint0 + buf * BT;
                // the epilogue warps hand the accumulator over zeroed (first time: initial zeroing)
                ok = mbar_wait(bar(B_ACC_EMPTY + buf), (ci >> 1) & 1, ab);
                if (!ok) break;
                tc_fence_after();
                const int nst = (w.kb1 - w.kb0 + KS - 1) / KS;
                const bool mid = !C::ProducerLr && MID && issuer == 0 && lr_mid_tile(C::NL, w.has_lr, lr_chunks, nst);
                int lc = 0;                // low-rank chunks of this item multiplied so far
                // one chunk: wait for its conversion, multiply, hand the slot back
                auto lr_chunk = [&](int c) {
                    const int s = cl % C::NL;
                    if (!mbar_wait(bar(B_CONV_LR + s), (cl / C::NL) & 1, ab)) return false;
                    tc_fence_after();
                    const uint64_t adesc = smem_desc_sw128(sbase + C::OffLb + s * C::LbBytes);
                    const uint64_t bdesc = smem_desc_sw128(sbase + C::OffT + s * C::TBytes);
                    int steps = (p.r - c * 64) / 16;
                    if (steps > 4) steps = 4;
                    for (int kk = 0; kk < steps; ++kk)
                        mma_f16_ss(tm_dlr, adesc + 2 * kk, bdesc + 2 * kk, idesc_f16,
                                   (c != 0 || kk != 0) ? 1u : 0u);
                    tc_commit(bar(B_EMPTY_LR + s));
                    ++cl;
                    return true;
                };
                int st_idx = 0;
                for (int kb = w.kb0; kb < w.kb1 && ok; kb += KS, ++st_idx) {
                    const int nkb = (w.kb1 - kb < KS) ? (w.kb1 - kb) : KS;
                    const int sx = ca % C::NX;   // ca counts stages
                    if (mid && lc < lr_chunks - 1 && st_idx == lr_mma_stage(lc, lr_chunks, nst)) {
                        // the epilogue of the previous item has read the low-rank accumulator
                        if (lc == 0) ok = mbar_wait(bar(B_DLR_EMPTY), (clr_items & 1) ^ 1, ab);
                        ok = ok && lr_chunk(lc);
                        if (!ok) break;
                        ++lc;
                    }
                    if ((int)(ca & 1u) != issuer) { ++ca; continue; }
                    ok = mbar_wait(bar(B_X_FULL + sx), (ca / C::NX) & 1, ab);
                    if (!ok) break;
                    const uint64_t xdesc = smem_desc_sw128(sbase + C::OffX + sx * C::XBytes);
#pragma unroll
                    for (int sub = 0; sub < C::SPS; ++sub) {
                        const uint32_t cs = ca * C::SPS + sub;          // running A-slot counter
                        const int sa = cs % C::NA;
                        ok = ok && mbar_wait(bar(B_READY + sa), (cs / C::NA) & 1, ab);
                        if (!ok) break;
                        tc_fence_after();
                        const uint32_t a_tm = tm_a0 + sa * C::ASlotCols;
#pragma unroll
                        for (int jj = 0; jj < C::KA; ++jj) {
                            const int j = sub * C::KA + jj;
                            if (j < nkb) {
#pragma unroll
                                for (int kk = 0; kk < 4; ++kk)
                                    mma_i8_ts(d_int, a_tm + jj * 32 + kk * 8,
                                              xdesc + (uint64_t)(j * (C::XTile >> 4) + 2 * kk), idesc_i8, 1u);
                            }
                        }
                        tc_commit(bar(B_FREE + sa));   // an empty slot (ragged last stage) still hands over
                    }
                    if (!ok) break;
                    tc_commit(bar(B_X_FREE + sx));
                    ++ca;
                }
                if (!C::ProducerLr && ok && w.has_lr && issuer == 0) {
                    if (lc == 0) ok = mbar_wait(bar(B_DLR_EMPTY), (clr_items & 1) ^ 1, ab);
                    for (int c = lc; c < lr_chunks && ok; ++c) ok = lr_chunk(c);
                    ++clr_items;
                }
                if (ok) tc_commit(bar(B_ACC_FULL + buf));
                ++ci;
            }
            if (*abort_flag) dump_role(p.status, 2 + issuer, ca, cl, ci, (uint32_t)w.tile, ((uint32_t)w.kb0 << 16) | (uint32_t)w.kb1);
        }
    } else if (warp < 10) {
        // =================== unpack warps: int4 -> int8 (x16) into tensor memory ===================
        const int q = warp & 3;                    // TMEM lane quarter this warp may touch
        const int row = q * 32 + lane;             // weight row inside the 128-row tile
        const int group = (warp - 2) >> 2;         // stages alternate between the two groups
        const int gwarp = (warp - 2) & 3;          // warp within its group
        const int t128 = gwarp * 32 + lane;        // 0..127 within the group
        const bool leader = (t128 == 0);           // polls and signals the mbarriers for the group
        Cursor cur;
        cur.init(u_begin, u_end, p);
        Work w;
        uint32_t cw = 0, cl = 0;
        bool ok = true;
        // T chunk in slot cl % NL: bf16 -> fp16 in place (same element size, same swizzled position)
        auto convert_chunk = [&]() {
            const int s = cl % C::NL;
            if (!group_mbar_wait(bar(B_FULL_LR + s), (cl / C::NL) & 1, ab, leader, group)) return false;
            uint8_t* tb = smem + C::OffT + s * C::TBytes;
            for (int i = t128; i < C::TBytes / 16; i += 128) {
                uint4 raw = *reinterpret_cast<uint4*>(tb + i * 16);
                uint32_t in[4] = {raw.x, raw.y, raw.z, raw.w}, out[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float lo = __uint_as_float(in[e] << 16);
                    float hi = __uint_as_float(in[e] & 0xFFFF0000u);
                    __half2 h = __floats2half2_rn(lo, hi);
                    out[e] = *reinterpret_cast<uint32_t*>(&h);
                }
                *reinterpret_cast<uint4*>(tb + i * 16) = make_uint4(out[0], out[1], out[2], out[3]);
            }
            fence_proxy_async_smem();
            group_bar_sync(group);
            if (leader) mbar_arrive(bar(B_CONV_LR + s));
            ++cl;
            return true;
        };
        while (ok && next_work(cur, p, w)) {
            const int nst = (w.kb1 - w.kb0 + KS - 1) / KS;
            const bool mid = MID && group == 0 && lr_mid_tile(C::NL, w.has_lr, lr_chunks, nst);
            int lc = 0;                    // low-rank chunks of this item converted so far
            int st_idx = 0;
            for (int kb = w.kb0; kb < w.kb1 && ok; kb += KS, ++st_idx) {
                const int nkb = (w.kb1 - kb < KS) ? (w.kb1 - kb) : KS;
                const int sw = cw % C::NW;   // cw counts stages
                if (mid && lc < lr_chunks - 1 && st_idx >= lr_mma_stage(lc, lr_chunks, nst) - 2) {
                    // Never WAIT for a chunk in mid-tile: it is loaded only after the chunk before
                    // it has been multiplied, by the thread that also feeds the activation ring,
                    // and that thread gets back to the chunks only while the stages keep flowing
                    // (the first chunk of an item also needs the previous epilogue to have read
                    // the accumulator).  A chunk that has not landed is looked at again at the
                    // next stage; what is left at the end of the item is waited for there, when
                    // every activation stage of the item has been issued.
                    bool landed = true;
                    if (leader) landed = mbar_try_wait(bar(B_FULL_LR + cl % C::NL), (cl / C::NL) & 1);
                    if (group_bar_all(group, landed)) {
                        ok = convert_chunk();
                        if (!ok) break;
                        ++lc;
                    }
                }
                if ((int)(cw & 1u) != group) { ++cw; continue; }
                ok = group_mbar_wait(bar(B_W_FULL + sw), (cw / C::NW) & 1, ab, leader, group);
                if (!ok) break;
                const uint8_t* wsrc = smem + C::OffW + sw * C::WBytes + row * 16;
#pragma unroll
                for (int sub = 0; sub < C::SPS; ++sub) {
                    const uint32_t cs = cw * C::SPS + sub;              // running A-slot counter
                    const int sa = cs % C::NA;
                    ok = ok && group_mbar_wait(bar(B_FREE + sa), ((cs / C::NA) & 1) ^ 1, ab, leader, group);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t a_tm = tm_a0 + sa * C::ASlotCols + ((uint32_t)(q * 32) << 16);
#pragma unroll
                    for (int jj = 0; jj < C::KA; ++jj) {
                        const int j = sub * C::KA + jj;
                        if (j < nkb) {
                            uint32_t v[32];
#pragma unroll
                            for (int s4 = 0; s4 < 4; ++s4) {
                                uint4 x = *reinterpret_cast<const uint4*>(wsrc + j * kWkBlockBytes + s4 * 2048);
                                const uint32_t xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                                for (int i = 0; i < 4; ++i) {
                                    v[s4 * 8 + 2 * i] = (xs[i] << 4) & 0xF0F0F0F0u;   // columns c0 .. c0+3
                                    v[s4 * 8 + 2 * i + 1] = xs[i] & 0xF0F0F0F0u;      // columns c0+4 .. c0+7
                                }
                            }
                            tmem_st32(a_tm + jj * 32, v);
                        }
                    }
                    tmem_wait_st();
                    tc_fence_before();
                    group_bar_sync(group);              // the whole group has written its rows
                    if (leader) {
                        mbar_arrive(bar(B_READY + sa));
                        // ... and, after the last block, has the weight slot in registers: refill it
                        if (sub == C::SPS - 1) mbar_arrive(bar(B_W_FREE + sw));
                    }
                }
                if (!ok) break;
                ++cw;
            }
            if (ok && w.has_lr && group == 0)
                for (int c = lc; c < lr_chunks && ok; ++c) ok = convert_chunk();
        }
        if (leader && *abort_flag) dump_role(p.status, 4 + group, cw, cl, 0u, (uint32_t)w.tile, ((uint32_t)w.kb0 << 16) | (uint32_t)w.kb1);
    } else if (warp < 10 + C::EW) {
        // =================== epilogue warps ===================
        const int q = warp & 3;
        const int nl = q * 32 + lane;              // row of D = output channel inside the tile
        const int et = (warp - 10) * 32 + lane;     // index among the epilogue threads
        const int half = (warp - 10) >> 2;          // which of the quarter's two warps: it takes
        constexpr int kChunkStep = 16 * (C::EW / 4);   // every other 16-column chunk
        const uint32_t lane_sel = (uint32_t)(q * 32) << 16;
        Cursor cur;
        cur.init(u_begin, u_end, p);
        Work w;
        uint32_t ci = 0, lr_seen = 0;
        int partial_idx = 0;                       // 0: first partial item of this CTA, 1: second
        bool ok = true;
        // both integer accumulators start at zero: every integer MMA accumulates
        for (int c0 = 16 * half; c0 < 2 * BT; c0 += kChunkStep) tmem_zero16(tm_dint0 + lane_sel + c0);
        tmem_wait_st();
        grid_dep_wait();            // a_scale comes from the kernel launched before this one
        tc_fence_before();
        __syncwarp();
        if (lane == 0) { mbar_arrive(bar(B_ACC_EMPTY + 0)); mbar_arrive(bar(B_ACC_EMPTY + 1)); }
        while (ok && next_work(cur, p, w)) {
            const int buf = ci & 1;
            ok = warp_mbar_wait(bar(B_ACC_FULL + buf), (ci >> 1) & 1, ab, lane);
            if (C::ProducerLr && w.has_lr) {            // ... and the item's low-rank MMAs (the producer commits them)
                if (ok) ok = warp_mbar_wait(bar(B_LR_DONE), lr_seen & 1, ab, lane);
                ++lr_seen;
            }
            ok = named_bar_all(1, C::EpiThreads, ok);   // the 128 epilogue threads go on or give up together
            if (!ok) break;
            tc_fence_after();
            const int n = w.nt * 128 + nl;
            const bool n_ok = n < p.N;
            const float ws = n_ok ? __ldg(p.w_scale + n) : 0.f;
            const float ws16 = ws * 0.0625f;
            const int tok0 = w.tt * BT;
            const int valid = (p.M - tok0 < BT) ? (p.M - tok0) : BT;   // tokens of this tile inside M
            const uint32_t d_int = tm_dint0 + buf * BT + lane_sel;
            int32_t* pint = p.part_int + ((size_t)cta * 2 + partial_idx) * (BT * 128);
            float* plr = p.part_lr + (size_t)cta * (BT * 128);
#pragma unroll 1
            for (int c0 = 16 * half; c0 < BT; c0 += kChunkStep) {
                uint32_t vi[16], vf[16];
                tmem_ld16(d_int + c0, vi);
                if (w.has_lr) tmem_ld16(tm_dlr + lane_sel + c0, vf);
                tmem_wait_ld(vi);
                if (w.has_lr) tmem_wait_ld(vf);
                if (w.whole) {
                    // The accumulator holds 16 * sum(q x); 1/16 is folded into the scale (exact).
                    // Straight-line code: one vector load of the token scales, then per column
                    // convert, fused multiply-add, round to fp16, predicated 2-byte store.
                    float as[16];
                    if (c0 + 16 <= valid) {
                        const float4* ap = reinterpret_cast<const float4*>(p.a_scale + tok0 + c0);
#pragma unroll
                        for (int v4 = 0; v4 < 4; ++v4) {
                            const float4 a4 = __ldg(ap + v4);
                            as[4 * v4] = a4.x; as[4 * v4 + 1] = a4.y; as[4 * v4 + 2] = a4.z; as[4 * v4 + 3] = a4.w;
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 16; ++j) as[j] = (c0 + j < valid) ? __ldg(p.a_scale + tok0 + c0 + j) : 0.f;
                    }
                    const uint32_t row0 = (uint32_t)(tok0 + c0) * (uint32_t)p.N + (uint32_t)n;
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const float lr = w.has_lr ? __uint_as_float(vf[j]) : 0.f;
                        const float y = fmaf((float)(int)vi[j], as[j] * ws16, lr);
                        // streaming store: Y is written once and not read by this kernel, so it
                        // should not displace the operands that other CTAs still re-read from L2
                        if (c0 + j < valid && n_ok)
                            __stcs(reinterpret_cast<unsigned short*>(p.Y + row0 + (uint32_t)j * (uint32_t)p.N),
                                   __half_as_ushort(__float2half_rn(y)));
                    }
                    if (p.acc_debug) {
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            if (c0 + j < valid && n_ok)
                                p.acc_debug[row0 + (uint32_t)j * (uint32_t)p.N] = ((int)vi[j]) >> 4;
                    }
                } else {
                    // partial tiles are stored [token / 4][row][4 tokens]: every thread moves 16
                    // bytes and a warp 512 contiguous bytes per instruction
                    uint4* pi = reinterpret_cast<uint4*>(pint + (c0 / 4) * 512 + nl * 4);
                    uint4* pf = reinterpret_cast<uint4*>(plr + (c0 / 4) * 512 + nl * 4);
#pragma unroll
                    for (int v4 = 0; v4 < 4; ++v4) {
                        pi[v4 * 128] = make_uint4(vi[4 * v4], vi[4 * v4 + 1], vi[4 * v4 + 2], vi[4 * v4 + 3]);
                        if (w.has_lr) pf[v4 * 128] = make_uint4(vf[4 * v4], vf[4 * v4 + 1], vf[4 * v4 + 2], vf[4 * v4 + 3]);
                    }
                }
            }
            for (int c0 = 16 * half; c0 < BT; c0 += kChunkStep) tmem_zero16(d_int + c0);   // hand it back zeroed
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(bar(B_ACC_EMPTY + buf));
                if (w.has_lr) mbar_arrive(bar(B_DLR_EMPTY));
            }
            ++ci;
            if (!w.whole) {
                // ---- shared tile: publish the partial, the last CTA to arrive finishes it ----
                ++partial_idx;
                const int first_unit = w.tile * p.KB;
                const int c_first = unit_owner(p.units, first_unit, G);
                const int c_last = unit_owner(p.units, first_unit + p.KB - 1, G);
                named_bar_sync(1, C::EpiThreads);            // every partial store of this CTA precedes ...
                if (et == 0) {                     // ... this release; the last arriver acquires all
                    int old;
                    // A CTA owns the first unit of at most one shared tile (the one cut off at the
                    // end of its range), so c_first names the tile's counter: the counter array
                    // has a fixed size and place whatever the problem's shape.
                    asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;"
                                 : "=r"(old) : "l"(p.counters + c_first) : "memory");
                    *last_flag = (old == c_last - c_first) ? 1 : 0;
                }
                named_bar_sync(1, C::EpiThreads);
                const bool last = *last_flag != 0;
                named_bar_sync(1, C::EpiThreads);           // everyone has read the flag before it is reused
                if (last) {
                    if (et == 0) p.counters[c_first] = 0;  // ready for the next launch
                    // Slot of every contributor, computed once (by one thread each) instead of
                    // per chunk: CTA c's items in order are a tile cut off at the start of its
                    // range (slot 0), whole tiles, a tile cut off at the end of its range.
                    const int ncontrib = c_last - c_first + 1;
                    if (et < ncontrib && et < kMaxContrib) {
                        const int c = c_first + et;
                        const int bc = range_begin(p.units, c, G);
                        contrib_slot[et] = c * 2 + ((bc >= first_unit) ? 0 : ((bc % p.KB != 0) ? 1 : 0));
                    }
                    named_bar_sync(1, C::EpiThreads);
#pragma unroll 1
                    for (int c0 = 16 * half; c0 < BT; c0 += kChunkStep) {
                        if (tok0 + c0 >= p.M) break;
                        int sum[16];
#pragma unroll
                        for (int j = 0; j < 16; ++j) sum[j] = 0;
                        uint4 lr4[4];
                        if (p.r > 0) {
                            const uint4* lsrc = reinterpret_cast<const uint4*>(
                                p.part_lr + (size_t)c_first * (BT * 128) + (c0 / 4) * 512 + nl * 4);
#pragma unroll
                            for (int v4 = 0; v4 < 4; ++v4) lr4[v4] = __ldcg(lsrc + v4 * 128);
                        }
                        for (int cb = 0; cb < ncontrib; cb += 2) {
                            // two contributors' loads (eight 16-byte loads) in flight at a time
                            uint4 v[2][4];
#pragma unroll
                            for (int u = 0; u < 2; ++u) {
                                if (cb + u < ncontrib) {
                                    // contributors past the table lie strictly inside the tile: slot 0
                                    const int slot = (cb + u < kMaxContrib) ? contrib_slot[cb + u]
                                                                            : (c_first + cb + u) * 2;
                                    const uint4* src = reinterpret_cast<const uint4*>(
                                        p.part_int + (size_t)slot * (BT * 128) + (c0 / 4) * 512 + nl * 4);
#pragma unroll
                                    for (int v4 = 0; v4 < 4; ++v4) v[u][v4] = __ldcg(src + v4 * 128);
                                } else {
#pragma unroll
                                    for (int v4 = 0; v4 < 4; ++v4) v[u][v4] = make_uint4(0, 0, 0, 0);
                                }
                            }
#pragma unroll
                            for (int u = 0; u < 2; ++u)
#pragma unroll
                                for (int v4 = 0; v4 < 4; ++v4) {
                                    sum[4 * v4] += (int)v[u][v4].x; sum[4 * v4 + 1] += (int)v[u][v4].y;
                                    sum[4 * v4 + 2] += (int)v[u][v4].z; sum[4 * v4 + 3] += (int)v[u][v4].w;
                                }
                        }
                        const uint32_t row0 = (uint32_t)(tok0 + c0) * (uint32_t)p.N + (uint32_t)n;
                        const uint32_t* lrw = reinterpret_cast<const uint32_t*>(lr4);
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            if (c0 + j < valid && n_ok) {
                                const float lr = (p.r > 0) ? __uint_as_float(lrw[j]) : 0.f;
                                const float y = fmaf((float)sum[j], __ldg(p.a_scale + tok0 + c0 + j) * ws16, lr);
                                __stcs(reinterpret_cast<unsigned short*>(p.Y + row0 + (uint32_t)j * (uint32_t)p.N),
                                       __half_as_ushort(__float2half_rn(y)));
                                if (p.acc_debug) p.acc_debug[row0 + (uint32_t)j * (uint32_t)p.N] = sum[j] >> 4;
                            }
                        }
                    }
                }
            }
        }
        if (et == 0 && *abort_flag) dump_role(p.status, 6, ci, (uint32_t)partial_idx, 0u, (uint32_t)w.tile, ((uint32_t)w.kb0 << 16) | (uint32_t)w.kb1);
    }

    // =================== teardown ===================
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                     ::"r"(tmem), "r"((uint32_t)C::TmemCols)
                     : "memory");
    }
}

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------
// 2-D row-major tensor [rows, cols] of `esize`-byte elements, box = [box_rows, box_cols],
// 128-byte swizzle, out-of-range elements read as zero.
int make_map_2d(CUtensorMap* map, CUtensorMapDataType dt, int esize, const void* base,
                uint64_t rows, uint64_t cols, uint32_t box_rows, uint32_t box_cols) {
    return encode_map_2d(map, dt, esize, base, rows, cols, box_rows, box_cols,
                         CU_TENSOR_MAP_SWIZZLE_128B);
}

// Xq [M, K] int8 viewed as [K/128 column blocks][M tokens][128 bytes]; box = KS blocks x BT
// tokens x 128 bytes, 128-byte swizzle.  In shared memory each block's BT x 128-byte tile is
// contiguous, which is the K-major operand layout the MMA descriptor expects.
int make_map_x(CUtensorMap* map, const void* base, uint64_t M, uint64_t K, uint32_t BT, uint32_t KS) {
    MapKey k = make_key(base, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, CU_TENSOR_MAP_SWIZZLE_128B);
    k.dims[0] = 128; k.dims[1] = M; k.dims[2] = K / 128;
    k.strides[0] = K; k.strides[1] = 128;
    k.box[0] = 128; k.box[1] = BT; k.box[2] = KS;
    return encode_tiled(map, k, "cuTensorMapEncodeTiled (Xq)");
}

int pick_bt(int M) { return M <= 16 ? 16 : M <= 32 ? 32 : M <= 64 ? 64 : 128; }

struct Layout {
    int BT, NT, TT, KB;
    long long units;   // must stay below 2^31
    size_t off_counters, off_part_int, off_part_lr, total;
};

Layout make_layout(int M, int N, int K, int r) {
    Layout L;
    L.BT = pick_bt(M);
    L.NT = (N + 127) / 128;
    L.TT = (M + L.BT - 1) / L.BT;
    L.KB = K / 128;
    L.units = (long long)L.NT * L.TT * L.KB;
    // Status word and counters sit at the same offsets for every shape, and a launch leaves the
    // counters at zero again, so one workspace serves calls of different shapes in turn.
    L.off_counters = kWsHeaderBytes;
    L.off_part_int = kWsZeroedBytes;
    static_assert(kWsHeaderBytes + kMaxCtas * 4 <= kWsZeroedBytes, "counter region");
    L.off_part_lr = L.off_part_int + (size_t)kMaxCtas * 2 * L.BT * 128 * 4;
    L.total = L.off_part_lr + (r > 0 ? (size_t)kMaxCtas * L.BT * 128 * 4 : 0);
    return L;
}

template <int BT, bool MID>
int launch_bt(const CUtensorMap& mx, const CUtensorMap& mlb, const CUtensorMap& mt, const Params& p,
              int grid, cudaStream_t st, bool overlap_prev) {
    using C = Cfg<BT>;
    static bool configured[kMaxDevices] = {false};
    int dev = 0;
    const int drc = current_device(&dev);
    if (drc != ASER_OK) return drc;
    if (!configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(linear_tc_kernel<BT, MID>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, C::SmemBytes);
        if (e != cudaSuccess) return record_cuda_error(e, "linear_tc smem attribute");
        configured[dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(C::Threads, 1, 1);
    cfg.dynamicSmemBytes = C::SmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap_prev ? 1 : 0;
    cudaError_t e = cudaLaunchKernelEx(&cfg, linear_tc_kernel<BT, MID>, mx, mlb, mt, p);
    if (e != cudaSuccess) return record_cuda_error(e, "linear_tc_kernel");
    return check_launch("linear_tc_kernel");
}

}  // namespace

size_t linear_tc_workspace_bytes(int M, int N, int K, int r) {
    if (M <= 0 || N <= 0) return kWsZeroedBytes - kWsHeaderBytes;
    return make_layout(M, N, K, r).total - kWsHeaderBytes;
}

size_t linear_tc_zeroed_prefix_bytes(int, int, int, int) { return kWsZeroedBytes; }

int linear_tc_check(int M, int N, int K, int r, size_t workspace_bytes) {
    const Layout L = make_layout(M, N, K, r);
    if (workspace_bytes < L.total) return record_error(ASER_ERR_WORKSPACE, "workspace too small");
    if (L.units >= (1ll << 31) / kMaxCtas * kMaxCtas)
        return record_error(ASER_ERR_SHAPE, "M * N * K beyond the kernel's 31-bit work-unit count");
    if ((long long)(M + 128) * N >= (1ll << 32))   // 32-bit element indices in the epilogue
        return record_error(ASER_ERR_SHAPE, "M * N beyond the kernel's 32-bit output index");
    return ASER_OK;
}

int launch_linear_tc(const int8_t* Xq, const float* a_scale, const uint8_t* Wk,
                     const float* w_scale, const __nv_bfloat16* T, const __half* LB,
                     int M, int N, int K, int r, __half* Y, int32_t* acc_debug,
                     void* workspace, size_t workspace_bytes, cudaStream_t st, bool overlap_prev, int ldt,
                     CatSplit cat) {
    Layout L = make_layout(M, N, K, r);
    const int pre = linear_tc_check(M, N, K, r, workspace_bytes);
    if (pre != ASER_OK) return pre;

    int num_sms = 0;
    {
        const int rc = device_sm_count(&num_sms);
        if (rc != ASER_OK) return rc;
    }
    int grid = num_sms < kMaxCtas ? num_sms : kMaxCtas;
    long long want = (L.units + 1) / 2;   // at least two units per CTA on tiny problems
    if (want < 1) want = 1;
    if (grid > want) grid = (int)want;
    // Tiles that have to be split anyway are split evenly: with a grid that divides the units
    // into equal shares of a whole fraction of a tile, every CTA has exactly one (partial) work
    // item instead of up to three, at the price of a few idle SMs.
    {
        const long long KBl = K / 128;
        for (int g = grid; g >= grid - grid / 6 && g >= 1; --g) {
            if (L.units % g) continue;
            const long long share = L.units / g;
            if (share < KBl && KBl % share == 0) { grid = g; break; }
        }
        // 128-token tiles: a grid that gives every CTA WHOLE tiles has no shared tile at all.  A
        // shared 128 x 128 tile costs a 128 KB partial (int32 + fp32) per contributor through the
        // workspace and a serial tail in the last CTA while the accumulators wait; measured, a
        // launch with shared tiles pays about as much as 64 more column blocks per CTA (20 us at
        // K = 4096; about half of that where tiles are long and hide it).  So: the smallest
        // whole-tile share among the grids down to a third of the SM count, taken if it beats the
        // split share plus that fee.  Measured at 128 against 148 CTAs: 2 tiles of 32 blocks
        // -28 %, 8 x 32 -6 %, 14 x 32 -3 %, 4 x 64 -2 %; at 112 CTAs 2 x 64 -27 %; 28 x 32,
        // 16 x 64 and 4 x 112 are faster split and stay so.
        if (L.BT == 128) {
            const long long fee = (KBl <= 64) ? 64 : 32;
            long long best = (L.units + grid - 1) / grid + fee;
            int best_g = 0;
            for (int g = num_sms < kMaxCtas ? num_sms : kMaxCtas; g >= num_sms / 3 && g >= 1; --g) {
                if (L.units % ((long long)g * KBl)) continue;
                const long long share = L.units / g;
                if (share < best) { best = share; best_g = g; }
            }
            if (best_g) grid = best_g;
        }
    }

    CUtensorMap mx, mlb, mt;
    const int ks = L.BT == 16 ? Cfg<16>::KS : L.BT == 32 ? Cfg<32>::KS : L.BT == 64 ? Cfg<64>::KS : Cfg<128>::KS;
    int rc = make_map_x(&mx, Xq, M, K, L.BT, ks);
    if (rc != ASER_OK) return rc;
    if (r > 0) {
        rc = make_map_2d(&mlb, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, LB, N, r, 128, 64);
        if (rc != ASER_OK) return rc;
        rc = encode_map_2d_ld(&mt, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, T, M, r * cat.layers, ldt > 0 ? ldt : r * cat.layers, L.BT, 64,
                              CU_TENSOR_MAP_SWIZZLE_128B);
        if (rc != ASER_OK) return rc;
    } else {
        mlb = mx;
        mt = mx;
    }

    uint8_t* ws = static_cast<uint8_t*>(workspace);
    Params p;
    p.Wk = Wk; p.a_scale = a_scale; p.w_scale = w_scale; p.Y = Y; p.acc_debug = acc_debug;
    p.status = reinterpret_cast<uint32_t*>(ws);
    p.counters = reinterpret_cast<int*>(ws + L.off_counters);
    p.part_int = reinterpret_cast<int32_t*>(ws + L.off_part_int);
    p.part_lr = reinterpret_cast<float*>(ws + L.off_part_lr);
    p.M = M; p.N = N; p.K = K; p.r = r;
    p.cat = cat;
    p.KB = L.KB; p.TT = L.TT; p.NT = L.NT; p.units = (int)L.units;
    // Both shared tiles first where a tile is long enough (K >= 8192) to hide two cross-CTA
    // reductions behind the next tiles' MMAs; with shorter tiles the epilogue warps fall behind
    // and range order (head part, whole tiles, tail part) is faster.  Measured: K = 14336
    // -12 %, K = 8192 -2..-6 %, K = 4096 +5 % if it were applied there.
    p.tail_first = (L.KB >= 64) ? 1 : 0;
    // Tile numbering.  The CTAs work on about one grid's worth of consecutive tiles at a time, and
    // what those tiles touch should stay in L2: with the weight tile outer that is ALL of Xq plus a
    // few row tiles of the weights, with the token tile outer a few token tiles plus ALL packed
    // weights.  Take the smaller set (4096 tokens into the 14336 -> 4096 projection: Xq is 59 MB and
    // was read from DRAM ten times over with the weight tile outer).
    p.tt_outer = ((long long)M * K > (long long)N * K / 2) ? 1 : 0;

    switch (L.BT) {
        case 16: return launch_bt<16, false>(mx, mlb, mt, p, grid, st, overlap_prev);
        case 32: return launch_bt<32, false>(mx, mlb, mt, p, grid, st, overlap_prev);
        case 64: return launch_bt<64, false>(mx, mlb, mt, p, grid, st, overlap_prev);
        default:
            if (r > 64) return launch_bt<128, true>(mx, mlb, mt, p, grid, st, overlap_prev);
            return launch_bt<128, false>(mx, mlb, mt, p, grid, st, overlap_prev);
    }
}

}  // namespace aser
