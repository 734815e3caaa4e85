// Single-pass tensor-core-unit scan for sm_100a: device code.
//
// One persistent CTA per SM processes 128 x 128-element tiles.  Roles (warps):
//   0        TMA producer: claims the next tile and loads it into a shared-memory ring
//   1        MMA issuer, local scans: tcgen05.mma  D[128 x 128] = X[128 x 128] * (I (x) U_s)  into one of
//            three TMEM accumulators (Algorithm 1, up-sweep round t = 0: every length-s chunk
//            becomes its own scan)
//   2        MMA issuer, row totals: tcgen05.mma  R[128 x 16] = X[128 x 128] * ones  into a ring of
//            eight small TMEM accumulators, issued as soon as the tile has landed - long before a
//            full accumulator is free - so that the cross-tile carry scan starts early
//   12-15    totals: scan the 128 row totals (up-sweep rounds t >= 1), publish the tile total
//   3, 16-19 carry scan across tiles: decoupled look-back over per-tile records in global memory
//            (Section 2.2 steps 2-3: totals of the segments, and their scan)
//   4-11     carry add and store (two groups of four warps taking alternate tiles): add chunk, row
//            and tile carries to every element on the vector ALUs (down-sweep; the paper's
//            discussion section recommends a vector unit for this add), transpose through a
//            swizzled shared-memory slab, write whole 128-byte lines with st.global.v4
// Every wait is bounded; a wait that runs out records TCU_ERR_TIMEOUT in the workspace
// header, and the CTA winds down (drains its copies, frees TMEM) instead of spinning.
#pragma once

#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace tcu {

// ---- compile-time knobs (the defaults are the measured best; the others exist for A/B builds)
#ifndef TCU_STORE_GROUPS
#define TCU_STORE_GROUPS 2      // groups of four store warps (2 or 3)
#endif
#ifndef TCU_PREFETCH_DIST
#define TCU_PREFETCH_DIST 256   // tiles ahead of the claimed one that are prefetched into L2 (0 = off)
#endif
#ifndef TCU_ST_HINT
#define TCU_ST_HINT 0           // output stores: 0 = plain, 1 = st.global.cs (streaming), 2 = st.global.L1::no_allocate
#endif
#ifndef TCU_LD_HINT
#define TCU_LD_HINT 0           // input TMA loads: 1 = L2 evict-first hint (every tile is read once)
#endif
#ifndef TCU_PDL
#define TCU_PDL 1               // programmatic dependent launch: set-up overlaps the tail of the previous kernel in the stream
#endif
#ifndef TCU_TMA_STORE
#define TCU_TMA_STORE 0         // 1 = write the output with TMA stores instead of st.global
#endif
#ifndef TCU_SLABS
#define TCU_SLABS 2             // staging slabs per store warp in the TMA-store build
#endif
#ifndef TCU_SETMAXNREG
#define TCU_SETMAXNREG 1        // move registers from the control warps to the store warps
#endif
#ifndef TCU_LOOKBACK
#define TCU_LOOKBACK 1          // windows of 32 records fetched per look-back round
#endif
#ifndef TCU_STATIC_TILES
#define TCU_STATIC_TILES 0      // 1 = tile j of CTA b is b + j * gridDim.x instead of the next ticket
#endif
#ifndef TCU_MAX_STAGES
#define TCU_MAX_STAGES 10       // most input stages the host will ask for
#endif
#ifndef TCU_PIPE_STORE
#define TCU_PIPE_STORE 0        // 1 = fetch the next 32 TMEM columns before the current ones are stored
#endif

constexpr int kTileRows = 128;          // rows of a tile = M of the MMA = TMEM lanes
constexpr int kTileCols = 128;          // elements per tile row
constexpr int kTileElems = kTileRows * kTileCols;
constexpr int kNumAcc = 3;              // TMEM accumulators of the local scans (128 columns each)
constexpr int kNumTot = 8;              // TMEM accumulators of the row totals (16 columns each)
constexpr int kTotCols = 16;
constexpr int kTotBase = kNumAcc * kTileCols;            // first TMEM column of the totals ring
static_assert(kTotBase + kNumTot * kTotCols <= 512, "TMEM has 512 columns");
constexpr int kStoreGroups = TCU_STORE_GROUPS;           // group g takes the tiles with j % kStoreGroups == g
constexpr int kSlabBytes = 32 * 4 * 32;                  // output staging unit: 32 columns x 32 rows of 4 bytes, written by one warp
constexpr int kSlabsPerWarp = TCU_TMA_STORE ? TCU_SLABS : 1;   // TMA stores read the slab asynchronously: ring of slabs
constexpr int kOutRingBytes = kStoreGroups * 4 * kSlabsPerWarp * kSlabBytes;   // staging slabs of the store warps
constexpr int kNumCarry = 16;           // tiles a CTA may have between "row totals known" and "stored": ring of carry entries
constexpr int kTileRing = 32;           // ring of claimed tile numbers (must exceed the tiles a CTA has in flight)
constexpr uint32_t kNoTile = 0xFFFFFFFFu;   // "no more tiles" marker pushed through the pipeline
constexpr int kNumLookbackWarps = 5;
constexpr int kNumMarkers = kNumLookbackWarps;   // markers pushed: one per look-back warp
constexpr int kMaxInStages = 12;        // size of the barrier arrays
constexpr int kUseInStages = TCU_MAX_STAGES;
constexpr uint32_t kPrefetchDist = TCU_PREFETCH_DIST;
constexpr int kLookBack = TCU_LOOKBACK;
constexpr int kAtomBytes = 128 * kTileRows;   // one 128-byte-swizzled block of 128 rows
constexpr int kOnesBytes = 16 * 128;          // constant operand of the row-total product: 16 rows of ones
constexpr int kDownBytes = (kStoreGroups + 1) * kAtomBytes;   // carry-product variant: one carry operand per store group + a ones operand
constexpr int kUpperBytes = kAtomBytes + 16 * 128;   // limb variant: strictly lower triangular ones (128 x 128 int8) + limb operand
constexpr int kEpilogueThreads = 128;
// Registers per thread after re-allocation.  The pool is what the CTA was launched with (80 x 768 or
// 96 x 640 = 61440 registers), so 128 x (64 + 64 + 40 + kStoreGroups x kStoreRegs) must not exceed it:
// an increase that cannot be granted would block.
constexpr int kStoreRegs = (kStoreGroups == 3) ? 104 : 128;
static_assert(128 * (64 + 64 + 40 + kStoreGroups * kStoreRegs) <= 61440, "register pool");
constexpr int kFirstStoreWarp = 4;                                   // carry add and store: kStoreGroups x 4 warps
constexpr int kFirstTotalsWarp = kFirstStoreWarp + 4 * kStoreGroups; // totals of rows and tile: 4 warps
constexpr int kFirstLookbackWarp = kFirstTotalsWarp + 4;             // cross-tile look-back (warp 3 is one more)
constexpr int kThreads = 32 * (kFirstLookbackWarp + kNumLookbackWarps - 1);

// workspace: 256-byte header, then one 16-byte record per tile
constexpr int kHeaderBytes = 256;
constexpr uint32_t kStatusPartial = 1;    // record holds the tile's own total
constexpr uint32_t kStatusInclusive = 2;  // record holds the sum of everything up to and including the tile
struct WsHeader {
    uint32_t epoch;      // launches completed on this workspace
    uint32_t done;       // CTAs of the running launch that have finished
    uint32_t error;      // tcu_status_t recorded by a bounded wait that ran out
    uint32_t ticket;     // next tile number to hand out (tiles are claimed in increasing order)
    uint32_t pad[60];
};
static_assert(sizeof(WsHeader) == kHeaderBytes, "header size");

#ifdef TCU_PROFILE
// Debug build only: per-CTA cycle counters of where each role waits (64 counters per CTA).
__device__ unsigned long long *g_prof = nullptr;
#define PROF_DECL long long prof_t = 0; unsigned long long prof_a[8] = {0, 0, 0, 0, 0, 0, 0, 0}; (void)prof_t;
#define PROF_T0() prof_t = clock64()
#define PROF_ADD(k) do { long long n_ = clock64(); prof_a[k] += (unsigned long long)(n_ - prof_t); prof_t = n_; } while (0)
#define PROF_INC(k, v) prof_a[k] += (v)
#define PROF_FLUSH(base, cnt) do { if (g_prof) for (int i_ = 0; i_ < (cnt); ++i_) g_prof[blockIdx.x * 64 + (base) + i_] = prof_a[i_]; } while (0)
__device__ unsigned long long *g_trace = nullptr;   // 8 time stamps per tile
__device__ __forceinline__ unsigned long long prof_now() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
#define TRACE(tile, k) do { if (g_trace) g_trace[size_t(tile) * 8 + (k)] = prof_now(); } while (0)
#define TRACE_V(tile, k, v) do { if (g_trace) g_trace[size_t(tile) * 8 + (k)] = (v); } while (0)
#define PROF_STAMP(k) do { if (g_prof && threadIdx.x == 0) g_prof[blockIdx.x * 64 + 48 + (k)] = prof_now(); } while (0)
#else
#define PROF_STAMP(k)
#define TRACE(tile, k)
#define TRACE_V(tile, k, v)
#define PROF_DECL
#define PROF_T0()
#define PROF_ADD(k)
#define PROF_INC(k, v)
#define PROF_FLUSH(base, cnt)
#endif

constexpr long long kSpinLimitCycles = 2000000000LL;   // about one second at B200 clocks

struct alignas(64) ScanParams {
    CUtensorMap tmap_in;      // (128, rows128, batch) view of the input, box 128 B x 128 rows
    CUtensorMap tmap_out;     // (128, rows128, batch) view of the output, box 32 x 32 (used by the TMA-store variant)
    void *ws;
    void *out;                // output array (4-byte elements)
    const void *carry_in;     // optional: one output-typed value added to every element of a single-array scan (or NULL)
    uint64_t scan_pitch;      // elements between consecutive scans (batched), unused for a single array
    uint32_t rows128;         // full 128-element rows of one scan
    uint32_t tiles_total;     // all tiles of the launch
    uint32_t tiles_per_row;   // tiles of one scan (carry chain restarts every tiles_per_row tiles)
    uint32_t in_stages;       // depth of the input ring
    uint32_t b_bytes;         // shared memory reserved for the constant operand I (x) U_s
    uint32_t dtype;           // tcu_dtype_t
    uint32_t level0_only;     // debug: stop after the U_s product (no carries)
    uint32_t prefilled;       // two-sweep variant: the records already hold every tile's inclusive sum
    uint32_t down_tc;         // 16-bit input, s = 128 only: add the row carries with a tensor-core product (B_s-style down-sweep)
    uint32_t upper_tc;        // int8 only: scan the 128 row totals with a second triangular product on 8-bit limbs
};

// shared-memory bookkeeping (lives at the 1024-aligned base of dynamic shared memory)
struct SmemCtl {
    uint64_t full[kMaxInStages];     // TMA -> both MMA issuers
    uint64_t empty[kMaxInStages];    // both MMA issuers -> TMA
    uint64_t acc_full[kNumAcc];      // scan MMAs -> store warps
    uint64_t acc_empty[kNumAcc];     // store warps -> scan MMA issuer
    uint64_t tot_full[kNumTot];      // row-total MMAs -> totals warps
    uint64_t tot_empty[kNumTot];     // totals warps -> row-total MMA issuer (read done)
    uint64_t ring_free[kNumCarry];   // store warps -> totals warps (the carry ring entry may be reused)
    uint64_t agg_ready[kNumCarry];   // totals warps -> look-back warp
    uint64_t carry_ready[kNumCarry]; // look-back warp -> store warps
    uint64_t agg_slot[kNumCarry];    // tile total (bits of a double, or a zero-extended uint32)
    uint64_t carry_slot[kNumCarry];  // sum of all earlier tiles of the same scan
    uint32_t warp_tot[2][4];         // cross-warp hop of the 128-row scan (double buffered)
    uint32_t tile_of[kTileRing];     // tile number of the j-th tile claimed by this CTA
    uint32_t tmem_base;
    uint32_t epoch;
    uint32_t carry_in_bits;          // value at *carry_in (0 when there is none)
    uint64_t epoch_ready;            // thread 0 -> totals and look-back warps: epoch and carry_in_bits are written
    uint64_t up_done;                // limb product of the row totals -> totals warps
    uint64_t down_done[kStoreGroups];   // carry product -> store warps of a group
    volatile uint32_t abort_flag;
};
constexpr int kCtlBytes = 2048;
static_assert(sizeof(SmemCtl) <= kCtlBytes, "control block too large");
constexpr int kRowPrefBytes = kNumCarry * kTileRows * 4;
constexpr int kConstOffset = kCtlBytes + kRowPrefBytes;   // 10240: 1024-aligned
static_assert(kConstOffset % 1024 == 0, "operand regions must be 1024-byte aligned");

// ------------------------------------------------------------------------------------ PTX
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}
__device__ __forceinline__ void fence_barrier_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async_smem() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, int x, int y, int z, uint32_t bar) {
#if TCU_LD_HINT
    uint64_t policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3, %4}], [%5], %6;"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(bar), "l"(policy)
        : "memory");
    return;
#endif
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(bar)
        : "memory");
}
// Ask the TMA unit to bring a box into L2 only (no shared-memory destination, no completion signal).
__device__ __forceinline__ void tma_prefetch_l2_3d(const CUtensorMap *map, int x, int y, int z) {
    asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];"
                 ::"l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z)
                 : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap *map, uint32_t src, int x, int y, int z) {
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
                 ::"l"(reinterpret_cast<uint64_t>(map)), "r"(src), "r"(x), "r"(y), "r"(z)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void named_barrier_sync(int id, int threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
// barrier over `threads` threads that also ORs a predicate; every caller gets the same answer
__device__ __forceinline__ bool named_barrier_or(int id, int threads, bool pred) {
    uint32_t res;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\t"
        "bar.red.or.pred p, %2, %3, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(res)
        : "r"(uint32_t(pred)), "r"(id), "r"(threads)
        : "memory");
    return res != 0;
}
// Register re-allocation between warpgroups (4 consecutive warps): the store warps need many
// registers, every other role few.  All four warps of a group must execute the same instruction.
template <int N>
__device__ __forceinline__ void reg_dec() {
#if TCU_SETMAXNREG
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N));
#endif
}
template <int N>
__device__ __forceinline__ void reg_inc() {
#if TCU_SETMAXNREG
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N));
#endif
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
template <bool IS_INT>
__device__ __forceinline__ void mma_issue(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    if (IS_INT) {
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
            : "memory");
    } else {
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
            : "memory");
    }
}
__device__ __forceinline__ uint32_t tmem_ld1(uint32_t taddr) {
    uint32_t v;
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(v) : "r"(taddr) : "memory");
    return v;
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void ld_shared_v4(uint32_t addr, uint32_t &a, uint32_t &b, uint32_t &c, uint32_t &d) {
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(a), "=r"(b), "=r"(c), "=r"(d) : "r"(addr) : "memory");
}
__device__ __forceinline__ void st_global_v4(void *p, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
#if TCU_ST_HINT == 1
    asm volatile("st.global.cs.v4.b32 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
#elif TCU_ST_HINT == 2
    asm volatile("st.global.L1::no_allocate.v4.b32 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
#else
    asm volatile("st.global.v4.b32 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
#endif
}
__device__ __forceinline__ void ld_record(const void *p, uint64_t &flag, uint64_t &val) {
    asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];" : "=l"(flag), "=l"(val) : "l"(p) : "memory");
}
__device__ __forceinline__ void st_record(void *p, uint64_t flag, uint64_t val) {
    asm volatile("st.relaxed.gpu.global.v2.u64 [%0], {%1, %2};" ::"l"(p), "l"(flag), "l"(val) : "memory");
}
__device__ __forceinline__ uint32_t ld_relaxed_u32(const uint32_t *p) {
    uint32_t v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// ------------------------------------------------------------------------------------ descriptors
// Shared-memory matrix descriptor of tcgen05.mma for a K-major operand stored as rows of
// 128 bytes with the 128-byte swizzle: start address >> 4 in bits [0,14), stride between
// 8-row groups (1024 B) >> 4 in bits [32,46), descriptor version 1 in bits [46,48), swizzle
// mode 2 (128 B) in bits [61,64).  The leading-dimension offset is not used by this layout.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((saddr >> 4) & 0x3FFF);
    d |= static_cast<uint64_t>(1) << 16;
    d |= static_cast<uint64_t>(1024 >> 4) << 32;
    d |= static_cast<uint64_t>(1) << 46;
    d |= static_cast<uint64_t>(2) << 61;
    return d;
}
// Instruction descriptor: accumulator format in bits [4,6) (1 = fp32, 2 = int32), A / B
// formats in bits [7,10) / [10,13) (f16 kinds: 0 = fp16, 1 = bf16; i8 kind: 1 = signed),
// both operands K-major (bits 15, 16 clear), N >> 3 in bits [17,23), M >> 4 in bits [24,29).
__device__ __forceinline__ uint32_t make_idesc(uint32_t dtype, uint32_t n) {
    uint32_t cfmt = (dtype == 0) ? 2u : 1u;
    uint32_t abfmt = (dtype == 0) ? 1u : (dtype == 2 ? 1u : 0u);
    return (cfmt << 4) | (abfmt << 7) | (abfmt << 10) | ((n >> 3) << 17) | ((128u >> 4) << 24);
}

// ------------------------------------------------------------------------------------ helpers
struct Waiter {
    SmemCtl *ctl;
    WsHeader *hdr;
    // Wait for the phase of `bar` with the given parity; false when the wait was given up.
    __device__ __forceinline__ bool wait(uint32_t bar, uint32_t parity) const {
        if (mbar_try_wait(bar, parity)) return true;
        long long t0 = clock64();
        uint32_t spins = 0;
        while (!mbar_try_wait(bar, parity)) {
            if ((++spins & 0xFF) == 0) {
                if (ctl->abort_flag) return false;
                if (clock64() - t0 > kSpinLimitCycles) {
                    ctl->abort_flag = 1;
                    atomicExch(&hdr->error, 5u);
                    return false;
                }
            }
        }
        return true;
    }
};

template <bool IS_INT> struct CarryOps;
template <> struct CarryOps<true> {
    using T = uint32_t;
    static __device__ __forceinline__ uint64_t enc(T v) { return v; }
    static __device__ __forceinline__ T dec(uint64_t b) { return static_cast<uint32_t>(b); }
};
template <> struct CarryOps<false> {
    using T = double;
    static __device__ __forceinline__ uint64_t enc(T v) { return static_cast<uint64_t>(__double_as_longlong(v)); }
    static __device__ __forceinline__ T dec(uint64_t b) { return __longlong_as_double(static_cast<long long>(b)); }
};
template <typename T>
__device__ __forceinline__ T warp_sum(T v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// element arithmetic of the epilogue on raw 32-bit registers
template <bool IS_INT>
__device__ __forceinline__ uint32_t add32(uint32_t a, uint32_t b) {
    if (IS_INT) return a + b;
    return __float_as_uint(__uint_as_float(a) + __uint_as_float(b));
}

// ------------------------------------------------------------------------------------ kernel
template <bool IS_INT, int S, bool EXCL>
__global__ void __launch_bounds__(kThreads, 1) tcu_scan_kernel(const __grid_constant__ ScanParams p) {
    using CO = CarryOps<IS_INT>;
    using CarryT = typename CO::T;
    constexpr int kElemBytes = IS_INT ? 1 : 2;
    constexpr int kPer32B = 32 / kElemBytes;                 // K of one MMA instruction
    constexpr int kSeff = (S > kPer32B) ? S : kPer32B;       // side of the block-diagonal constant I (x) U_s
    constexpr int kSegs = kTileCols / kSeff;                 // MMA groups per tile row
    constexpr int kKSteps = kSeff / kPer32B;                 // accumulating MMAs per group
    constexpr int kRowKSteps = kTileCols / kPer32B;          // accumulating MMAs of the row-total product
    constexpr int kStageBytes = kTileElems * kElemBytes;     // 16 KB (int8) or 32 KB (16-bit)
    constexpr int kInAtoms = kStageBytes / kAtomBytes;

    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    SmemCtl *ctl = reinterpret_cast<SmemCtl *>(smem);
    uint32_t *rowpref = reinterpret_cast<uint32_t *>(smem + kCtlBytes);
    uint8_t *ones_region = smem + kConstOffset;
    uint8_t *const_region = ones_region + kOnesBytes;
    uint8_t *in_ring = const_region + p.b_bytes;
    uint8_t *out_ring = in_ring + p.in_stages * kStageBytes;
    uint8_t *upper_a = out_ring + kOutRingBytes;          // only present when p.upper_tc
    uint8_t *upper_b = upper_a + kAtomBytes;
    uint8_t *down_a = out_ring + kOutRingBytes;           // only present when p.down_tc (never together with upper_tc)
    uint8_t *down_b = down_a + kStoreGroups * kAtomBytes;

    WsHeader *hdr = reinterpret_cast<WsHeader *>(p.ws);
    uint8_t *records = reinterpret_cast<uint8_t *>(p.ws) + kHeaderBytes;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t num_in = p.in_stages;

    // ---- set-up
    PROF_STAMP(0);
    uint32_t first_ticket = 0;                 // (thread 0 only) first tile of this CTA
    uint32_t prev_epoch = 0;                   // (thread 0 only) launches completed on the workspace so far
    if (threadIdx.x == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&p.tmap_in)) : "memory");
#if !TCU_PDL
        first_ticket = TCU_STATIC_TILES ? blockIdx.x : atomicAdd(&hdr->ticket, 1u);
        prev_epoch = ld_relaxed_u32(&hdr->epoch);
#endif
        mbar_init(smem_u32(&ctl->epoch_ready), 1);
        mbar_init(smem_u32(&ctl->up_done), 1);
        for (int g = 0; g < kStoreGroups; ++g) mbar_init(smem_u32(&ctl->down_done[g]), 1);
    }
    {
        // the barriers are the first kNumBarriers 64-bit words of the control block: one thread each
        constexpr int kNumBarriers = 2 * kMaxInStages + 2 * kNumAcc + 2 * kNumTot + 3 * kNumCarry;
        static_assert(kNumBarriers <= kThreads, "one thread per barrier");
        static_assert(offsetof(SmemCtl, agg_slot) == kNumBarriers * 8, "barriers must be contiguous");
        const int k = threadIdx.x;
        if (k < kNumBarriers) {
            uint32_t count = 1;                                                 // full, acc_full, tot_full, carry_ready
            if (k >= kMaxInStages && k < 2 * kMaxInStages) count = 2;           // empty: both MMA issuers
            const int kAccEmpty = 2 * kMaxInStages + kNumAcc, kTotEmpty = kAccEmpty + kNumAcc + kNumTot;
            const int kRingFree = kTotEmpty + kNumTot, kCarryReady = kRingFree + 2 * kNumCarry;
            if (k >= kAccEmpty && k < kAccEmpty + kNumAcc) count = kEpilogueThreads;        // acc_empty
            if (k >= kTotEmpty && k < kTotEmpty + kNumTot) count = kEpilogueThreads;        // tot_empty
            if (k >= kRingFree && k < kCarryReady) count = kEpilogueThreads;                // ring_free, agg_ready
            mbar_init(smem_u32(reinterpret_cast<uint64_t *>(ctl) + k), count);
            fence_barrier_init();
        }
    }
    if (threadIdx.x == 0) ctl->abort_flag = 0;
    if (warp == 1) {
        tmem_alloc(smem_u32(&ctl->tmem_base), 512);
        tmem_relinquish();
    }
    // Constant operands.  Row n of the K-major storage of I (x) U_s holds column n, i.e. ones at
    // k <= n inside the same s-block (U_s is L_s transposed: X U_s = (L_s X^T)^T).  The operand of
    // the row-total product is all ones, so every 32-byte K-slice of it is the same block.
    {
        const uint32_t one = IS_INT ? 0x01010101u : ((p.dtype == 2) ? 0x3F803F80u : 0x3C003C00u);
        uint32_t *oz = reinterpret_cast<uint32_t *>(ones_region);
        for (uint32_t i = threadIdx.x; i < kOnesBytes / 4; i += kThreads) oz[i] = one;
        uint32_t *cz = reinterpret_cast<uint32_t *>(const_region);
        for (uint32_t i = threadIdx.x; i < p.b_bytes / 4; i += kThreads) cz[i] = 0;
        __syncthreads();
        for (int e = threadIdx.x; e < kSeff * kSeff; e += kThreads) {
            int n = e / kSeff, k = e % kSeff;
            if ((n / S) == (k / S) && k <= n) {
                int kb = k * kElemBytes;
                int off = (kb >> 7) * kAtomBytes + n * 128 + ((((kb & 127) >> 4) ^ (n & 7)) << 4) + (kb & 15);
                if (IS_INT) {
                    const_region[off] = 1;
                } else {
                    *reinterpret_cast<uint16_t *>(const_region + off) = (p.dtype == 2) ? 0x3F80 : 0x3C00;
                }
            }
        }
        if (!IS_INT && p.down_tc) {
            // carry operands start as zeros (only 3 of the 16 K-entries of a row are ever written); the other
            // operand is all ones in bf16
            for (int e = threadIdx.x; e < kStoreGroups * kAtomBytes / 4; e += kThreads) reinterpret_cast<uint32_t *>(down_a)[e] = 0;
            for (int e = threadIdx.x; e < kAtomBytes / 4; e += kThreads) reinterpret_cast<uint32_t *>(down_b)[e] = 0x3F803F80u;
        }
        if (IS_INT && p.upper_tc) {
            // A[m][k] = 1 for k < m: its product with a column of row totals is their exclusive scan over the rows
            for (int e = threadIdx.x; e < kTileRows * kTileRows; e += kThreads) {
                const int m = e >> 7, k = e & 127;
                upper_a[m * 128 + ((((k >> 4) ^ (m & 7))) << 4) + (k & 15)] = (k < m) ? 1 : 0;
            }
            for (int e = threadIdx.x; e < 16 * 128 / 4; e += kThreads) reinterpret_cast<uint32_t *>(upper_b)[e] = 0;
        }
        fence_proxy_async_smem();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    PROF_STAMP(1);
    // Everything above touched only this CTA's shared memory and TMEM, so under programmatic dependent launch it
    // may run while the previous kernel of the stream is still finishing.  From here on global memory is read.
#if TCU_PDL
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
#endif
    const uint32_t tmem_base = ctl->tmem_base;
    Waiter w{ctl, hdr};
    uint32_t my_epoch = 0;                     // (thread 0 only) the epoch of this launch
    if (threadIdx.x == 0) {
#if TCU_PDL
        first_ticket = TCU_STATIC_TILES ? blockIdx.x : atomicAdd(&hdr->ticket, 1u);
        prev_epoch = ld_relaxed_u32(&hdr->epoch);
#endif
        my_epoch = prev_epoch + 1;
        ctl->epoch = my_epoch;
        // what precedes the whole scan (continuation of an earlier segment); only single-array calls pass one
        ctl->carry_in_bits = p.carry_in ? *reinterpret_cast<const uint32_t *>(p.carry_in) : 0u;
        mbar_arrive(smem_u32(&ctl->epoch_ready));
    }

    // The j-th tile handled by this CTA is number tile_of[j % kTileRing]: either blockIdx.x + j * gridDim.x
    // (static order) or the next ticket from the workspace (tiles claimed at run time, in increasing order:
    // whoever holds tile t knows that every tile before t is held by a CTA that is already running).  When
    // the tiles run out the producer pushes kNumMarkers "no more tiles" markers through the pipeline, so
    // that every role - and each of the look-back warps - sees one and stops.
    // ------------------------------------------------------------------ cross-tile carry scan (role of warp 3 and warps 20-23)
    auto lookback_role = [&](const uint32_t lbw) {
        if (!__all_sync(0xffffffffu, w.wait(smem_u32(&ctl->epoch_ready), 0))) return;
        const uint32_t epoch = ctl->epoch;
        const CarryT carry_in = IS_INT ? CarryT(ctl->carry_in_bits) : CarryT(__uint_as_float(ctl->carry_in_bits));
        // ------------------------------------------------------------------ cross-tile carry scan
        // kNumLookbackWarps warps take the tiles in turn, so that the look-backs of the tiles in flight overlap.
        PROF_DECL
        PROF_T0();
        for (uint32_t j = lbw;; j += kNumLookbackWarps) {
            const uint32_t ts = j % kNumCarry, ut = j / kNumCarry;
            if (!__all_sync(0xffffffffu, w.wait(smem_u32(&ctl->agg_ready[ts]), ut & 1))) break;
            PROF_ADD(0);
            const uint32_t t = ctl->tile_of[j % kTileRing];
            if (t == kNoTile) {
                if (lane == 0) mbar_arrive(smem_u32(&ctl->carry_ready[ts]));
                break;
            }
            if (lane == 0) TRACE(t, 4);
            const CarryT agg = CO::dec(ctl->agg_slot[ts]);
            const int t0 = static_cast<int>(t - t % p.tiles_per_row);   // first tile of this scan
            CarryT prefix = (static_cast<int>(t) == t0) ? carry_in : CarryT(0);
            if (static_cast<int>(t) != t0) {       // (the first tile's record was published by the totals warps)
                int pos = static_cast<int>(t) - 1;
                bool gave_up = false;
                while (true) {
                    // Every lane fetches kLookBack records at once (distance d = k * 32 + lane behind pos), so
                    // that a window of 32 * kLookBack predecessors costs one round trip to L2.  The windows
                    // are then examined nearest first, and only a window that is actually needed is waited
                    // for: the walk stops at the nearest record that already holds an inclusive sum.
                    uint64_t flag[kLookBack], val[kLookBack];
#pragma unroll
                    for (int k = 0; k < kLookBack; ++k) {
                        int idx = pos - (k * 32 + lane);
                        flag[k] = 0;
                        val[k] = 0;
                        if (idx >= t0) ld_record(records + size_t(idx) * 16, flag[k], val[k]);
                    }
                    CarryT part = CarryT(0);
                    bool done = false;
#pragma unroll
                    for (int k = 0; k < kLookBack; ++k) {
                        if (!done) {                               // warp-uniform
                            const int idx = pos - (k * 32 + lane);
                            const bool valid = idx >= t0;
                            if (valid && static_cast<uint32_t>(flag[k] >> 2) != epoch) {
                                const void *rec = records + size_t(idx) * 16;
                                long long c0 = clock64();
                                uint32_t spins = 0;
                                while (true) {
                                    __nanosleep(20);
                                    ld_record(rec, flag[k], val[k]);
                                    if (static_cast<uint32_t>(flag[k] >> 2) == epoch) break;
                                    if ((++spins & 0x3F) == 0 && (ctl->abort_flag || clock64() - c0 > kSpinLimitCycles)) {
                                        gave_up = true;
                                        flag[k] = kStatusInclusive;   // treat as a chain end so that the walk stops
                                        val[k] = 0;
                                        break;
                                    }
                                }
                            }
                            const bool incl = valid && ((flag[k] & 3) == kStatusInclusive);
                            const unsigned m = __ballot_sync(0xffffffffu, incl);
                            CarryT v = valid ? CO::dec(val[k]) : CarryT(0);
                            if (m) {
                                int first = __ffs(m) - 1;          // nearest predecessor whose record is inclusive
                                if (lane > first) v = CarryT(0);
                                done = true;
                            }
                            part += v;
                            if (pos - (k * 32 + 31) <= t0) done = true;   // the window reached the first tile of the scan
                        }
                    }
                    prefix += warp_sum(part);
                    PROF_INC(2, 1);
                    if (done) break;
                    pos -= 32 * kLookBack;
                    if (pos < t0) break;
                }
                if (__any_sync(0xffffffffu, gave_up)) {
                    if (lane == 0) {
                        ctl->abort_flag = 1;
                        atomicExch(&hdr->error, 5u);
                    }
                }
                // publish even after a give-up so that successors do not wait for this tile
                if (lane == 0 && !p.prefilled) st_record(records + size_t(t) * 16, (uint64_t(epoch) << 2) | kStatusInclusive, CO::enc(prefix + agg));
            }
            if (lane == 0) {
                TRACE(t, 5);
                ctl->carry_slot[ts] = CO::enc(prefix);
                mbar_arrive(smem_u32(&ctl->carry_ready[ts]));
            }
            __syncwarp();
            PROF_ADD(1);
            PROF_INC(3, 1);
        }
        if (lane == 0) PROF_FLUSH(12 + 4 * (lbw % 4), 4);
    };

    if (warp < 4) {
    reg_dec<64>();                                     // producer, MMA issuers, one look-back warp
    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t issued = 0, markers = 0;
            PROF_DECL
            PROF_T0();
            for (uint32_t j = 0;; ++j) {
                uint32_t stage = j % num_in, u = j / num_in;
                if (!w.wait(smem_u32(&ctl->empty[stage]), (u & 1) ^ 1)) break;
                PROF_ADD(0);
                uint32_t t = kNoTile;
                if (markers == 0) {
                    if (j == 0) t = first_ticket;
                    else t = TCU_STATIC_TILES ? (blockIdx.x + j * gridDim.x) : atomicAdd(&hdr->ticket, 1u);
                }
                if (t >= p.tiles_total) t = kNoTile;
                PROF_ADD(1);
                PROF_INC(3, 1);
                ctl->tile_of[j % kTileRing] = t;
                uint32_t bar = smem_u32(&ctl->full[stage]);
                if (t == kNoTile) {
                    mbar_arrive(bar);
                    if (++markers == kNumMarkers) break;
                    continue;
                }
                TRACE(t, 0);
                mbar_expect_tx(bar, kStageBytes);
                int scan_row = t / p.tiles_per_row, lt = t % p.tiles_per_row;
#pragma unroll
                for (int a = 0; a < kInAtoms; ++a)
                    tma_load_3d(smem_u32(in_ring + stage * kStageBytes + a * kAtomBytes), &p.tmap_in,
                                a * (128 / kElemBytes), lt * kTileRows, scan_row, bar);
                issued = j + 1;
                // Tiles are claimed in increasing order by all CTAs, so tile t + kPrefetchDist will be claimed by
                // somebody a few microseconds from now: start its trip from DRAM to L2 now.  Its later load then
                // costs an L2 hit, which takes the DRAM latency - and its spread - out of the carry chain.
                if (kPrefetchDist > 0 && t + kPrefetchDist < p.tiles_total) {
                    const uint32_t tp = t + kPrefetchDist;
                    const int prow = tp / p.tiles_per_row, plt = tp % p.tiles_per_row;
#pragma unroll
                    for (int a = 0; a < kInAtoms; ++a)
                        tma_prefetch_l2_3d(&p.tmap_in, a * (128 / kElemBytes), plt * kTileRows, prow);
                }
                PROF_ADD(2);
            }
            PROF_FLUSH(0, 4);
            if (ctl->abort_flag) {
                // drain: loads already issued must land before the CTA may exit
                uint32_t lo = issued > num_in ? issued - num_in : 0;
                for (uint32_t j = lo; j < issued; ++j) {
                    uint32_t bar = smem_u32(&ctl->full[j % num_in]);
                    uint32_t par = (j / num_in) & 1;
                    long long t0 = clock64();
                    while (!mbar_try_wait(bar, par) && clock64() - t0 < kSpinLimitCycles) {}
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer: local scans
        if (lane == 0) {
            const uint32_t idesc = make_idesc(p.dtype, kSeff);
            const uint32_t b_base = smem_u32(const_region);
            uint32_t markers = 0;
            PROF_DECL
            PROF_T0();
            for (uint32_t j = 0;; ++j) {
                uint32_t stage = j % num_in, u = j / num_in;
                uint32_t slot = j % kNumAcc, ua = j / kNumAcc;
                if (!w.wait(smem_u32(&ctl->full[stage]), u & 1)) break;
                PROF_ADD(0);
                if (ctl->tile_of[j % kTileRing] == kNoTile) {
                    mbar_arrive(smem_u32(&ctl->empty[stage]));
                    if (++markers == kNumMarkers) break;
                    continue;
                }
                if (!w.wait(smem_u32(&ctl->acc_empty[slot]), (ua & 1) ^ 1)) break;
                PROF_ADD(1);
                tc_fence_after();
                const uint32_t a_base = smem_u32(in_ring + stage * kStageBytes);
#pragma unroll
                for (int g = 0; g < kSegs; ++g) {
#pragma unroll
                    for (int kk = 0; kk < kKSteps; ++kk) {
                        int a_off = (g * kKSteps + kk) * 32;
                        int b_off = kk * 32;
                        uint64_t adesc = make_smem_desc(a_base + (a_off >> 7) * kAtomBytes + (a_off & 127));
                        uint64_t bdesc = make_smem_desc(b_base + (b_off >> 7) * kAtomBytes + (b_off & 127));
                        mma_issue<IS_INT>(tmem_base + slot * kTileCols + g * kSeff, adesc, bdesc, idesc, kk > 0 ? 1u : 0u);
                    }
                }
                mma_commit(smem_u32(&ctl->empty[stage]));      // the stage may be refilled once both issuers' MMAs have read it
                mma_commit(smem_u32(&ctl->acc_full[slot]));
                PROF_ADD(2);
            }
            PROF_FLUSH(4, 3);
        }
    } else if (warp == 2) {
        // ------------------------------------------------------------------ MMA issuer: row totals
        if (lane == 0) {
            const uint32_t idesc = make_idesc(p.dtype, kTotCols);
            const uint64_t bdesc = make_smem_desc(smem_u32(ones_region));
            uint32_t markers = 0;
            PROF_DECL
            PROF_T0();
            for (uint32_t j = 0;; ++j) {
                uint32_t stage = j % num_in, u = j / num_in;
                uint32_t ts = j % kNumTot, ut = j / kNumTot;
                if (!w.wait(smem_u32(&ctl->full[stage]), u & 1)) break;
                PROF_ADD(0);
                if (!w.wait(smem_u32(&ctl->tot_empty[ts]), (ut & 1) ^ 1)) break;
                PROF_ADD(1);
                if (ctl->tile_of[j % kTileRing] == kNoTile) {
                    mbar_arrive(smem_u32(&ctl->empty[stage]));
                    mbar_arrive(smem_u32(&ctl->tot_full[ts]));
                    if (++markers == kNumMarkers) break;
                    continue;
                }
                TRACE(ctl->tile_of[j % kTileRing], 1);
                tc_fence_after();
                const uint32_t a_base = smem_u32(in_ring + stage * kStageBytes);
#pragma unroll
                for (int kk = 0; kk < kRowKSteps; ++kk) {
                    int a_off = kk * 32;
                    uint64_t adesc = make_smem_desc(a_base + (a_off >> 7) * kAtomBytes + (a_off & 127));
                    mma_issue<IS_INT>(tmem_base + kTotBase + ts * kTotCols, adesc, bdesc, idesc, kk > 0 ? 1u : 0u);
                }
                mma_commit(smem_u32(&ctl->empty[stage]));
                mma_commit(smem_u32(&ctl->tot_full[ts]));
                PROF_ADD(2);
            }
            PROF_FLUSH(8, 3);
        }
    } else {
        lookback_role(0);
    }
    } else if (warp >= kFirstLookbackWarp) {
        reg_dec<64>();
        lookback_role(uint32_t(warp - kFirstLookbackWarp + 1));
    } else if (warp >= kFirstTotalsWarp) {
        reg_dec<40>();
        // ------------------------------------------------------------------ totals (up-sweep above the product)
        // Takes the 128 row totals from the small accumulator, scans them across the rows, and
        // publishes the tile total - as soon as the tile has landed, so that the cross-tile look-back
        // has several tile times to complete before the store warps need its result.
        const int r = threadIdx.x - kFirstTotalsWarp * 32;          // tile row owned by this thread = TMEM lane
        const int wq = r >> 5;
        const uint32_t lane_base = tmem_base + (uint32_t(wq * 32) << 16);
        const bool epoch_ok = w.wait(smem_u32(&ctl->epoch_ready), 0);
        const uint32_t epoch = ctl->epoch;
        const CarryT carry_in = IS_INT ? CarryT(ctl->carry_in_bits) : CarryT(__uint_as_float(ctl->carry_in_bits));
        uint32_t markers = 0;
        PROF_DECL
        PROF_T0();
        for (uint32_t j = 0;; ++j) {
            const uint32_t tt = j % kNumTot, utt = j / kNumTot;      // row-total accumulator in TMEM
            const uint32_t ts = j % kNumCarry, ut = j / kNumCarry;   // carry ring entry
            // a wait that ran out is voted on, so that all 128 threads leave together
            bool ok = w.wait(smem_u32(&ctl->tot_full[tt]), utt & 1) && epoch_ok;
            ok = w.wait(smem_u32(&ctl->ring_free[ts]), (ut & 1) ^ 1) && ok;
            PROF_ADD(0);
            if (named_barrier_or(2, kEpilogueThreads, !ok)) break;
            const uint32_t t = ctl->tile_of[j % kTileRing];
            if (t == kNoTile) {
                mbar_arrive(smem_u32(&ctl->tot_empty[tt]));
                mbar_arrive(smem_u32(&ctl->agg_ready[ts]));
                if (++markers == kNumMarkers) break;
                continue;
            }
            if (r == 0) TRACE(t, 2);
            tc_fence_after();
            const uint32_t rowtot = tmem_ld1(lane_base + kTotBase + tt * kTotCols);
            tmem_ld_wait();
            if (IS_INT && p.upper_tc) {
                // Paper-faithful variant of this level: the scan over the 128 row totals is itself a product
                // with a triangular all-ones matrix.  Row totals are int32, not a tensor-core input type, so
                // each is split into two signed 8-bit limbs (total = 128 h + l, |total| <= 2^14), the limbs
                // are scanned by one kind::i8 product, and the two results are recombined exactly.
                const int32_t tot = int32_t(rowtot);
                const uint32_t ub = smem_u32(upper_b);
                const uint32_t off = ((r >> 4) << 4) + (r & 15);         // k = r inside a 128-byte row, before the swizzle
                asm volatile("st.shared.u8 [%0], %1;" ::"r"(ub + 0 * 128 + ((((r >> 4) ^ 0) << 4) | (r & 15))), "r"(tot & 127) : "memory");
                asm volatile("st.shared.u8 [%0], %1;" ::"r"(ub + 1 * 128 + ((((r >> 4) ^ 1) << 4) | (r & 15))), "r"((tot >> 7) & 0xFF) : "memory");
                (void)off;
                fence_proxy_async_smem();
                named_barrier_sync(2, kEpilogueThreads);
                if (r == 0) {
                    tc_fence_after();
                    const uint32_t idesc = make_idesc(0, kTotCols);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        mma_issue<true>(tmem_base + kTotBase + tt * kTotCols, make_smem_desc(smem_u32(upper_a) + kk * 32),
                                        make_smem_desc(ub + kk * 32), idesc, kk > 0 ? 1u : 0u);
                    mma_commit(smem_u32(&ctl->up_done));
                }
                (void)w.wait(smem_u32(&ctl->up_done), j & 1);              // (a wait that ran out is caught by the next vote)
                tc_fence_after();
                const uint32_t d0 = tmem_ld1(lane_base + kTotBase + tt * kTotCols);
                const uint32_t d1 = tmem_ld1(lane_base + kTotBase + tt * kTotCols + 1);
                tmem_ld_wait();
                tc_fence_before();
                mbar_arrive(smem_u32(&ctl->tot_empty[tt]));            // the small accumulator may be refilled
                const uint32_t exc_all = d0 + (d1 << 7);                   // sum of the totals of rows 0 .. r-1
                rowpref[ts * kTileRows + r] = exc_all;
                if (r == kTileRows - 1) {
                    const CarryT a = CarryT(exc_all + rowtot);
                    const bool first = (t % p.tiles_per_row == 0);
                    const uint32_t status = first ? kStatusInclusive : kStatusPartial;
                    if (!p.prefilled) st_record(records + size_t(t) * 16, (uint64_t(epoch) << 2) | status, CO::enc(first ? a + carry_in : a));
                    ctl->agg_slot[ts] = CO::enc(a);
                }
                mbar_arrive(smem_u32(&ctl->agg_ready[ts]));
                PROF_ADD(1);
                continue;
            }
            tc_fence_before();
            mbar_arrive(smem_u32(&ctl->tot_empty[tt]));                // the small accumulator may be refilled
            uint32_t inc = rowtot;                                    // inclusive scan across the warp's 32 rows
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                uint32_t up = __shfl_up_sync(0xffffffffu, inc, o);
                if (lane >= o) inc = add32<IS_INT>(inc, up);
            }
            uint32_t exc = __shfl_up_sync(0xffffffffu, inc, 1);
            if (lane == 0) exc = 0;
            const int pb = j & 1;
            if (lane == 31) ctl->warp_tot[pb][wq] = inc;
            named_barrier_sync(2, kEpilogueThreads);
            uint32_t w0 = ctl->warp_tot[pb][0], w1 = ctl->warp_tot[pb][1], w2 = ctl->warp_tot[pb][2], w3 = ctl->warp_tot[pb][3];
            uint32_t before = 0;                                      // rows of the earlier warps
            if (wq >= 1) before = w0;
            if (wq >= 2) before = add32<IS_INT>(before, w1);
            if (wq >= 3) before = add32<IS_INT>(before, w2);
            rowpref[ts * kTileRows + r] = (wq == 0) ? exc : add32<IS_INT>(before, exc);
            if (r == 0) {
                uint32_t tile_tot = add32<IS_INT>(add32<IS_INT>(w0, w1), add32<IS_INT>(w2, w3));
                CarryT a = IS_INT ? CarryT(tile_tot) : CarryT(__uint_as_float(tile_tot));
                // the first tile of a scan has nothing before it: its total is already inclusive
                const bool first = (t % p.tiles_per_row == 0);
                const uint32_t status = first ? kStatusInclusive : kStatusPartial;
                if (!p.prefilled) st_record(records + size_t(t) * 16, (uint64_t(epoch) << 2) | status, CO::enc(first ? a + carry_in : a));
                TRACE(t, 3);
                ctl->agg_slot[ts] = CO::enc(a);
            }
            // every thread arrives (release) after its own rowpref entry is written: the look-back warp,
            // and through it the store warps, then see all 128 entries
            mbar_arrive(smem_u32(&ctl->agg_ready[ts]));
            PROF_ADD(1);
        }
        if (r == 0) PROF_FLUSH(28, 2);
    } else {
        reg_inc<kStoreRegs>();
        // ------------------------------------------------------------------ carry add and store (down-sweep)
        // Every warp works alone on its 32 rows: TMEM -> registers (one row per lane) -> add carries ->
        // swizzled 4 KB slab in shared memory -> read back with eight lanes per row -> st.global.v4,
        // so that every store instruction writes four complete 128-byte lines.  No barrier between warps.
        const int group = (warp - kFirstStoreWarp) >> 2;
        const int wq = warp & 3;                                    // TMEM lane quarter this warp may read
        const int r = wq * 32 + lane;                               // tile row owned by this thread
        const uint32_t lane_base = tmem_base + (uint32_t(wq * 32) << 16);
        const uint32_t slab0 = smem_u32(out_ring) + (warp - kFirstStoreWarp) * kSlabsPerWarp * kSlabBytes;
        uint32_t slab_counter = 0;
        (void)slab_counter;
        const int sub = lane >> 3, piece = lane & 7;                // read-back role: row sub (+4i) of the slab, 16-byte piece
        uint32_t *const out32 = reinterpret_cast<uint32_t *>(p.out);
        PROF_DECL
        PROF_T0();
        for (uint32_t j = group;; j += kStoreGroups) {
            const uint32_t ts = j % kNumCarry, ut = j / kNumCarry;
            const uint32_t slot = j % kNumAcc, ua = j / kNumAcc;
            bool ok = w.wait(smem_u32(&ctl->carry_ready[ts]), ut & 1);
            if (!__all_sync(0xffffffffu, ok)) break;
            PROF_ADD(0);
            const uint32_t t = ctl->tile_of[j % kTileRing];
            if (t == kNoTile) break;
            ok = w.wait(smem_u32(&ctl->acc_full[slot]), ua & 1);
            if (!__all_sync(0xffffffffu, ok)) break;
            PROF_ADD(1);
            PROF_INC(5, 1);
            if (lane == 0 && wq == 0) TRACE(t, 6);
            tc_fence_after();
            const uint32_t scan_row = t / p.tiles_per_row, lt = t % p.tiles_per_row;
            uint32_t base;                                            // sum of everything before this row
            {
                CarryT carry = CO::dec(ctl->carry_slot[ts]);
                uint32_t rp = rowpref[ts * kTileRows + r];
                if (IS_INT) base = uint32_t(carry) + rp;
                else base = __float_as_uint(static_cast<float>(double(carry) + double(__uint_as_float(rp))));
            }
            const bool level0 = p.level0_only != 0;
            if (level0) base = 0;
            uint32_t run = base;                                      // sum of everything before the current chunk
            uint32_t prev = base;                                     // value of the element to the left (exclusive form)
            if (!IS_INT && S == 128 && p.down_tc && !level0) {
                // Paper-faithful variant of the down-sweep (the B_s product: one carry added to a whole vector):
                // the accumulator gets D += C * 1, where row r of C holds the row's carry split exactly into
                // three bf16 terms and 1 is an all-ones operand.  128 x 128 x 16 multiply-adds for 16 Ki useful
                // additions - the low utilisation the paper's discussion predicts for this step.
                const float b0 = __uint_as_float(base);
                const uint32_t hi = __float_as_uint(b0) & 0xFFFF0000u;
                const float r1 = b0 - __uint_as_float(hi);
                const uint32_t mid = __float_as_uint(r1) & 0xFFFF0000u;
                const float r2 = r1 - __uint_as_float(mid);
                const uint32_t lo = __float_as_uint(r2) & 0xFFFF0000u;             // r2 has at most 8 significant bits
                const uint32_t da = smem_u32(down_a) + group * kAtomBytes;
                const uint32_t row_addr = da + r * 128 + ((0 ^ (r & 7)) << 4);       // K entries 0..7 of row r
                asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(row_addr), "r"((hi >> 16) | mid), "r"(lo >> 16) : "memory");
                fence_proxy_async_smem();
                named_barrier_sync(3 + group, kEpilogueThreads);
                if (wq == 0 && lane == 0) {
                    tc_fence_after();
                    mma_issue<false>(tmem_base + slot * kTileCols, make_smem_desc(da), make_smem_desc(smem_u32(down_b)),
                                     make_idesc(2, kTileCols), 1u);
                    mma_commit(smem_u32(&ctl->down_done[group]));
                }
                if (!__all_sync(0xffffffffu, w.wait(smem_u32(&ctl->down_done[group]), (j / kStoreGroups) & 1))) break;
                tc_fence_after();
                run = 0;                                              // the carry is inside the accumulator now
            }
            const uint32_t row0 = lt * kTileRows + wq * 32;           // first 128-element row of this warp's part of the tile
            uint32_t *const gbase = out32 + size_t(scan_row) * p.scan_pitch + size_t(row0) * kTileCols + piece * 4;
            const int rows_here = int(p.rows128) - int(row0);         // rows of this part that exist (ragged last tile)
            uint32_t d[32];
            tmem_ld32(lane_base + slot * kTileCols, d);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                tmem_ld_wait();
                PROF_ADD(2);
                uint32_t o[32];
#pragma unroll
                for (int c = 0; c < 32; ++c) {
                    uint32_t v = add32<IS_INT>(d[c], run);
                    o[c] = EXCL ? prev : v;
                    prev = v;
                    const bool chunk_end = (S <= 32) ? (((c + 1) % S) == 0) : (c == 31 && (((q + 1) * 32) % S) == 0);
                    if (chunk_end && !level0) run = v;                // end of a chunk: its total joins the carry
                }
                if (level0 && EXCL) {                                 // not a meaningful combination; keep it defined
#pragma unroll
                    for (int c = 0; c < 32; ++c) o[c] = d[c];
                }
                // fetch the next 32 columns while this chunk is transposed and stored
                if (TCU_PIPE_STORE && q < 3) tmem_ld32(lane_base + slot * kTileCols + (q + 1) * 32, d);
#if TCU_TMA_STORE
                if (lane == 0) bulk_wait_read<kSlabsPerWarp - 1>();    // the slab about to be written has been drained
                __syncwarp();
                const uint32_t slab = slab0 + (slab_counter % kSlabsPerWarp) * kSlabBytes;
                const uint32_t buf = slab + lane * 128;
#pragma unroll
                for (int c4 = 0; c4 < 8; ++c4)
                    st_shared_v4(buf + ((c4 ^ (lane & 7)) << 4), o[4 * c4], o[4 * c4 + 1], o[4 * c4 + 2], o[4 * c4 + 3]);
                fence_proxy_async_smem();
                __syncwarp();
                PROF_ADD(3);
                if (lane == 0) {
                    tma_store_3d(&p.tmap_out, slab, q * 32, row0, scan_row);
                    bulk_commit();
                }
                ++slab_counter;
#else
                const uint32_t slab = slab0;
                __syncwarp();                                         // the slab has been read back by every lane
                const uint32_t buf = slab + lane * 128;
#pragma unroll
                for (int c4 = 0; c4 < 8; ++c4)
                    st_shared_v4(buf + ((c4 ^ (lane & 7)) << 4), o[4 * c4], o[4 * c4 + 1], o[4 * c4 + 2], o[4 * c4 + 3]);
                __syncwarp();
                PROF_ADD(3);
                uint32_t a[32];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int rr = 4 * i + sub;                       // slab row = tile row row0 + rr
                    ld_shared_v4(slab + rr * 128 + ((piece ^ (rr & 7)) << 4), a[4 * i], a[4 * i + 1], a[4 * i + 2], a[4 * i + 3]);
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int rr = 4 * i + sub;
                    if (rr < rows_here)
                        st_global_v4(gbase + size_t(rr) * kTileCols + q * 32, a[4 * i], a[4 * i + 1], a[4 * i + 2], a[4 * i + 3]);
                }
#endif
                PROF_ADD(4);
                if (!TCU_PIPE_STORE && q < 3) tmem_ld32(lane_base + slot * kTileCols + (q + 1) * 32, d);
            }
            if (lane == 0 && wq == 0) TRACE(t, 7);
            tc_fence_before();
            mbar_arrive(smem_u32(&ctl->acc_empty[slot]));
            // the carry ring entry of this tile (row prefixes, carry, barriers) may be reused
            mbar_arrive(smem_u32(&ctl->ring_free[ts]));
        }
        if (TCU_TMA_STORE && lane == 0) bulk_wait_all();
        if (lane == 0 && wq == 0) PROF_FLUSH(32 + 8 * group, 6);
    }

    // ---- tear-down
    PROF_STAMP(2);
    tc_fence_before();
    __syncthreads();
    PROF_STAMP(3);
    tc_fence_after();
    if (warp == 1) tmem_dealloc(tmem_base, 512);
    if (threadIdx.x == 0) {
        __threadfence();
        uint32_t old = atomicAdd(&hdr->done, 1u);
        if (old == gridDim.x - 1) {          // last CTA: the launch is over, open the next epoch
            hdr->done = 0;
            hdr->ticket = 0;
            __threadfence();
            hdr->epoch = my_epoch;
        }
    }
    PROF_STAMP(4);
}

// Tail of a single-array scan: the n % 128 elements after the last full 128-element row.
// Runs after the main kernel on the same stream; the carry is the inclusive record of the
// last tile (or nothing when there is no full row).
template <bool IS_INT, bool EXCL>
__global__ void tcu_scan_tail_kernel(const void *in, void *out, size_t start0, size_t pitch, uint32_t count, const void *ws,
                                     uint32_t tiles_per_row, uint32_t dtype, const void *carry_in) {
    // one block per scan (blockIdx.x = row of a batched scan)
    const size_t start = start0 + size_t(blockIdx.x) * pitch;
    const uint32_t tiles = (blockIdx.x + 1) * tiles_per_row;      // index + 1 of this scan's last tile record
    using CO = CarryOps<IS_INT>;
    using CarryT = typename CO::T;
    __shared__ CarryT warp_tot[4];
    const int tid = threadIdx.x, lane = tid & 31, wq = tid >> 5;
    CarryT carry = CarryT(0);
    if (carry_in && tiles_per_row == 0) {       // no full row before the tail: the continuation value is all there is
        const uint32_t bits = *reinterpret_cast<const uint32_t *>(carry_in);
        carry = IS_INT ? CarryT(bits) : CarryT(__uint_as_float(bits));
    }
    if (tiles_per_row > 0) {
        uint64_t flag, val;
        ld_record(reinterpret_cast<const uint8_t *>(ws) + kHeaderBytes + size_t(tiles - 1) * 16, flag, val);
        carry = CO::dec(val);
    }
    CarryT x = CarryT(0);
    if (tid < int(count)) {
        if (IS_INT) {
            x = CarryT(int32_t(reinterpret_cast<const int8_t *>(in)[start + tid]));
        } else {
            uint16_t b = reinterpret_cast<const uint16_t *>(in)[start + tid];
            float f = (dtype == 2) ? __uint_as_float(uint32_t(b) << 16) : __half2float(__ushort_as_half(b));
            x = CarryT(f);
        }
    }
    CarryT inc = x;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        CarryT up = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += up;
    }
    if (lane == 31) warp_tot[wq] = inc;
    __syncthreads();
    CarryT before = carry;
    for (int k = 0; k < wq; ++k) before += warp_tot[k];
    CarryT y = before + (EXCL ? (inc - x) : inc);
    if (EXCL && !IS_INT) {   // avoid the subtraction's rounding: rebuild the exclusive value from the neighbour
        CarryT left = __shfl_up_sync(0xffffffffu, inc, 1);
        y = before + (lane == 0 ? CarryT(0) : left);
    }
    if (tid < int(count)) {
        if (IS_INT) reinterpret_cast<uint32_t *>(out)[start + tid] = uint32_t(y);
        else reinterpret_cast<float *>(out)[start + tid] = float(y);
    }
}

// ---- two-sweep variant (for comparison with the single pass): sweep 1 reduces every tile to its
// total, a one-block scan turns the totals into inclusive sums and writes them as the records the main
// kernel's look-back expects, sweep 2 is the main kernel, whose look-back then succeeds at once.
template <bool IS_INT>
__global__ void __launch_bounds__(256) tcu_tile_totals_kernel(const void *in, void *ws, uint64_t valid_elems, uint32_t dtype) {
    using CO = CarryOps<IS_INT>;
    using CarryT = typename CO::T;
    __shared__ CarryT part[8];
    const uint32_t t = blockIdx.x;
    const uint64_t base = uint64_t(t) * kTileElems;
    CarryT acc = CarryT(0);
    if (IS_INT) {
        const int4 *src = reinterpret_cast<const int4 *>(reinterpret_cast<const int8_t *>(in) + base);
        int sum = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t idx = i * 256 + threadIdx.x;                   // 16-byte piece of the tile
            if (base + uint64_t(idx) * 16 < valid_elems) {
                int4 v = src[idx];
                sum = __dp4a(v.x, 0x01010101, sum);
                sum = __dp4a(v.y, 0x01010101, sum);
                sum = __dp4a(v.z, 0x01010101, sum);
                sum = __dp4a(v.w, 0x01010101, sum);
            }
        }
        acc = CarryT(uint32_t(sum));
    } else {
        const int4 *src = reinterpret_cast<const int4 *>(reinterpret_cast<const uint16_t *>(in) + base);
        float sum = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t idx = i * 256 + threadIdx.x;                   // 16-byte piece = 8 elements
            if (base + uint64_t(idx) * 8 < valid_elems) {
                int4 v = src[idx];
                const uint32_t w[4] = {uint32_t(v.x), uint32_t(v.y), uint32_t(v.z), uint32_t(v.w)};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    float lo, hi;
                    if (dtype == 2) {
                        lo = __uint_as_float(w[k] << 16);
                        hi = __uint_as_float(w[k] & 0xFFFF0000u);
                    } else {
                        lo = __half2float(__ushort_as_half(uint16_t(w[k] & 0xFFFF)));
                        hi = __half2float(__ushort_as_half(uint16_t(w[k] >> 16)));
                    }
                    sum += lo + hi;
                }
            }
        }
        acc = CarryT(sum);
    }
    acc = warp_sum(acc);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        CarryT tot = CarryT(0);
        for (int k = 0; k < 8; ++k) tot += part[k];
        reinterpret_cast<uint64_t *>(reinterpret_cast<uint8_t *>(ws) + kHeaderBytes)[2 * size_t(t) + 1] = CO::enc(tot);
    }
}

template <bool IS_INT>
__global__ void __launch_bounds__(1024) tcu_totals_scan_kernel(void *ws, uint32_t tiles) {
    using CO = CarryOps<IS_INT>;
    using CarryT = typename CO::T;
    __shared__ CarryT warp_part[32];
    __shared__ CarryT running;
    WsHeader *hdr = reinterpret_cast<WsHeader *>(ws);
    uint64_t *rec = reinterpret_cast<uint64_t *>(reinterpret_cast<uint8_t *>(ws) + kHeaderBytes);
    const uint64_t flag = (uint64_t(hdr->epoch + 1) << 2) | kStatusInclusive;   // the epoch the main kernel will use
    const uint32_t per = (tiles + 1023) / 1024;
    const uint32_t lo = threadIdx.x * per, hi = min(lo + per, tiles);
    CarryT mine = CarryT(0);
    for (uint32_t i = lo; i < hi; ++i) mine += CO::dec(rec[2 * size_t(i) + 1]);
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    CarryT inc = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        CarryT up = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += up;
    }
    if (lane == 31) warp_part[wid] = inc;
    __syncthreads();
    if (threadIdx.x == 0) {
        CarryT r = CarryT(0);
        for (int k = 0; k < 32; ++k) {
            CarryT v = warp_part[k];
            warp_part[k] = r;
            r += v;
        }
        running = r;
    }
    __syncthreads();
    CarryT acc = warp_part[wid] + (inc - mine);        // sum of everything before this thread's run
    for (uint32_t i = lo; i < hi; ++i) {
        acc += CO::dec(rec[2 * size_t(i) + 1]);
        rec[2 * size_t(i) + 1] = CO::enc(acc);
        rec[2 * size_t(i)] = flag;
    }
}

// Self-test of the bounded wait: one warp polls a tile record that nothing publishes, with a short
// limit, records TCU_ERR_TIMEOUT in the workspace header exactly as the scan kernel does, and returns.
__global__ void tcu_scan_timeout_selftest_kernel(void *ws, long long limit_cycles) {
    WsHeader *hdr = reinterpret_cast<WsHeader *>(ws);
    const uint8_t *rec = reinterpret_cast<const uint8_t *>(ws) + kHeaderBytes;
    const uint32_t epoch = ld_relaxed_u32(&hdr->epoch) + 1;     // a launch that never happens
    uint64_t flag = 0, val = 0;
    const long long c0 = clock64();
    bool gave_up = false;
    while (true) {
        __nanosleep(100);
        ld_record(rec, flag, val);
        if (static_cast<uint32_t>(flag >> 2) == epoch) break;
        if (clock64() - c0 > limit_cycles) {
            gave_up = true;
            break;
        }
    }
    if (__any_sync(0xffffffffu, gave_up) && threadIdx.x == 0) atomicExch(&hdr->error, 5u);
}

}  // namespace tcu
