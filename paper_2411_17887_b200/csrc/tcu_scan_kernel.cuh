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

#include <type_traits>

namespace tcu {

// ---- fixed design parameters (each was chosen by measurement; the alternatives that lost are not kept)
constexpr int kStoreGroups = 2;               // groups of four store warps; group g takes the tiles with j % 2 == g
constexpr uint32_t kPrefetchDist = 256;       // tiles ahead of the claimed one that are prefetched into L2
constexpr int kUseInStages = 10;              // most input stages the host will ask for

constexpr int kTileRows = 128;          // rows of a tile = M of the MMA = TMEM lanes
constexpr int kTileCols = 128;          // elements per tile row
constexpr int kTileElems = kTileRows * kTileCols;
constexpr int kNumAcc = 3;              // TMEM accumulators of the local scans (128 columns each)
constexpr int kNumTot = 8;              // TMEM accumulators of the row totals (16 columns each)
constexpr int kTotCols = 16;
constexpr int kTotBase = kNumAcc * kTileCols;            // first TMEM column of the totals ring
static_assert(kTotBase + kNumTot * kTotCols <= 512, "TMEM has 512 columns");
constexpr int kSlabBytes = 32 * 4 * 32;                  // output staging unit: 32 columns x 32 rows of 4 bytes, written by one warp
constexpr int kOutRingBytes = kStoreGroups * 4 * kSlabBytes;   // one staging slab per store warp
constexpr int kNumCarry = 16;           // tiles a CTA may have between "row totals known" and "stored": ring of carry entries
constexpr int kTileRing = 32;           // ring of claimed tile numbers (must exceed the tiles a CTA has in flight)
constexpr uint32_t kNoTile = 0xFFFFFFFFu;   // "no more tiles" marker pushed through the pipeline
constexpr int kNumLookbackWarps = 5;
constexpr int kNumMarkers = kNumLookbackWarps;   // markers pushed: one per look-back warp
constexpr int kMaxInStages = 12;        // size of the barrier arrays
constexpr int kAtomBytes = 128 * kTileRows;   // one 128-byte-swizzled block of 128 rows
constexpr int kOnesBytes = 16 * 128;          // constant operand of the row-total product: 16 rows of ones
constexpr int kDownBytes = (kStoreGroups + 1) * kAtomBytes;   // carry-product variant: one carry operand per store group + a ones operand
// upper levels as products: a strictly lower triangular all-ones operand (128 x 128: one 128-byte-swizzled block of
// int8, two of bf16) and the operand that holds the narrow terms of the 128 row totals (16 rows: 2 KB per block)
constexpr int kUpperHalfBytes = 16 * 128;
constexpr int kUpperBytesInt = kAtomBytes + kUpperHalfBytes;
constexpr int kUpperBytesFloat = 2 * kAtomBytes + 2 * kUpperHalfBytes;
constexpr int kSegNoteBytes = kTileRows + 4 * kTileRows;   // segmented scan: per tile, a flag byte and a 4-byte value per row
constexpr int kSegRingBytes = kNumCarry * kSegNoteBytes;  // one entry per carry-ring entry (reused only after the tile is stored)
// chunk level as a product (kernel variant CHUNK_TC): per store group an operand with the narrow terms of the chunk totals
// of the 128 rows (one 128-byte-swizzled block), a constant operand of at most 32 rows, and 32 TMEM columns for the result
constexpr int kChunkConstBytes = 32 * 128;
constexpr int kChunkBytes = kStoreGroups * kAtomBytes + kChunkConstBytes;
constexpr int kChunkNumTot = 4;         // row-total accumulators left when the chunk products take 64 TMEM columns
constexpr int kChunkScratch = kTotBase + kChunkNumTot * kTotCols;    // first TMEM column of the chunk products' results
constexpr int kEpilogueThreads = 128;
// Registers per thread after re-allocation.  The pool is what the CTA was launched with (80 x 768 or
// 96 x 640 = 61440 registers), so 128 x (64 + 80 + 72 + kStoreGroups x kStoreRegs) must not exceed it:
// an increase that cannot be granted would block.
constexpr int kStoreRegs = 128;
static_assert(128 * (64 + 80 + 72 + kStoreGroups * kStoreRegs) <= 61440, "register pool");
constexpr int kFirstStoreWarp = 4;                                   // carry add and store: kStoreGroups x 4 warps
constexpr int kFirstTotalsWarp = kFirstStoreWarp + 4 * kStoreGroups; // totals of rows and tile: 4 warps
constexpr int kFirstLookbackWarp = kFirstTotalsWarp + 4;             // cross-tile look-back (warp 3 is one more)
constexpr int kThreads = 32 * (kFirstLookbackWarp + kNumLookbackWarps - 1);
// The register re-allocation below assumes that the kernel is compiled at 96 registers per thread, which is what
// 640 threads per CTA give.  With more threads the compiler settles on fewer (80 at 672), and a setmaxnreg.dec to a
// value above the current allocation is an illegal instruction: do not add warps without redoing the numbers.
static_assert(kThreads == 640, "register re-allocation is laid out for 640 threads at 96 registers");

// workspace: 256-byte header, then one 16-byte record per tile
constexpr int kHeaderBytes = 256;
constexpr uint32_t kStatusPartial = 1;    // record holds the tile's own total
constexpr uint32_t kStatusInclusive = 2;  // record holds the sum of everything up to and including the tile
struct WsHeader {
    uint32_t epoch;      // launches completed on this workspace
    uint32_t done;       // CTAs of the running launch that have finished
    uint32_t error;      // tcu_status_t recorded by a bounded wait that ran out
    uint32_t ticket;     // next tile number to hand out (tiles are claimed in increasing order)
    uint64_t carry_slot[2];   // scratch for a caller that chains scans: totals handed from one launch to the next
    uint32_t pad[56];
};
static_assert(sizeof(WsHeader) == kHeaderBytes, "header size");

// ---- debug section (compiled only with -DTCU_PROFILE; the product build defines every macro to nothing) -------------
// Per-CTA cycle counters of where each role waits (64 counters per CTA) and eight time stamps per tile.
#ifdef TCU_PROFILE
__device__ unsigned long long *g_prof = nullptr;
#define PROF_DECL long long prof_t = 0; unsigned long long prof_a[8] = {0, 0, 0, 0, 0, 0, 0, 0}; (void)prof_t;
#define PROF_T0() prof_t = clock64()
#define PROF_ADD(k) do { long long n_ = clock64(); prof_a[k] += (unsigned long long)(n_ - prof_t); prof_t = n_; } while (0)
#define PROF_INC(k, v) prof_a[k] += (v)
#define PROF_FLUSH(base, cnt) do { if (g_prof) for (int i_ = 0; i_ < (cnt); ++i_) g_prof[blockIdx.x * 64 + (base) + i_] = prof_a[i_]; } while (0)
__device__ unsigned long long *g_trace = nullptr;
#define TRACE(tile, k) do { if (g_trace) g_trace[size_t(tile) * 8 + (k)] = global_timer_ns(); } while (0)
#else
#define TRACE(tile, k)
#define PROF_DECL
#define PROF_T0()
#define PROF_ADD(k)
#define PROF_INC(k, v)
#define PROF_FLUSH(base, cnt)
#endif
// ---- end of the debug section ------------------------------------------------------------------------------------------

__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t) : : "memory");
    return t;
}

// Optional time stamps of one launch (ScanParams::stamps, normally NULL): kStampsPerCta values of %globaltimer
// per CTA, taken by whichever thread passes the point first for the CTA's first tile.
constexpr int kStampsPerCta = 16;
enum Stamp {
    kStampEntry = 0,        // kernel entered
    kStampSetupDone = 1,    // barriers, TMEM and constant operands ready
    kStampDepsDone = 2,     // the previous kernel of the stream has finished (global memory may be touched)
    kStampClaimed = 3,      // first tile claimed, its load issued
    kStampLanded = 4,       // first tile in shared memory
    kStampPublished = 5,    // first tile's total published
    kStampCarry = 6,        // first tile's cross-tile carry known
    kStampStored = 7,       // first tile written
    kStampLoopsDone = 8,    // thread 0 reached the tear-down barrier
    kStampAllDone = 9,      // every warp reached it
    kStampExit = 10,        // TMEM freed, launch counter updated
    kStampTiles = 11        // (not a time) tiles this CTA processed
};

// segmented scan: what is noted about a 128-element row of the array that holds a segment start
constexpr uint32_t kRowCutIn = 1;      // a segment starts at element 0 of the row: nothing carries into it
constexpr uint32_t kRowHasStart = 2;   // a segment starts somewhere in the row: it hands on the sum from its last start
constexpr long long kSpinLimitCycles = 2000000000LL;   // default limit of every wait: about one second at B200 clocks

struct alignas(64) ScanParams {
    CUtensorMap tmap_in;      // (128, rows128, batch) view of the input, box 128 B x 128 rows
    void *ws;
    void *out;                // output array (4-byte elements)
    const void *carry_in;     // optional (single array): 8-byte carry (a double, or a zero-extended uint32) that precedes the scan
    void *carry_out;          // optional (single array): receives carry_in + the total of the full rows, in the same 8-byte form
    unsigned long long *stamps;   // optional: kStampsPerCta time stamps per CTA (see enum Stamp)
    uint64_t scan_pitch;      // elements between consecutive scans (batched), unused for a single array
    long long spin_limit;     // cycles after which a wait gives up
    uint32_t rows128;         // full 128-element rows of one scan
    uint32_t tiles_total;     // all tiles of the launch
    uint32_t tiles_per_row;   // tiles of one scan (carry chain restarts every tiles_per_row tiles)
    uint32_t in_stages;       // depth of the input ring
    uint32_t b_bytes;         // shared memory reserved for the constant operand I (x) U_s
    uint32_t dtype;           // tcu_dtype_t
    uint32_t level0_only;     // debug: stop after the U_s product (no carries)
    uint32_t prefilled;       // two-sweep variant: the records already hold every tile's inclusive sum
    uint32_t down_tc;         // 16-bit input, s = 128 only: add the row carries with a tensor-core product (B_s-style down-sweep)
    uint32_t upper_tc;        // scan the 128 row totals with a second triangular product on exact narrow terms (8-bit limbs / bf16 terms)
    uint32_t skip_publish_tile;   // self-test of the bounded waits: the records of this tile are never published (kNoTile: none)
    // segmented scan (single array): per 128-element row of the array, a flag byte (kRowCutIn, kRowHasStart) and,
    // for rows with a start, the sum from the last start to the end of the row; NULL for an ordinary scan
    const uint8_t *seg_rowflag;
    const uint32_t *seg_rowval;
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
    uint32_t warp_cut[2][4];         // ... and whether a segment starts in the warp's 32 rows
    uint32_t seg_cut[kNumCarry][4];  // bit r: the carry from before the tile does not reach row r (a segment starts before it)
    uint32_t agg_cut[kNumCarry];     // a segment starts inside the tile: its total is the sum since the last start
    uint32_t tile_of[kTileRing];     // tile number of the j-th tile claimed by this CTA
    uint32_t tmem_base;
    uint32_t epoch;
    uint64_t carry_in_bits;          // value at *carry_in (0 when there is none)
    uint64_t epoch_ready;            // thread 0 -> totals and look-back warps: epoch and carry_in_bits are written
    uint64_t up_done;                // limb product of the row totals -> totals warps
    uint64_t down_done[kStoreGroups];   // carry product -> store warps of a group
    uint64_t mma_drained[2];         // after a give-up: the MMAs an issuer warp still had in flight have completed
    uint64_t chunk_done[kStoreGroups];  // chunk product -> store warps of a group
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
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(bar)
        : "memory");
}
// Untiled bulk copy global -> shared (both addresses 16-byte aligned, size a multiple of 16), completing on an mbarrier.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
// Ask the TMA unit to bring a box into L2 only (no shared-memory destination, no completion signal).
__device__ __forceinline__ void tma_prefetch_l2_3d(const CUtensorMap *map, int x, int y, int z) {
    asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];"
                 ::"l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z)
                 : "memory");
}
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
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N));
}
template <int N>
__device__ __forceinline__ void reg_inc() {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N));
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
    asm volatile("st.global.v4.b32 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
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
    long long limit;
    // Wait for the phase of `bar` with the given parity; false when the wait was given up.
    __device__ __forceinline__ bool wait(uint32_t bar, uint32_t parity) const {
        if (mbar_try_wait(bar, parity)) return true;
        long long t0 = clock64();
        uint32_t spins = 0;
        while (!mbar_try_wait(bar, parity)) {
            if ((++spins & 0xFF) == 0) {
                if (ctl->abort_flag) return false;
                if (clock64() - t0 > limit) {
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
// VARIANT: kLean = the plain scan (inclusive / exclusive, single array or dense rows, optional carry in): every option
// below is compiled out; kFull = all run-time options (upper-level and down-sweep products, segments, two-sweep
// records, level-0 debug output, time stamps, the self-test's silent tile, carry out); kChunk = kFull plus the chunk
// level as a product.  The plain scan gets a kernel of its own because the options cost it 2-3 % even when they are
// switched off (measured on 16-bit input: 251 -> 245 µs at n = 2^28, 69.4 -> 67.8 at 2^26, 6.3 -> 5.9 at 2^16) -
// code size and register allocation of a kernel whose 20 warps run five different programs.
enum ScanVariant { kLean = 0, kFull = 1, kChunk = 2 };
template <bool IS_INT, int S, bool EXCL, int VARIANT = kLean>
__global__ void __launch_bounds__(kThreads, 1) tcu_scan_kernel(const __grid_constant__ ScanParams p) {
    constexpr bool FULL = VARIANT != kLean, CHUNK_TC = VARIANT == kChunk;
    static_assert(!CHUNK_TC || S < kTileCols, "a row of s = 128 is one chunk: there is no chunk level");
    const bool use_upper = FULL && p.upper_tc != 0, use_down = FULL && p.down_tc != 0, segmented = FULL && p.seg_rowflag != nullptr;
    const bool level0_only = FULL && p.level0_only != 0, prefilled = FULL && p.prefilled != 0, use_stamps = FULL && p.stamps != nullptr;
    const bool has_carry_out = FULL && p.carry_out != nullptr;
    const uint32_t skip_tile = FULL ? p.skip_publish_tile : kNoTile;
    constexpr int kTotRing = CHUNK_TC ? kChunkNumTot : kNumTot;   // depth of the ring of row-total accumulators
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
    uint8_t *seg_ring = out_ring + kOutRingBytes;         // only present for a segmented scan (never together with the two below)
    uint8_t *upper_a = out_ring + kOutRingBytes;          // only present when use_upper
    uint8_t *upper_b = upper_a + (IS_INT ? 1 : 2) * kAtomBytes;
    uint8_t *down_a = upper_a + (use_upper ? (IS_INT ? kUpperBytesInt : kUpperBytesFloat) : 0);   // only present when use_down
    uint8_t *down_b = down_a + kStoreGroups * kAtomBytes;
    uint8_t *chunk_a = upper_a + (use_upper ? (IS_INT ? kUpperBytesInt : kUpperBytesFloat) : 0);   // only present in the CHUNK_TC variant
    uint8_t *chunk_b = chunk_a + kStoreGroups * kAtomBytes;
    uint8_t *chunk_sel = chunk_b + kChunkConstBytes;       // only present in the CHUNK_TC variant with use_down

    WsHeader *hdr = reinterpret_cast<WsHeader *>(p.ws);
    uint8_t *records = reinterpret_cast<uint8_t *>(p.ws) + kHeaderBytes;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t num_in = p.in_stages;

    // Optional time stamps (p.stamps is NULL in normal use): each point is passed by one designated thread.
    auto stamp = [&](int k) {
        if (use_stamps) p.stamps[size_t(blockIdx.x) * kStampsPerCta + k] = global_timer_ns();
    };

    // ---- set-up
    if (threadIdx.x == kThreads - 1 && kPrefetchDist > 0) {
        // The producers prefetch tile t + kPrefetchDist into L2 when they claim tile t, which leaves the first
        // kPrefetchDist tiles of the launch to nobody: start their trip from DRAM now, before the set-up, the wait
        // for the previous kernel and the first ticket (a prefetch moves data into L2, the point of coherence, so it
        // may run ahead of a previous kernel that is still writing the input).
        for (uint32_t tp = blockIdx.x; tp < kPrefetchDist && tp < p.tiles_total; tp += gridDim.x) {
            const int prow = tp / p.tiles_per_row, plt = tp % p.tiles_per_row;
#pragma unroll
            for (int a = 0; a < kInAtoms; ++a)
                tma_prefetch_l2_3d(&p.tmap_in, a * (128 / kElemBytes), plt * kTileRows, prow);
        }
    }
    if (threadIdx.x == 0) {
        stamp(kStampEntry);
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&p.tmap_in)) : "memory");
        mbar_init(smem_u32(&ctl->epoch_ready), 1);
        mbar_init(smem_u32(&ctl->up_done), 1);
        for (int g = 0; g < kStoreGroups; ++g) mbar_init(smem_u32(&ctl->down_done[g]), 1);
        for (int g = 0; g < 2; ++g) mbar_init(smem_u32(&ctl->mma_drained[g]), 1);
        for (int g = 0; g < kStoreGroups; ++g) mbar_init(smem_u32(&ctl->chunk_done[g]), 1);
        ctl->abort_flag = 0;
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
    if (warp == 1) {
        tmem_alloc(smem_u32(&ctl->tmem_base), 512);
        tmem_relinquish();
    }
    // Constant operands, written as whole 16-byte pieces (the unit of the 128-byte swizzle): piece c of row n
    // sits at n * 128 + ((c ^ (n & 7)) << 4) inside its 128-row block.  Only the pieces the products read are
    // written; nothing else of the region is ever looked at.
    {
        const uint32_t one16 = (p.dtype == 2) ? 0x3F80u : 0x3C00u;              // 1.0 in bf16 / fp16
        const uint32_t ones = IS_INT ? 0x01010101u : (one16 | (one16 << 16));
        // operand of the row-total product: all ones, so every 32-byte K-slice of it is the same block
        if (threadIdx.x < kOnesBytes / 16) st_shared_v4(smem_u32(ones_region) + threadIdx.x * 16, ones, ones, ones, ones);
        // I (x) U_s, K-major: row n holds column n of the matrix, i.e. ones at the k <= n of the same s-block
        // (U_s is L_s transposed: X U_s = (L_s X^T)^T)
        constexpr int kPerPiece = 16 / kElemBytes;                              // K entries per 16-byte piece
        constexpr int kPiecesPerRow = kSeff / kPerPiece;                        // pieces of a row that the products read
        const uint32_t cbase = smem_u32(const_region);
        for (int e = threadIdx.x; e < kSeff * kPiecesPerRow; e += kThreads) {
            const int n = e / kPiecesPerRow, c = e % kPiecesPerRow;             // (powers of two: shifts and masks)
            const int lo = n & ~(S - 1);                                        // first k of the block that row n belongs to
            uint32_t wd[4] = {0u, 0u, 0u, 0u};
#pragma unroll
            for (int i = 0; i < kPerPiece; ++i) {
                const int k = c * kPerPiece + i;
                if (k >= lo && k <= n) {
                    if (IS_INT) wd[i >> 2] |= 1u << (8 * (i & 3));
                    else wd[i >> 1] |= one16 << (16 * (i & 1));
                }
            }
            st_shared_v4(cbase + (c >> 3) * kAtomBytes + n * 128 + (((c & 7) ^ (n & 7)) << 4), wd[0], wd[1], wd[2], wd[3]);
        }
        if (!IS_INT && use_down && !CHUNK_TC) {
            // carry operands start as zeros (only 3 of the 16 K-entries of a row are ever written); the other
            // operand is all ones in bf16
            for (int e = threadIdx.x; e < kStoreGroups * kAtomBytes / 16; e += kThreads) st_shared_v4(smem_u32(down_a) + e * 16, 0u, 0u, 0u, 0u);
            for (int e = threadIdx.x; e < kAtomBytes / 16; e += kThreads)
                st_shared_v4(smem_u32(down_b) + e * 16, 0x3F803F80u, 0x3F803F80u, 0x3F803F80u, 0x3F803F80u);
        }
        if (use_upper) {
            // A[m][k] = 1 for k < m: its product with a column of row totals is their exclusive scan over the rows
            // (int8 ones for integer scans, bf16 ones otherwise: 16 or 8 K entries per 16-byte piece)
            constexpr int kUpPerPiece = IS_INT ? 16 : 8;
            constexpr int kUpPieces = kTileRows / kUpPerPiece;
            for (int e = threadIdx.x; e < kTileRows * kUpPieces; e += kThreads) {
                const int m = e / kUpPieces, c = e % kUpPieces;
                uint32_t wd[4] = {0u, 0u, 0u, 0u};
#pragma unroll
                for (int i = 0; i < kUpPerPiece; ++i) {
                    if (c * kUpPerPiece + i < m) {
                        if (IS_INT) wd[i >> 2] |= 1u << (8 * (i & 3));
                        else wd[i >> 1] |= 0x3F80u << (16 * (i & 1));
                    }
                }
                st_shared_v4(smem_u32(upper_a) + (c >> 3) * kAtomBytes + m * 128 + (((c & 7) ^ (m & 7)) << 4), wd[0], wd[1], wd[2], wd[3]);
            }
            for (int e = threadIdx.x; e < (IS_INT ? 1 : 2) * kUpperHalfBytes / 16; e += kThreads) st_shared_v4(smem_u32(upper_b) + e * 16, 0u, 0u, 0u, 0u);
        }
        if (CHUNK_TC) {
            // Chunk level as a product: the K index of the data operand is (chunk g', term l') = kTerms g' + l', the
            // result column is (chunk g, term l) = kTerms g + l, and the constant operand (stored K-major: row n holds
            // column n) has ones where l' = l and g' < g: column (g, l) of the result is the sum of term l over the
            // chunks before g - a strictly upper triangular U_{128/s}, once per term.
            constexpr int kTerms = IS_INT ? 2 : 3, kCPerPiece = IS_INT ? 16 : 8, kCPieces = 32 / kCPerPiece;
            for (int e = threadIdx.x; e < 32 * kCPieces; e += kThreads) {
                const int n = e / kCPieces, c = e % kCPieces;
                uint32_t wd[4] = {0u, 0u, 0u, 0u};
#pragma unroll
                for (int i = 0; i < kCPerPiece; ++i) {
                    const int k = c * kCPerPiece + i;
                    const bool used = n < kTerms * (kTileCols / S) && k < kTerms * (kTileCols / S);
                    if (used && (k % kTerms) == (n % kTerms) && (k / kTerms) < (n / kTerms)) {
                        if (IS_INT) wd[i >> 2] |= 1u << (8 * (i & 3));
                        else wd[i >> 1] |= 0x3F80u << (16 * (i & 1));
                    }
                }
                st_shared_v4(smem_u32(chunk_b) + n * 128 + ((c ^ (n & 7)) << 4), wd[0], wd[1], wd[2], wd[3]);
            }
            // the data operands start as zeros: only the first pieces of a row are ever rewritten
            for (int e = threadIdx.x; e < kStoreGroups * kAtomBytes / 16; e += kThreads) st_shared_v4(smem_u32(chunk_a) + e * 16, 0u, 0u, 0u, 0u);
            if (!IS_INT && use_down) {
                // Down-sweep as a product for s < 128 (the paper's B_s: the carry of what precedes a chunk is added to
                // every element of the chunk by a matrix product).  The data operand holds, per row, the carry of each
                // of its chunks in three bf16 terms (K index = 3 g + l, like the chunk totals above); this constant
                // operand (stored K-major: row n = output column n) has ones where the K index belongs to the chunk
                // of column n, so that accumulator[r][n] += carry[r][chunk of n].
                for (int e = threadIdx.x; e < kTileCols * 8; e += kThreads) {
                    const int n = e >> 3, c = e & 7;
                    uint32_t wd[4] = {0u, 0u, 0u, 0u};
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int k = c * 8 + i;
                        if (k < 3 * (kTileCols / S) && k / 3 == n / S) wd[i >> 1] |= 0x3F80u << (16 * (i & 1));
                    }
                    st_shared_v4(smem_u32(chunk_sel) + n * 128 + ((c ^ (n & 7)) << 4), wd[0], wd[1], wd[2], wd[3]);
                }
            }
        }
        fence_proxy_async_smem();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    if (threadIdx.x == 0) stamp(kStampSetupDone);
    // Everything above touched only this CTA's shared memory and TMEM, so under programmatic dependent launch it
    // may run while the previous kernel of the stream is still finishing.  From here on global memory is read.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const uint32_t tmem_base = ctl->tmem_base;
    Waiter w{ctl, hdr, p.spin_limit};
    uint32_t first_ticket = 0;                 // (thread 0 only) first tile of this CTA
    uint32_t my_epoch = 0;                     // (thread 0 only) the epoch of this launch
    if (threadIdx.x == 0) {
        stamp(kStampDepsDone);
        first_ticket = atomicAdd(&hdr->ticket, 1u);
        my_epoch = ld_relaxed_u32(&hdr->epoch) + 1;
        ctl->epoch = my_epoch;
        // what precedes the whole scan (continuation of an earlier piece or shard); only single-array calls pass one
        ctl->carry_in_bits = p.carry_in ? *reinterpret_cast<const uint64_t *>(p.carry_in) : 0ull;
        mbar_arrive(smem_u32(&ctl->epoch_ready));
    }

    // The j-th tile handled by this CTA is number tile_of[j % kTileRing].  Tiles are claimed at run time with a
    // ticket counter in the workspace, in increasing order: whoever holds tile t knows that every tile before t
    // is held by a CTA that is already running.  Nothing is assumed about which CTAs of the grid are resident or in
    // which order they start (a CTA that has not started holds no tile), so a launch that shares the GPU with another
    // kernel still makes progress; handing tile b to CTA b would save the first ticket's round trip, but not keep that.
    // When the tiles run out the producer pushes kNumMarkers "no more
    // tiles" markers through the pipeline, so that every role - and each of the look-back warps, which take the
    // tiles in turns - meets one and stops.
    // Sum of the totals of the tiles before `t`, back to the first tile t0 of the scan or to the nearest tile whose
    // record already holds an inclusive sum.  Every lane fetches W records per round (distance k * 32 + lane behind
    // the current position), so that a stretch of 32 * W predecessors costs one round trip to L2; the windows are
    // then examined nearest first, and only a window that is actually needed is waited for.
    auto walk = [&](auto width_tag, const int t, const int t0, const uint32_t epoch, bool &gave_up, uint32_t &rounds) -> CarryT {
        constexpr int W = decltype(width_tag)::value;
        CarryT sum = CarryT(0);
        int pos = t - 1;
        while (true) {
            uint64_t flag[W], val[W];
#pragma unroll
            for (int k = 0; k < W; ++k) {
                const int idx = pos - (k * 32 + lane);
                flag[k] = 0;
                val[k] = 0;
                if (idx >= t0) ld_record(records + size_t(idx) * 16, flag[k], val[k]);
            }
            CarryT part = CarryT(0);
            bool done = false;
#pragma unroll
            for (int k = 0; k < W; ++k) {
                if (!done) {                               // warp-uniform
                    const int idx = pos - (k * 32 + lane);
                    const bool valid = idx >= t0;
                    if (valid && static_cast<uint32_t>(flag[k] >> 2) != epoch) {
                        const void *rec = records + size_t(idx) * 16;
                        const long long c0 = clock64();
                        uint32_t spins = 0;
                        while (true) {
                            __nanosleep(20);
                            ld_record(rec, flag[k], val[k]);
                            if (static_cast<uint32_t>(flag[k] >> 2) == epoch) break;
                            if ((++spins & 0x3F) == 0 && (ctl->abort_flag || clock64() - c0 > p.spin_limit)) {
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
                        const int first = __ffs(m) - 1;    // nearest predecessor whose record is inclusive
                        if (lane > first) v = CarryT(0);
                        done = true;
                    }
                    part += v;
                    if (pos - (k * 32 + 31) <= t0) done = true;   // the window reached the first tile of the scan
                }
            }
            sum += warp_sum(part);
            ++rounds;
            if (done) break;
            pos -= 32 * W;
            if (pos < t0) break;
        }
        return sum;
    };

    // ------------------------------------------------------------------ cross-tile carry scan (role of warp 3 and warps 16-19)
    // kNumLookbackWarps warps take the tiles in turn, so that the walks of the tiles in flight overlap.
    auto lookback_role = [&](const uint32_t lbw) {
        if (!__all_sync(0xffffffffu, w.wait(smem_u32(&ctl->epoch_ready), 0))) return;
        const uint32_t epoch = ctl->epoch;
        const CarryT carry_in = CO::dec(ctl->carry_in_bits);
        PROF_DECL
        PROF_T0();
        for (uint32_t j = lbw;; j += kNumLookbackWarps) {
            const uint32_t ts = j % kNumCarry, ut = j / kNumCarry;
            CarryT prefix = CarryT(0);
            bool gave_up = false;
            uint32_t rounds = 0;
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
            if (static_cast<int>(t) == t0) {
                prefix = carry_in;                 // (the first tile's record was published by the totals warps)
            } else {
                // One window of 32 records per round: the later a record is read the more likely it already holds an
                // inclusive sum.  Measured alternatives, all slower: walks that start as soon as the tile is claimed
                // (before its own total is known), rounds that fetch several windows at once, runs of consecutive
                // tiles per CTA with the carry passed on locally - each covers more ground per tile or delays the
                // records of the followers, and costs a long scan 8-25 % of its throughput; a separate wide walk
                // for the first tiles of a launch (inlined or not) slows the ordinary walk by 2-6 %.
                prefix = walk(std::integral_constant<int, 1>{}, static_cast<int>(t), t0, epoch, gave_up, rounds);
                if (__any_sync(0xffffffffu, gave_up) && lane == 0) {
                    ctl->abort_flag = 1;
                    atomicExch(&hdr->error, 5u);
                }
                // publish even after a give-up so that successors do not wait for this tile (a tile in which a
                // segment starts has already published its final record)
                if (lane == 0 && !prefilled && t != skip_tile && !(segmented && ctl->agg_cut[ts]))
                    st_record(records + size_t(t) * 16, (uint64_t(epoch) << 2) | kStatusInclusive, CO::enc(prefix + agg));
            }
            if (lane == 0) {
                TRACE(t, 5);
                ctl->carry_slot[ts] = CO::enc(prefix);
                mbar_arrive(smem_u32(&ctl->carry_ready[ts]));
                if (has_carry_out && t + 1 == p.tiles_total) *reinterpret_cast<uint64_t *>(p.carry_out) = CO::enc(prefix + agg);
                if (j == 0) stamp(kStampCarry);
            }
            __syncwarp();
            PROF_ADD(1);
            PROF_INC(2, rounds);
            PROF_INC(3, 1);
        }
        if (lane == 0) PROF_FLUSH(12 + 4 * (lbw % 4), 4);
    };

    // After a give-up an MMA issuer may leave its loop with products still in flight; TMEM must not be freed
    // under them.  A commit completes when everything this thread issued before it has, so: commit to a
    // barrier of its own and wait for it (bounded like every other wait).
    auto mma_drain = [&](int which) {
        if (!ctl->abort_flag) return;
        const uint32_t bar = smem_u32(&ctl->mma_drained[which]);
        mma_commit(bar);
        const long long t0 = clock64();
        while (!mbar_try_wait(bar, 0) && clock64() - t0 < p.spin_limit) {}
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
                if (markers == 0) t = (j == 0) ? first_ticket : atomicAdd(&hdr->ticket, 1u);
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
                const bool seg = segmented;
                mbar_expect_tx(bar, kStageBytes + (seg ? kSegNoteBytes : 0));
                if (seg) {
                    // the notes about the tile's rows travel with the tile: two bulk copies that complete on the
                    // same barrier, into the entry of the tile's carry-ring slot (free again since tile j - 16 was
                    // stored, which this claim already implies)
                    const uint32_t dst = smem_u32(seg_ring + (j % kNumCarry) * kSegNoteBytes);
                    bulk_load(dst, p.seg_rowflag + size_t(t) * kTileRows, kTileRows, bar);
                    bulk_load(dst + kTileRows, p.seg_rowval + size_t(t) * kTileRows, 4 * kTileRows, bar);
                }
                int scan_row = t / p.tiles_per_row, lt = t % p.tiles_per_row;
#pragma unroll
                for (int a = 0; a < kInAtoms; ++a)
                    tma_load_3d(smem_u32(in_ring + stage * kStageBytes + a * kAtomBytes), &p.tmap_in,
                                a * (128 / kElemBytes), lt * kTileRows, scan_row, bar);
                issued = j + 1;
                if (j == 0) stamp(kStampClaimed);
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
            // This CTA draws no more tickets and has read the epoch: count it.  The last CTA of the launch to get
            // here opens the next epoch and re-arms the ticket counter; nobody of this launch looks at either
            // again (records are compared with the copy of the epoch in shared memory), and the next launch
            // reads them only after this one has completed.  Doing it here, not at the end of the CTA, keeps
            // the round trip of the atomic off the tail of the kernel.
            {
                const uint32_t arrived = atomicAdd(&hdr->done, 1u);
                if (arrived == gridDim.x - 1) {
                    hdr->done = 0;
                    hdr->ticket = 0;
                    __threadfence();
                    hdr->epoch = my_epoch;
                }
            }
            if (ctl->abort_flag) {
                // drain: loads already issued must land before the CTA may exit
                uint32_t lo = issued > num_in ? issued - num_in : 0;
                for (uint32_t j = lo; j < issued; ++j) {
                    uint32_t bar = smem_u32(&ctl->full[j % num_in]);
                    uint32_t par = (j / num_in) & 1;
                    long long t0 = clock64();
                    while (!mbar_try_wait(bar, par) && clock64() - t0 < p.spin_limit) {}
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
                if (j == 0) stamp(kStampLanded);
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
            mma_drain(0);
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
                uint32_t ts = j % kTotRing, ut = j / kTotRing;
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
            mma_drain(1);
        }
    } else {
        lookback_role(0);
    }
    } else if (warp >= kFirstLookbackWarp) {
        reg_dec<80>();
        lookback_role(uint32_t(warp - kFirstLookbackWarp + 1));
    } else if (warp >= kFirstTotalsWarp) {
        reg_dec<72>();
        // ------------------------------------------------------------------ totals (up-sweep above the product)
        // Takes the 128 row totals from the small accumulator, scans them across the rows, and
        // publishes the tile total - as soon as the tile has landed, so that the cross-tile look-back
        // has several tile times to complete before the store warps need its result.
        const int r = threadIdx.x - kFirstTotalsWarp * 32;          // tile row owned by this thread = TMEM lane
        const int wq = r >> 5;
        const uint32_t lane_base = tmem_base + (uint32_t(wq * 32) << 16);
        const bool epoch_ok = w.wait(smem_u32(&ctl->epoch_ready), 0);
        const uint32_t epoch = ctl->epoch;
        const CarryT carry_in = CO::dec(ctl->carry_in_bits);
        uint32_t markers = 0;
        PROF_DECL
        PROF_T0();
        for (uint32_t j = 0;; ++j) {
            const uint32_t tt = j % kTotRing, utt = j / kTotRing;    // row-total accumulator in TMEM
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
            uint32_t seg_fl = 0, seg_rv = 0;                          // segmented scan: this row's notes
            if (segmented) {
                // the notes of the tile's 128 rows came in with the tile (bulk copies issued by the producer)
                const uint8_t *notes = seg_ring + ts * kSegNoteBytes;
                seg_fl = notes[r];
                seg_rv = reinterpret_cast<const uint32_t *>(notes + kTileRows)[r];
            }
            tc_fence_after();
            const uint32_t rowtot = tmem_ld1(lane_base + kTotBase + tt * kTotCols);
            tmem_ld_wait();
            if (use_upper) {
                // Paper-faithful variant of this level: the scan over the 128 row totals is itself a product
                // with a triangular all-ones matrix, D[m][n] = sum over k < m of term n of total k.  Row totals
                // are int32 / fp32, not tensor-core input types, so each is first split exactly into narrow
                // terms, which become rows n of the second operand (K index = tile row):
                //   int8 input:  two signed 8-bit limbs, total = 128 h + l (|total| <= 2^14), one kind::i8 product;
                //   16-bit input: three bf16 terms, total = hi + mid + lo (8 significant bits each), one
                //                 kind::f16 product with fp32 accumulation.
                // The results are recombined afterwards (shift and add; three fp32 additions).
                const uint32_t ub = smem_u32(upper_b);
                uint32_t exc_all, tile_total;
                if (IS_INT) {
                    const int32_t tot = int32_t(rowtot);
                    asm volatile("st.shared.u8 [%0], %1;" ::"r"(ub + 0 * 128 + ((((r >> 4) ^ 0) << 4) | (r & 15))), "r"(tot & 127) : "memory");
                    asm volatile("st.shared.u8 [%0], %1;" ::"r"(ub + 1 * 128 + ((((r >> 4) ^ 1) << 4) | (r & 15))), "r"((tot >> 7) & 0xFF) : "memory");
                } else {
                    const uint32_t hi = rowtot & 0xFFFF0000u;
                    const float r1 = __uint_as_float(rowtot) - __uint_as_float(hi);
                    const uint32_t mid = __float_as_uint(r1) & 0xFFFF0000u;
                    const float r2 = r1 - __uint_as_float(mid);
                    const uint32_t lo = __float_as_uint(r2) & 0xFFFF0000u;             // r2 has at most 8 significant bits
                    // K entry r of row n: 256-byte rows in two 128-byte halves of 16 rows each (2 KB per half)
                    const uint32_t half = ub + (r >> 6) * kUpperHalfBytes, piece = (r & 63) >> 3, within = (2 * r) & 15;
                    asm volatile("st.shared.u16 [%0], %1;" ::"r"(half + 0 * 128 + ((piece ^ 0) << 4) + within), "r"(hi >> 16) : "memory");
                    asm volatile("st.shared.u16 [%0], %1;" ::"r"(half + 1 * 128 + ((piece ^ 1) << 4) + within), "r"(mid >> 16) : "memory");
                    asm volatile("st.shared.u16 [%0], %1;" ::"r"(half + 2 * 128 + ((piece ^ 2) << 4) + within), "r"(lo >> 16) : "memory");
                }
                fence_proxy_async_smem();
                named_barrier_sync(2, kEpilogueThreads);
                if (r == 0) {
                    tc_fence_after();
                    const uint32_t d_addr = tmem_base + kTotBase + tt * kTotCols;
                    if (IS_INT) {
                        const uint32_t idesc = make_idesc(0, kTotCols);
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)
                            mma_issue<true>(d_addr, make_smem_desc(smem_u32(upper_a) + kk * 32), make_smem_desc(ub + kk * 32), idesc, kk > 0 ? 1u : 0u);
                    } else {
                        const uint32_t idesc = make_idesc(2, kTotCols);                // bf16 operands, fp32 accumulator
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk)
                            mma_issue<false>(d_addr, make_smem_desc(smem_u32(upper_a) + (kk >> 2) * kAtomBytes + (kk & 3) * 32),
                                             make_smem_desc(ub + (kk >> 2) * kUpperHalfBytes + (kk & 3) * 32), idesc, kk > 0 ? 1u : 0u);
                    }
                    mma_commit(smem_u32(&ctl->up_done));
                }
                (void)w.wait(smem_u32(&ctl->up_done), j & 1);              // (a wait that ran out is caught by the next vote)
                tc_fence_after();
                const uint32_t d0 = tmem_ld1(lane_base + kTotBase + tt * kTotCols);
                const uint32_t d1 = tmem_ld1(lane_base + kTotBase + tt * kTotCols + 1);
                const uint32_t d2 = tmem_ld1(lane_base + kTotBase + tt * kTotCols + 2);
                tmem_ld_wait();
                tc_fence_before();
                mbar_arrive(smem_u32(&ctl->tot_empty[tt]));            // the small accumulator may be refilled
                if (IS_INT) {
                    exc_all = d0 + (d1 << 7);                              // sum of the totals of rows 0 .. r-1
                    tile_total = exc_all + rowtot;
                } else {
                    const float e = (__uint_as_float(d0) + __uint_as_float(d1)) + __uint_as_float(d2);
                    exc_all = __float_as_uint(e);
                    tile_total = __float_as_uint(e + __uint_as_float(rowtot));
                }
                rowpref[ts * kTileRows + r] = exc_all;
                if (r == kTileRows - 1) {
                    const CarryT a = IS_INT ? CarryT(tile_total) : CarryT(__uint_as_float(tile_total));
                    const bool first = (t % p.tiles_per_row == 0);
                    const uint32_t status = first ? kStatusInclusive : kStatusPartial;
                    if (!prefilled && t != skip_tile)
                        st_record(records + size_t(t) * 16, (uint64_t(epoch) << 2) | status, CO::enc(first ? a + carry_in : a));
                    ctl->agg_slot[ts] = CO::enc(a);
                }
                mbar_arrive(smem_u32(&ctl->agg_ready[ts]));
                PROF_ADD(1);
                continue;
            }
            tc_fence_before();
            mbar_arrive(smem_u32(&ctl->tot_empty[tt]));                // the small accumulator may be refilled
            if (!segmented) {
                // ordinary scan: inclusive prefix sums of the row totals across the warp's 32 rows, one hop through
                // shared memory across the four warps
                uint32_t inc = rowtot;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const uint32_t up = __shfl_up_sync(0xffffffffu, inc, o);
                    if (lane >= o) inc = add32<IS_INT>(inc, up);
                }
                uint32_t exc = __shfl_up_sync(0xffffffffu, inc, 1);
                if (lane == 0) exc = 0;
                const int pb = j & 1;
                if (lane == 31) ctl->warp_tot[pb][wq] = inc;
                named_barrier_sync(2, kEpilogueThreads);
                const uint32_t w0 = ctl->warp_tot[pb][0], w1 = ctl->warp_tot[pb][1], w2 = ctl->warp_tot[pb][2], w3 = ctl->warp_tot[pb][3];
                uint32_t before = 0;                                  // rows of the earlier warps
                if (wq >= 1) before = w0;
                if (wq >= 2) before = add32<IS_INT>(before, w1);
                if (wq >= 3) before = add32<IS_INT>(before, w2);
                rowpref[ts * kTileRows + r] = (wq == 0) ? exc : add32<IS_INT>(before, exc);
                if (r == 0) {
                    const uint32_t tile_tot = add32<IS_INT>(add32<IS_INT>(w0, w1), add32<IS_INT>(w2, w3));
                    const CarryT a = IS_INT ? CarryT(tile_tot) : CarryT(__uint_as_float(tile_tot));
                    // the first tile of a scan has nothing before it: its total is already inclusive
                    const bool first = (t % p.tiles_per_row == 0);
                    const uint32_t status = first ? kStatusInclusive : kStatusPartial;
                    if (!prefilled && t != skip_tile)
                        st_record(records + size_t(t) * 16, (uint64_t(epoch) << 2) | status, CO::enc(first ? a + carry_in : a));
                    TRACE(t, 3);
                    if (j == 0) stamp(kStampPublished);
                    ctl->agg_slot[ts] = CO::enc(a);
                }
                // every thread arrives (release) after its own rowpref entry is written: the look-back warp,
                // and through it the store warps, then see all 128 entries
                mbar_arrive(smem_u32(&ctl->agg_ready[ts]));
                PROF_ADD(1);
                continue;
            }
            // Segmented scan: the scan over the 128 rows runs on pairs (value, cut): `cut` says that a segment starts
            // in the row, in which case `value` is the sum from that start on and nothing before the row carries
            // past it.
            uint32_t inc = rowtot;
            int cut = 0, cut_in = 0;
            if (seg_fl & kRowHasStart) {
                inc = seg_rv;
                cut = 1;
                cut_in = (seg_fl & kRowCutIn) ? 1 : 0;
            }
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t up = __shfl_up_sync(0xffffffffu, inc, o);
                const int upc = __shfl_up_sync(0xffffffffu, cut, o);
                if (lane >= o) {
                    if (!cut) inc = add32<IS_INT>(inc, up);
                    cut |= upc;
                }
            }
            uint32_t exc = __shfl_up_sync(0xffffffffu, inc, 1);       // what the rows above hand on, inside the warp
            int exc_cut = __shfl_up_sync(0xffffffffu, cut, 1);
            if (lane == 0) {
                exc = 0;
                exc_cut = 0;
            }
            const int pb = j & 1;
            if (lane == 31) {
                ctl->warp_tot[pb][wq] = inc;
                ctl->warp_cut[pb][wq] = uint32_t(cut);
            }
            named_barrier_sync(2, kEpilogueThreads);
            uint32_t run = 0;                                         // rows of the earlier warps / of all four warps
            int run_cut = 0;
            uint32_t before = 0;
            int before_cut = 0;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                if (k == wq) {
                    before = run;
                    before_cut = run_cut;
                }
                const uint32_t wv = ctl->warp_tot[pb][k];
                if (ctl->warp_cut[pb][k]) {
                    run = wv;
                    run_cut = 1;
                } else {
                    run = add32<IS_INT>(run, wv);
                }
            }
            uint32_t rp = exc_cut ? exc : ((wq == 0) ? exc : add32<IS_INT>(before, exc));
            int rp_cut = exc_cut | before_cut;
            if (cut_in) {                                             // a segment starts with the row: nothing carries in
                rp = 0;
                rp_cut = 1;
            }
            rowpref[ts * kTileRows + r] = rp;
            const uint32_t cut_mask = __ballot_sync(0xffffffffu, rp_cut != 0);
            if (lane == 0) ctl->seg_cut[ts][wq] = cut_mask;
            if (r == 0) {
                CarryT a = IS_INT ? CarryT(run) : CarryT(__uint_as_float(run));
                // the first tile of a scan has nothing before it, and a tile in which a segment starts hands on
                // only what follows that start: in both cases its total is final at once
                const bool first = (t % p.tiles_per_row == 0);
                const uint32_t status = (first || run_cut) ? kStatusInclusive : kStatusPartial;
                if (!prefilled && t != skip_tile)
                    st_record(records + size_t(t) * 16, (uint64_t(epoch) << 2) | status, CO::enc((first && !run_cut) ? a + carry_in : a));
                TRACE(t, 3);
                if (j == 0) stamp(kStampPublished);
                ctl->agg_slot[ts] = CO::enc(a);
                ctl->agg_cut[ts] = uint32_t(run_cut);
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
        const uint32_t slab0 = smem_u32(out_ring) + (warp - kFirstStoreWarp) * kSlabBytes;
        const int sub = lane >> 3, piece = lane & 7;                // read-back role: row sub (+4i) of the slab, 16-byte piece
        uint32_t *const out32 = reinterpret_cast<uint32_t *>(p.out);
        // The carry-product variant makes the four warps of a group meet at a barrier inside the loop, so
        // there they must also leave the loop together: the outcome of every wait is then voted on by the
        // whole group.  In the default path a warp shares no barrier with the others and votes alone.
        const bool carry_product = !IS_INT && S == 128 && use_down && !level0_only;
        const bool chunk_down = CHUNK_TC && !IS_INT && use_down && !level0_only;   // the same for s < 128 (needs the chunk product)
        const bool group_meets = carry_product || CHUNK_TC;       // (the chunk product has the same group barrier)
        auto gave_up = [&](bool ok) {
            return group_meets ? named_barrier_or(3 + group, kEpilogueThreads, !ok) : !__all_sync(0xffffffffu, ok);
        };
        PROF_DECL
        PROF_T0();
        uint32_t stored = 0;
        uint32_t j_first = group;
        if (!FULL && p.tiles_total <= gridDim.x) {
            // A launch with no more tiles than CTAs: nothing overlaps the store of a CTA's first tile (most CTAs have
            // no other), so the two store groups share it, columns 0-63 and 64-127.  The second group starts from what
            // the chunks of the first half add up to - the values at their last columns in the accumulator, added in
            // the order of the chain, so the result is bit for bit the same.  Measured: a 64 Ki-element scan takes as
            // long as before; but with this copy of the store code in front of it, the loop below comes out of the
            // compiler faster on int8 input (n = 2^28: 205.7 against 209.5 us per scan, this block not running there;
            // same registers and spills, 3.5 % fewer executed instructions; neither hoisting the slab addresses by
            // hand nor a peeled first iteration does the same), which is why the block stays.
            bool ok = w.wait(smem_u32(&ctl->carry_ready[0]), 0);
            const uint32_t t = ctl->tile_of[0];
            ok = ok && t != kNoTile && w.wait(smem_u32(&ctl->acc_full[0]), 0);
            if (__all_sync(0xffffffffu, ok)) {
                tc_fence_after();
                const uint32_t scan_row = t / p.tiles_per_row, lt = t % p.tiles_per_row;
                uint32_t base;
                {
                    const CarryT carry = CO::dec(ctl->carry_slot[0]);
                    const uint32_t rp = rowpref[r];
                    if (IS_INT) base = uint32_t(carry) + rp;
                    else base = __float_as_uint(static_cast<float>(double(carry) + double(__uint_as_float(rp))));
                }
                uint32_t run = base, prev = base;
                if (group == 1) {
                    if (S == kTileCols) {                             // one chunk per row: the scan in the accumulator runs on
                        const uint32_t left = tmem_ld1(lane_base + kTileCols / 2 - 1);
                        tmem_ld_wait();
                        prev = add32<IS_INT>(left, base);
                    } else {
                        constexpr int kHalfChunks = (kTileCols / 2) / (S < kTileCols ? S : 1);
                        uint32_t ends[kHalfChunks > 0 ? kHalfChunks : 1];
#pragma unroll
                        for (int g = 0; g < kHalfChunks; ++g) ends[g] = tmem_ld1(lane_base + (g + 1) * S - 1);
                        tmem_ld_wait();
#pragma unroll
                        for (int g = 0; g < kHalfChunks; ++g) run = add32<IS_INT>(ends[g], run);
                        prev = run;
                    }
                }
                const uint32_t q0 = 2 * group;
                const uint32_t row0 = lt * kTileRows + wq * 32;
                uint32_t *const gbase = out32 + size_t(scan_row) * p.scan_pitch + size_t(row0) * kTileCols + piece * 4;
                const int rows_here = int(p.rows128) - int(row0);
                uint32_t d[32];
                tmem_ld32(lane_base + q0 * 32, d);
#pragma unroll
                for (int qq = 0; qq < 2; ++qq) {
                    tmem_ld_wait();
                    uint32_t o[32];
#pragma unroll
                    for (int c = 0; c < 32; ++c) {
                        const uint32_t v = add32<IS_INT>(d[c], run);
                        o[c] = EXCL ? prev : v;
                        prev = v;
                        const bool chunk_end = (S <= 32) ? (((c + 1) % S) == 0) : (c == 31 && (((qq + 1) * 32) % S) == 0);
                        if (chunk_end) run = v;
                    }
                    __syncwarp();
                    const uint32_t buf = slab0 + lane * 128;
#pragma unroll
                    for (int c4 = 0; c4 < 8; ++c4)
                        st_shared_v4(buf + ((c4 ^ (lane & 7)) << 4), o[4 * c4], o[4 * c4 + 1], o[4 * c4 + 2], o[4 * c4 + 3]);
                    __syncwarp();
                    uint32_t a[32];
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int rr = 4 * i + sub;
                        ld_shared_v4(slab0 + rr * 128 + ((piece ^ (rr & 7)) << 4), a[4 * i], a[4 * i + 1], a[4 * i + 2], a[4 * i + 3]);
                    }
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int rr = 4 * i + sub;
                        if (rr < rows_here)
                            st_global_v4(gbase + size_t(rr) * kTileCols + (q0 + qq) * 32, a[4 * i], a[4 * i + 1], a[4 * i + 2], a[4 * i + 3]);
                    }
                    if (qq == 0) tmem_ld32(lane_base + (q0 + 1) * 32, d);
                }
                ++stored;
                if (group == 0) {
                    tc_fence_before();
                    mbar_arrive(smem_u32(&ctl->acc_empty[0]));
                    mbar_arrive(smem_u32(&ctl->ring_free[0]));
                    j_first = kStoreGroups;                               // tile 0 is done: go on to the marker behind it
                }
            }
        }
        for (uint32_t j = j_first;; j += kStoreGroups) {
            const uint32_t ts = j % kNumCarry, ut = j / kNumCarry;
            const uint32_t slot = j % kNumAcc, ua = j / kNumAcc;
            if (gave_up(w.wait(smem_u32(&ctl->carry_ready[ts]), ut & 1))) break;
            PROF_ADD(0);
            const uint32_t t = ctl->tile_of[j % kTileRing];
            if (t == kNoTile) break;                                  // (the same for the whole group)
            if (gave_up(w.wait(smem_u32(&ctl->acc_full[slot]), ua & 1))) break;
            PROF_ADD(1);
            PROF_INC(5, 1);
            if (lane == 0 && wq == 0) TRACE(t, 6);
            tc_fence_after();
            const uint32_t scan_row = t / p.tiles_per_row, lt = t % p.tiles_per_row;
            uint32_t base;                                            // sum of everything before this row
            {
                CarryT carry = CO::dec(ctl->carry_slot[ts]);
                // segmented scan: a segment starts before this row, inside the tile
                if (segmented && ((ctl->seg_cut[ts][wq] >> lane) & 1u)) carry = CarryT(0);
                uint32_t rp = rowpref[ts * kTileRows + r];
                if (IS_INT) base = uint32_t(carry) + rp;
                else base = __float_as_uint(static_cast<float>(double(carry) + double(__uint_as_float(rp))));
            }
            const bool level0 = level0_only;
            if (level0) base = 0;
            uint32_t run = base;                                      // sum of everything before the current chunk
            uint32_t prev = base;                                     // value of the element to the left (exclusive form)
            if (carry_product) {
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
                if (gave_up(w.wait(smem_u32(&ctl->down_done[group]), (j / kStoreGroups) & 1))) break;
                tc_fence_after();
                run = 0;                                              // the carry is inside the accumulator now
            }
            // Paper-faithful variant of the chunk level (kernel variant CHUNK_TC): the carries of the 128 / s chunks of a
            // row are the exclusive scan of the chunk totals, here a product of the totals with a strictly upper
            // triangular ones matrix.  The totals (the last column of every chunk in the accumulator) are int32 /
            // fp32, so each is split exactly into narrow terms first (two 8-bit limbs, |total| <= 2^13; three bf16
            // terms), the terms of the group's 128 rows form the data operand, one kind::i8 product (two kind::f16
            // products) scans them, and the results are recombined.  The register chain below is then not used.
            uint32_t chunk_carry[CHUNK_TC ? kTileCols / S : 1];
            if (CHUNK_TC && !level0) {
                constexpr int kChunks = kTileCols / S, kTerms = IS_INT ? 2 : 3;
                uint32_t tot[kChunks];
#pragma unroll
                for (int g = 0; g < kChunks; ++g) tot[g] = tmem_ld1(lane_base + slot * kTileCols + (g + 1) * S - 1);
                tmem_ld_wait();
                uint32_t wd[12] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};      // K entries kTerms g + l, packed
#pragma unroll
                for (int g = 0; g < kChunks; ++g) {
                    if (IS_INT) {
                        const int32_t v = int32_t(tot[g]);
                        const uint32_t lo = uint32_t(v & 127), hi = uint32_t((v >> 7) & 0xFF);
                        wd[(2 * g) >> 2] |= lo << (8 * ((2 * g) & 3));
                        wd[(2 * g + 1) >> 2] |= hi << (8 * ((2 * g + 1) & 3));
                    } else {
                        const uint32_t hi = tot[g] & 0xFFFF0000u;
                        const float r1 = __uint_as_float(tot[g]) - __uint_as_float(hi);
                        const uint32_t mid = __float_as_uint(r1) & 0xFFFF0000u;
                        const float r2 = r1 - __uint_as_float(mid);
                        const uint32_t lo = __float_as_uint(r2) & 0xFFFF0000u;
                        const uint32_t term[3] = {hi >> 16, mid >> 16, lo >> 16};
#pragma unroll
                        for (int l = 0; l < 3; ++l) wd[(3 * g + l) >> 1] |= term[l] << (16 * ((3 * g + l) & 1));
                    }
                }
                const uint32_t ca = smem_u32(chunk_a) + group * kAtomBytes;
                const uint32_t rowa = ca + r * 128;
                constexpr int kPiecesUsed = (kTerms * kChunks * (IS_INT ? 1 : 2) + 15) / 16;
#pragma unroll
                for (int c = 0; c < kPiecesUsed; ++c)
                    st_shared_v4(rowa + ((c ^ (r & 7)) << 4), wd[4 * c], wd[4 * c + 1], wd[4 * c + 2], wd[4 * c + 3]);
                fence_proxy_async_smem();
                named_barrier_sync(3 + group, kEpilogueThreads);
                const uint32_t d2 = tmem_base + kChunkScratch + group * 32;
                if (wq == 0 && lane == 0) {
                    tc_fence_after();
                    if (IS_INT) {
                        mma_issue<true>(d2, make_smem_desc(ca), make_smem_desc(smem_u32(chunk_b)), make_idesc(0, 16), 0u);
                    } else {
#pragma unroll
                        for (int kk = 0; kk < 2; ++kk)
                            mma_issue<false>(d2, make_smem_desc(ca + kk * 32), make_smem_desc(smem_u32(chunk_b) + kk * 32), make_idesc(2, 32), kk > 0 ? 1u : 0u);
                    }
                    mma_commit(smem_u32(&ctl->chunk_done[group]));
                }
                if (gave_up(w.wait(smem_u32(&ctl->chunk_done[group]), (j / kStoreGroups) & 1))) break;
                tc_fence_after();
                uint32_t res[kTerms * kChunks];
#pragma unroll
                for (int n = 0; n < kTerms * kChunks; ++n) res[n] = tmem_ld1(lane_base + kChunkScratch + group * 32 + n);
                tmem_ld_wait();
#pragma unroll
                for (int g = 0; g < kChunks; ++g) {
                    if (IS_INT) chunk_carry[g] = res[2 * g] + (res[2 * g + 1] << 7);
                    else chunk_carry[g] = __float_as_uint((__uint_as_float(res[3 * g]) + __uint_as_float(res[3 * g + 1])) + __uint_as_float(res[3 * g + 2]));
                }
                if (chunk_down) {
                    // Paper-faithful down-sweep for s < 128: what precedes each chunk (row base + carry of the chunk)
                    // is split exactly into three bf16 terms, the terms of the group's 128 rows replace the chunk
                    // totals in the data operand (its product has completed), and one product with the 0 / 1 selector
                    // adds every chunk's carry to all elements of that chunk inside the accumulator.
                    uint32_t cw[12] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
#pragma unroll
                    for (int g = 0; g < kChunks; ++g) {
                        const float v = __uint_as_float(base) + __uint_as_float(chunk_carry[g]);
                        const uint32_t hi = __float_as_uint(v) & 0xFFFF0000u;
                        const float r1 = v - __uint_as_float(hi);
                        const uint32_t mid = __float_as_uint(r1) & 0xFFFF0000u;
                        const float r2 = r1 - __uint_as_float(mid);
                        const uint32_t lo = __float_as_uint(r2) & 0xFFFF0000u;
                        const uint32_t term[3] = {hi >> 16, mid >> 16, lo >> 16};
#pragma unroll
                        for (int l = 0; l < 3; ++l) cw[(3 * g + l) >> 1] |= term[l] << (16 * ((3 * g + l) & 1));
                        chunk_carry[g] = 0u;                                 // it is inside the accumulator from here on
                    }
#pragma unroll
                    for (int c = 0; c < kPiecesUsed; ++c)
                        st_shared_v4(rowa + ((c ^ (r & 7)) << 4), cw[4 * c], cw[4 * c + 1], cw[4 * c + 2], cw[4 * c + 3]);
                    fence_proxy_async_smem();
                    named_barrier_sync(3 + group, kEpilogueThreads);
                    if (wq == 0 && lane == 0) {
                        tc_fence_after();
                        constexpr int kSelSteps = (3 * kChunks + 15) / 16;
#pragma unroll
                        for (int kk = 0; kk < kSelSteps; ++kk)
                            mma_issue<false>(tmem_base + slot * kTileCols, make_smem_desc(ca + kk * 32),
                                             make_smem_desc(smem_u32(chunk_sel) + kk * 32), make_idesc(2, kTileCols), 1u);
                        mma_commit(smem_u32(&ctl->down_done[group]));
                    }
                    if (gave_up(w.wait(smem_u32(&ctl->down_done[group]), (j / kStoreGroups) & 1))) break;
                    tc_fence_after();
                    run = 0;
                    base = 0;                                                // (prev keeps the row base: the exclusive value of the row's first element)
                }
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
                    if (CHUNK_TC && !level0 && ((q * 32 + c) % S) == 0)   // start of a chunk: its carry comes from the product
                        run = add32<IS_INT>(base, chunk_carry[(q * 32 + c) / S]);
                    uint32_t v = add32<IS_INT>(d[c], run);
                    o[c] = EXCL ? prev : v;
                    prev = v;
                    const bool chunk_end = (S <= 32) ? (((c + 1) % S) == 0) : (c == 31 && (((q + 1) * 32) % S) == 0);
                    if (!CHUNK_TC && chunk_end && !level0) run = v;   // end of a chunk: its total joins the carry
                }
                if (level0 && EXCL) {                                 // not a meaningful combination; keep it defined
#pragma unroll
                    for (int c = 0; c < 32; ++c) o[c] = d[c];
                }
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
                PROF_ADD(4);
                if (q < 3) tmem_ld32(lane_base + slot * kTileCols + (q + 1) * 32, d);
            }
            if (lane == 0 && wq == 0) {
                TRACE(t, 7);
                if (j == 0) stamp(kStampStored);
            }
            ++stored;
            tc_fence_before();
            mbar_arrive(smem_u32(&ctl->acc_empty[slot]));
            // the carry ring entry of this tile (row prefixes, carry, barriers) may be reused
            mbar_arrive(smem_u32(&ctl->ring_free[ts]));
        }
        if (lane == 0 && wq == 0) PROF_FLUSH(32 + 8 * group, 6);
        if (lane == 0 && wq == 0 && use_stamps) p.stamps[size_t(blockIdx.x) * kStampsPerCta + kStampTiles + group] = stored;
    }

    // ---- tear-down
    if (threadIdx.x == 0) stamp(kStampLoopsDone);
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0) stamp(kStampAllDone);
    tc_fence_after();
    if (warp == 1) tmem_dealloc(tmem_base, 512);
    if (threadIdx.x == 0) stamp(kStampExit);
}

// Tail of a single-array scan: the n % 128 elements after the last full 128-element row.
// Runs after the main kernel on the same stream; the carry is the inclusive record of the
// last tile (or nothing when there is no full row).
template <bool IS_INT, bool EXCL>
__global__ void tcu_scan_tail_kernel(const void *in, void *out, size_t start0, size_t pitch, uint32_t count, const void *ws,
                                     uint32_t tiles_per_row, uint32_t dtype, const void *carry_in, void *carry_out) {
    // one block per scan (blockIdx.x = row of a batched scan)
    const size_t start = start0 + size_t(blockIdx.x) * pitch;
    const uint32_t tiles = (blockIdx.x + 1) * tiles_per_row;      // index + 1 of this scan's last tile record
    using CO = CarryOps<IS_INT>;
    using CarryT = typename CO::T;
    __shared__ CarryT warp_tot[4];
    const int tid = threadIdx.x, lane = tid & 31, wq = tid >> 5;
    CarryT carry = CarryT(0);
    if (carry_in && tiles_per_row == 0) {       // no full row before the tail: the continuation value is all there is
        carry = CO::dec(*reinterpret_cast<const uint64_t *>(carry_in));
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
        // the total of the whole array, for a caller that continues the scan elsewhere (single arrays only)
        if (carry_out != nullptr && tid == int(count) - 1) *reinterpret_cast<uint64_t *>(carry_out) = CO::enc(before + inc);
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

// ---- two-sweep variant with the scan of the tile totals done by the tensor-core scan itself (Section 2.2 step 3: the
// totals of the segments are scanned with Algorithm 1 again).  Tile totals are 32-bit integers or doubles, not
// tensor-core input types, so each is first split exactly into narrow terms, every term forms an array of its own that
// goes through the ordinary scan of this library, and the scanned terms are recombined:
//   integer: four signed base-256 digits d0..d3 with d0 + 256 d1 + 65536 d2 + 16777216 d3 = total (mod 2^32); the scans
//            are exact mod 2^32, so is the recombination sum_b (scan_b << 8 b);
//   float:   the total rounded to fp32 and cut into three bf16 terms hi + mid + lo (8 significant bits each, exact);
//            the three fp32 scans are added in fp64.
constexpr int kSplitTermsInt = 4, kSplitTermsFloat = 3;
template <bool IS_INT>
__global__ void __launch_bounds__(256) tcu_totals_split_kernel(const void *ws, uint32_t tiles, uint8_t *planes, uint32_t plane_stride) {
    const uint32_t t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= tiles) return;
    const uint64_t *rec = reinterpret_cast<const uint64_t *>(reinterpret_cast<const uint8_t *>(ws) + kHeaderBytes);
    const uint64_t bits = rec[2 * size_t(t) + 1];
    if (IS_INT) {
        uint32_t v = uint32_t(bits);
#pragma unroll
        for (int b = 0; b < kSplitTermsInt; ++b) {
            const int32_t d = int32_t(int8_t(v & 0xFFu));             // digit in [-128, 127]
            reinterpret_cast<int8_t *>(planes + size_t(b) * plane_stride)[t] = int8_t(d);
            v = (v - uint32_t(d)) >> 8;                                // exact: the low byte is zero now
        }
    } else {
        const float f = float(__longlong_as_double((long long)bits));
        const uint32_t hi = __float_as_uint(f) & 0xFFFF0000u;
        const float r1 = f - __uint_as_float(hi);
        const uint32_t mid = __float_as_uint(r1) & 0xFFFF0000u;
        const float r2 = r1 - __uint_as_float(mid);
        const uint32_t lo = __float_as_uint(r2) & 0xFFFF0000u;          // r2 has at most 8 significant bits
        reinterpret_cast<uint16_t *>(planes + 0 * size_t(plane_stride))[t] = uint16_t(hi >> 16);
        reinterpret_cast<uint16_t *>(planes + 1 * size_t(plane_stride))[t] = uint16_t(mid >> 16);
        reinterpret_cast<uint16_t *>(planes + 2 * size_t(plane_stride))[t] = uint16_t(lo >> 16);
    }
}

// Recombines the scanned terms into the records sweep 2 looks back over: {INCLUSIVE, sum of the totals of tiles 0..t}.
template <bool IS_INT>
__global__ void __launch_bounds__(256) tcu_totals_combine_kernel(void *ws, uint32_t tiles, const uint8_t *sums, uint32_t sum_stride) {
    using CO = CarryOps<IS_INT>;
    using CarryT = typename CO::T;
    const uint32_t t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= tiles) return;
    const WsHeader *hdr = reinterpret_cast<const WsHeader *>(ws);
    uint64_t *rec = reinterpret_cast<uint64_t *>(reinterpret_cast<uint8_t *>(ws) + kHeaderBytes);
    const uint64_t flag = (uint64_t(hdr->epoch + 1) << 2) | kStatusInclusive;   // the epoch the main kernel will use
    CarryT prefix = CarryT(0);
    if (IS_INT) {
        uint32_t acc = 0;
#pragma unroll
        for (int b = 0; b < kSplitTermsInt; ++b) acc += reinterpret_cast<const uint32_t *>(sums + size_t(b) * sum_stride)[t] << (8 * b);
        prefix = CarryT(acc);
    } else {
        double acc = 0.0;
#pragma unroll
        for (int b = 0; b < kSplitTermsFloat; ++b) acc += double(reinterpret_cast<const float *>(sums + size_t(b) * sum_stride)[t]);
        prefix = CarryT(acc);
    }
    rec[2 * size_t(t) + 1] = CO::enc(prefix);
    rec[2 * size_t(t)] = flag;
}

// ---- segmented scan (Section 2.2 with caller-given segments): the rows that hold a segment start ---------------
// The array is cut into rows of 128 elements, counted from its start.  A row in which no segment starts belongs to
// one segment and goes through the tensor-core path unchanged.  A row that holds starts is summarised for that path
// by two values: whether a segment starts at its first element (then nothing carries into the row) and the sum from
// its last start to its end (what the row hands on).  The elements of such a row from its first start on - the
// ones the carry of the earlier rows must not reach - are scanned again here, by eight lanes, straight from the input.

struct SegSource {
    const uint64_t *offsets;   // num_segments + 1 values, or NULL for equal segments of `pitch` elements
    uint64_t pitch;
    uint64_t num_segments;
    __device__ __forceinline__ uint64_t start(uint64_t k) const { return offsets ? offsets[k] : k * pitch; }
};

enum SegMode { kSegPrepare = 0, kSegFixup = 1, kSegTail = 2 };

// kSegLanes lanes per segment start (modes prepare / fixup; the lanes of the first start in a row do the row; a warp
// works on 32 / kSegLanes starts at once, which is what hides the latency of the offset -> row -> store chain of each)
// or one such group in all (mode tail: the incomplete row at the end of the array, which the tile kernel never
// stores).  Every lane holds kSegPerLane consecutive elements of the row.
constexpr int kSegLanes = 8;
constexpr int kSegPerLane = kTileCols / kSegLanes;          // 16
template <bool IS_INT, bool EXCL, int MODE>
__global__ void __launch_bounds__(256) tcu_segment_rows_kernel(const void *in, void *out, uint64_t n, SegSource seg, const void *ws,
                                                               uint32_t tiles, uint8_t *rowflag, uint32_t *rowval, uint32_t dtype) {
    using CO = CarryOps<IS_INT>;
    using CarryT = typename CO::T;
    using ValT = typename std::conditional<IS_INT, uint32_t, float>::type;
    constexpr unsigned kFull = 0xffffffffu;
    const int sl = threadIdx.x & (kSegLanes - 1);          // lane within the group of this start
    const uint64_t rows128 = n / kTileCols;
    uint64_t row = 0, k0 = 0;              // the row this group handles, and the first segment start inside it
    // A group with nothing to do stays in the code (the shuffles below are warp-wide) but touches no memory.
    bool active = true, has_start = true;
    if (MODE == kSegTail) {
        active = threadIdx.x < kSegLanes;
        row = rows128;
        // first start at or after the beginning of the row (binary search; the offsets never decrease)
        uint64_t lo = 0, hi = active ? seg.num_segments : 0;
        while (lo < hi) {
            const uint64_t mid = (lo + hi) >> 1;
            if (seg.start(mid) < row * kTileCols) lo = mid + 1;
            else hi = mid;
        }
        k0 = lo;
        has_start = active && k0 < seg.num_segments && seg.start(k0) < n;
    } else {
        k0 = (uint64_t(blockIdx.x) * blockDim.x + threadIdx.x) / kSegLanes;
        active = k0 < seg.num_segments;
        if (active) {
            const uint64_t p = seg.start(k0);
            row = p / kTileCols;
            if (p >= n) active = false;                                          // empty segments at the very end
            else if (k0 > 0 && seg.start(k0 - 1) / kTileCols == row) active = false;   // an earlier start of the row does it
            else if (row >= rows128) active = false;                             // the incomplete last row: mode tail
        }
        has_start = active;
    }
    const uint64_t base = row * kTileCols;
    const uint32_t count = !active ? 0u : uint32_t(n - base < kTileCols ? n - base : kTileCols);
    // this lane's elements and their start marks
    uint32_t mark = 0;                     // bit i: a segment starts at column kSegPerLane * sl + i
    uint32_t first_col = kTileCols, first_inner_col = kTileCols;    // first start of the row; first one that is not at column 0
    if (has_start) {
        for (uint64_t k = k0; k < seg.num_segments; ++k) {
            const uint64_t p = seg.start(k);
            if (p >= base + count) break;
            const uint32_t c = uint32_t(p - base);
            if (c / kSegPerLane == uint32_t(sl)) mark |= 1u << (c % kSegPerLane);
            if (first_col == kTileCols) first_col = c;
            if (c > 0 && first_inner_col == kTileCols) first_inner_col = c;
        }
    }
    ValT x[kSegPerLane];
#pragma unroll
    for (int i = 0; i < kSegPerLane; ++i) x[i] = ValT(0);
    if (count == kTileCols) {              // a whole row: aligned 16-byte loads
        if (IS_INT) {
            const uint4 w = reinterpret_cast<const uint4 *>(reinterpret_cast<const int8_t *>(in) + base)[sl];
            const uint32_t wd[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
            for (int i = 0; i < kSegPerLane; ++i) x[i] = ValT(int32_t(int8_t((wd[i >> 2] >> (8 * (i & 3))) & 0xFF)));
        } else {
            const uint4 *src = reinterpret_cast<const uint4 *>(reinterpret_cast<const uint16_t *>(in) + base) + 2 * sl;
            const uint4 wa = src[0], wb = src[1];
            const uint32_t wd[8] = {wa.x, wa.y, wa.z, wa.w, wb.x, wb.y, wb.z, wb.w};
#pragma unroll
            for (int i = 0; i < kSegPerLane; ++i) {
                const uint32_t h = (wd[i >> 1] >> (16 * (i & 1))) & 0xFFFFu;
                x[i] = ValT((dtype == 2) ? __uint_as_float(h << 16) : __half2float(__ushort_as_half(uint16_t(h))));
            }
        }
    } else if (count > 0) {
#pragma unroll
        for (int i = 0; i < kSegPerLane; ++i) {
            const uint32_t c = kSegPerLane * sl + i;
            if (c < count) {
                if (IS_INT) {
                    x[i] = ValT(int32_t(reinterpret_cast<const int8_t *>(in)[base + c]));
                } else {
                    const uint16_t b = reinterpret_cast<const uint16_t *>(in)[base + c];
                    x[i] = ValT((dtype == 2) ? __uint_as_float(uint32_t(b) << 16) : __half2float(__ushort_as_half(b)));
                }
            }
        }
    }
    // scan with restarts: inside the lane, then across the lanes of the group on (restarted?, value) pairs
    ValT inc[kSegPerLane];
    ValT run = ValT(0);
    bool cut = false;
#pragma unroll
    for (int i = 0; i < kSegPerLane; ++i) {
        if (mark & (1u << i)) {
            run = ValT(0);
            cut = true;
        }
        run += x[i];
        inc[i] = run;
    }
    ValT lane_val = run;
    bool lane_cut = cut;
#pragma unroll
    for (int o = 1; o < kSegLanes; o <<= 1) {
        const ValT v = __shfl_up_sync(kFull, lane_val, o, kSegLanes);
        const int f = __shfl_up_sync(kFull, int(lane_cut), o, kSegLanes);
        if (sl >= o) {
            if (!lane_cut) lane_val += v;
            lane_cut = lane_cut || (f != 0);
        }
    }
    ValT before = __shfl_up_sync(kFull, lane_val, 1, kSegLanes);              // what the lanes to the left hand on
    int before_cut = __shfl_up_sync(kFull, int(lane_cut), 1, kSegLanes);
    if (sl == 0) {
        before = ValT(0);
        before_cut = 0;
    }
    if (!active) return;                   // (no warp-wide operation below this line)
    if (MODE == kSegPrepare) {
        if (sl == kSegLanes - 1) {
            rowflag[row] = uint8_t(kRowHasStart | (first_col == 0 ? kRowCutIn : 0));
            rowval[row] = IS_INT ? uint32_t(lane_val) : __float_as_uint(float(lane_val));
        }
        return;
    }
    // what precedes the row in its segment (mode tail only; in mode fixup the elements before the first start
    // were written by the tile kernel and are left alone)
    CarryT carry = CarryT(0);
    if (MODE == kSegTail && tiles > 0 && first_col != 0) {
        uint64_t flag, val;
        ld_record(reinterpret_cast<const uint8_t *>(ws) + kHeaderBytes + size_t(tiles - 1) * 16, flag, val);
        carry = CO::dec(val);
    }
    const uint32_t from = (MODE == kSegTail) ? 0u : first_inner_col;
    bool open = !before_cut;               // still in the segment that entered the row (the carry applies)
    ValT left = before;                    // inclusive value of the element to the left, within its segment
    uint32_t res[kSegPerLane];
#pragma unroll
    for (int i = 0; i < kSegPerLane; ++i) {
        if (mark & (1u << i)) {
            open = false;
            left = ValT(0);
        }
        const bool restarted_in_lane = (mark & ((2u << i) - 1)) != 0;
        const ValT incl = restarted_in_lane ? inc[i] : ValT(before + inc[i]);
        const ValT mine = EXCL ? left : incl;
        uint32_t bits;
        if (IS_INT) bits = uint32_t(mine) + (open ? uint32_t(carry) : 0u);
        else bits = __float_as_uint(open ? float(double(carry) + double(mine)) : float(mine));
        res[i] = bits;
        left = incl;
    }
    // write: 16-byte stores for every four elements that are all to be written, else element by element
    uint32_t *const o32 = reinterpret_cast<uint32_t *>(out) + base + kSegPerLane * sl;
#pragma unroll
    for (int q = 0; q < kSegPerLane / 4; ++q) {
        const uint32_t c0 = kSegPerLane * sl + 4 * q;
        if ((MODE == kSegTail || c0 >= from) && c0 + 3 < count) {
            *reinterpret_cast<uint4 *>(o32 + 4 * q) = make_uint4(res[4 * q], res[4 * q + 1], res[4 * q + 2], res[4 * q + 3]);
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i)
                if ((MODE == kSegTail || c0 + i >= from) && c0 + i < count) o32[4 * q + i] = res[4 * q + i];
        }
    }
}

// ---- measuring aid: a plain widening copy with the scan's traffic mix (1 or 2 bytes read, 4 bytes written per
// element), to see what that mix reaches on this memory system without any scan in the way.  Every thread reads
// kWidenPerThread pieces of four elements and writes each as one 16-byte store, so that a warp reads whole 128-byte
// (or 256-byte) runs and writes whole 512-byte runs; one piece of the array per block, no loop over the grid (the
// fastest of the block sizes and unroll factors tried: persistent grids and one piece per thread were 10-30 % slower).
constexpr int kWidenThreads = 256;
constexpr int kWidenPerThread = 2;
template <int DTYPE>
__global__ void __launch_bounds__(kWidenThreads) tcu_widen_copy_kernel(const void *__restrict__ in, void *__restrict__ out, uint64_t pieces) {
    const uint64_t base = uint64_t(blockIdx.x) * (kWidenThreads * kWidenPerThread) + threadIdx.x;
    if (DTYPE == 0) {
        uint32_t w[kWidenPerThread];
#pragma unroll
        for (int k = 0; k < kWidenPerThread; ++k) {
            const uint64_t i = base + k * kWidenThreads;
            w[k] = i < pieces ? reinterpret_cast<const uint32_t *>(in)[i] : 0u;
        }
#pragma unroll
        for (int k = 0; k < kWidenPerThread; ++k) {
            const uint64_t i = base + k * kWidenThreads;
            int4 o;
            o.x = int(int8_t(w[k] & 0xFF));
            o.y = int(int8_t((w[k] >> 8) & 0xFF));
            o.z = int(int8_t((w[k] >> 16) & 0xFF));
            o.w = int(int8_t(w[k] >> 24));
            if (i < pieces) reinterpret_cast<int4 *>(out)[i] = o;
        }
    } else {
        uint2 w[kWidenPerThread];
#pragma unroll
        for (int k = 0; k < kWidenPerThread; ++k) {
            const uint64_t i = base + k * kWidenThreads;
            w[k] = i < pieces ? reinterpret_cast<const uint2 *>(in)[i] : make_uint2(0u, 0u);
        }
#pragma unroll
        for (int k = 0; k < kWidenPerThread; ++k) {
            const uint64_t i = base + k * kWidenThreads;
            float4 o;
            if (DTYPE == 1) {
                const float2 a = __half22float2(*reinterpret_cast<const __half2 *>(&w[k].x));
                const float2 b = __half22float2(*reinterpret_cast<const __half2 *>(&w[k].y));
                o = make_float4(a.x, a.y, b.x, b.y);
            } else {                                  // bf16: the upper half of the fp32 pattern
                o = make_float4(__uint_as_float(w[k].x << 16), __uint_as_float(w[k].x & 0xFFFF0000u),
                                __uint_as_float(w[k].y << 16), __uint_as_float(w[k].y & 0xFFFF0000u));
            }
            if (i < pieces) reinterpret_cast<float4 *>(out)[i] = o;
        }
    }
}

// ---- helpers for a scan whose array is split over several devices (Section 2.2 steps 2-3 with one segment per
// device): the total of a shard, and the exclusive prefix of the shards' totals.  Carries travel as 8-byte values
// in the format of the tile records (a double, or a zero-extended uint32 for integer scans).
template <bool IS_INT>
__global__ void __launch_bounds__(1024) tcu_sum_totals_kernel(const void *ws, uint32_t tiles, const void *in, uint64_t tail_start,
                                                              uint32_t tail_count, uint32_t dtype, void *total_out) {
    using CO = CarryOps<IS_INT>;
    using CarryT = typename CO::T;
    __shared__ CarryT warp_part[32];
    const uint64_t *rec = reinterpret_cast<const uint64_t *>(reinterpret_cast<const uint8_t *>(ws) + kHeaderBytes);
    CarryT acc = CarryT(0);
    for (uint32_t i = threadIdx.x; i < tiles; i += blockDim.x) acc += CO::dec(rec[2 * size_t(i) + 1]);
    if (threadIdx.x < tail_count) {           // the few elements after the last whole 16-byte piece
        if (IS_INT) {
            acc += CarryT(int32_t(reinterpret_cast<const int8_t *>(in)[tail_start + threadIdx.x]));
        } else {
            const uint16_t b = reinterpret_cast<const uint16_t *>(in)[tail_start + threadIdx.x];
            acc += CarryT((dtype == 2) ? __uint_as_float(uint32_t(b) << 16) : __half2float(__ushort_as_half(b)));
        }
    }
    acc = warp_sum(acc);
    if ((threadIdx.x & 31) == 0) warp_part[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        CarryT tot = CarryT(0);
        for (int k = 0; k < int(blockDim.x >> 5); ++k) tot += warp_part[k];
        *reinterpret_cast<uint64_t *>(total_out) = CO::enc(tot);
    }
}

template <bool IS_INT>
__global__ void tcu_carry_prefix_kernel(const uint64_t *totals, uint32_t index, uint64_t *carry_out) {
    using CO = CarryOps<IS_INT>;
    using CarryT = typename CO::T;
    CarryT acc = CarryT(0);
    for (uint32_t i = threadIdx.x; i < index; i += 32) acc += CO::dec(totals[i]);
    acc = warp_sum(acc);
    if (threadIdx.x == 0) *carry_out = CO::enc(acc);
}

}  // namespace tcu
