// Host side of the C ABI declared in include/tcu_scan.h: argument checks, workspace
// sizing, TMA tensor-map encoding, variant dispatch, launch and bookkeeping.
#include "tcu_scan.h"

#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cstring>
#include <mutex>

#include "tcu_scan_kernel.cuh"
#include "tcu_split.cuh"

namespace {

using namespace tcu;

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static std::once_flag once;
    static EncodeTiledFn fn = nullptr;
    std::call_once(once, [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}

// bookkeeping of the calling thread's most recent scan (nothing else outlives a call)
thread_local tcu_scan_stats_t t_stats;
thread_local bool t_have_stats = false;

int elem_bytes(tcu_dtype_t dt) { return dt == TCU_I8_I32 ? 1 : 2; }
bool valid_dtype(int dt) { return dt == TCU_I8_I32 || dt == TCU_F16_F32 || dt == TCU_BF16_F32; }
bool valid_s(int s) { return s == 16 || s == 64 || s == 128; }

constexpr uint64_t kMaxScanElements = 1ull << 37;       // elements of one scan (one row): 2^30 rows of 128

uint64_t tiles_for(uint64_t rows, uint64_t cols) {
    uint64_t rows128 = cols / kTileCols;                       // full 128-element rows of one scan
    uint64_t per = (rows128 + kTileRows - 1) / kTileRows;      // tiles of one scan
    return rows * per;
}

uint32_t floor_log(uint64_t n, uint64_t s) {
    uint32_t k = 0;
    uint64_t p = s;
    while (p <= n) {
        ++k;
        if (p > n / s) break;
        p *= s;
    }
    return k;
}

struct Shape {
    uint64_t rows, cols;
};

template <bool IS_INT, int S, bool EXCL, int VARIANT>
cudaError_t launch_main(const ScanParams &prm, dim3 grid, size_t smem, cudaStream_t stream) {
    static std::atomic<int> configured{-1};
    int dev = 0;
    cudaGetDevice(&dev);
    if (configured.load() != dev) {
        cudaError_t e = cudaFuncSetAttribute(tcu_scan_kernel<IS_INT, S, EXCL, VARIANT>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, 232448);
        if (e != cudaSuccess) return e;
        configured.store(dev);
    }
    // programmatic dependent launch: this kernel's set-up (barriers, TMEM, constant operands) may overlap the
    // tail of whatever runs before it in the stream; it waits (griddepcontrol.wait) before touching global memory
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, tcu_scan_kernel<IS_INT, S, EXCL, VARIANT>, prm);
}

// variant: kLean for the plain scan, kFull when any run-time option is in use, kChunk for the chunk-level product
template <bool IS_INT, int S, bool EXCL>
cudaError_t dispatch_variant(int variant, const ScanParams &prm, dim3 grid, size_t smem, cudaStream_t stream) {
    if constexpr (S < kTileCols) {
        if (variant == kChunk) return launch_main<IS_INT, S, EXCL, kChunk>(prm, grid, smem, stream);
    }
    if (variant != kLean) return launch_main<IS_INT, S, EXCL, kFull>(prm, grid, smem, stream);   // (s = 128: a row is one chunk)
    return launch_main<IS_INT, S, EXCL, kLean>(prm, grid, smem, stream);
}

template <bool IS_INT, bool EXCL>
cudaError_t dispatch_s(int s, int variant, const ScanParams &prm, dim3 grid, size_t smem, cudaStream_t stream) {
    switch (s) {
        case 16: return dispatch_variant<IS_INT, 16, EXCL>(variant, prm, grid, smem, stream);
        case 64: return dispatch_variant<IS_INT, 64, EXCL>(variant, prm, grid, smem, stream);
        default: return dispatch_variant<IS_INT, 128, EXCL>(variant, prm, grid, smem, stream);
    }
}

int sm_count() {
    static std::atomic<int> cached{0};
    int v = cached.load();
    if (v > 0) return v;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    cached.store(v);
    return v;
}

bool overlaps(const void *a, size_t an, const void *b, size_t bn) {
    auto pa = reinterpret_cast<uintptr_t>(a), pb = reinterpret_cast<uintptr_t>(b);
    return pa < pb + bn && pb < pa + an;
}

// Everything one scan launch needs to know.
struct Call {
    const void *d_in = nullptr;
    void *d_out = nullptr;
    size_t rows = 1, cols = 0;
    tcu_dtype_t dt = TCU_I8_I32;
    int s = 16;
    bool exclusive = false, level0 = false, two_sweep = false;
    bool nested = false;                 // an inner scan over the narrow terms of the tile totals (two-sweep variant)
    int upper_path = 0, down_path = 0, max_ctas = 0;
    const void *d_carry_in = nullptr;
    void *d_carry_out = nullptr;
    unsigned long long *d_stamps = nullptr;
    long long spin_limit = kSpinLimitCycles;
    uint32_t skip_tile = kNoTile;
    void *d_ws = nullptr;
    size_t ws_bytes = 0;
    cudaStream_t stream = nullptr;
    tcu_scan_stats_t *stats_out = nullptr;
    // segmented scan (rows == 1): segment starts inside the array, either listed on the device or every seg_pitch elements
    bool segmented = false;
    const uint64_t *d_offsets = nullptr;
    uint64_t seg_pitch = 0, num_segments = 0;
};

size_t round_up(size_t v, size_t to) { return (v + to - 1) / to * to; }
size_t record_bytes(uint64_t tiles) { return size_t(kHeaderBytes) + 16 * size_t(tiles) + 16; }
// workspace of a segmented scan of n elements: tile records, then one flag byte and one 4-byte value per row of 128
size_t seg_flag_offset(uint64_t n) { return round_up(record_bytes(tiles_for(1, n)), 256); }
// (both arrays are sized for whole tiles, plus the incomplete last row: the tile kernel copies them a tile at a time)
size_t seg_rows(uint64_t n) { return size_t(tiles_for(1, n)) * kTileRows + 1; }
size_t seg_val_offset(uint64_t n) { return seg_flag_offset(n) + round_up(seg_rows(n), 256); }
size_t seg_workspace_bytes(uint64_t n) { return seg_val_offset(n) + round_up(4 * seg_rows(n), 256); }
// Two-sweep variant with the scan of the tile totals done by this library's own scan (one array per narrow term of
// the totals): behind the records lie the term arrays (at most 4 planes of T one- or two-byte terms), their scans
// (4 planes of T four-byte sums) and the workspace of those inner scans.
size_t nested_offset(uint64_t tiles) { return round_up(record_bytes(tiles), 256); }
size_t nested_in_stride(uint64_t tiles) { return round_up(2 * size_t(tiles), 256); }
size_t nested_out_stride(uint64_t tiles) { return round_up(4 * size_t(tiles), 256); }
size_t nested_ws_bytes(uint64_t tiles) { return round_up(record_bytes(tiles_for(1, tiles)), 256); }
size_t nested_bytes(uint64_t tiles) { return 4 * nested_in_stride(tiles) + 4 * nested_out_stride(tiles) + nested_ws_bytes(tiles); }
bool totals_by_scan(const Call &c);
size_t needed_workspace(const Call &c) {
    if (c.segmented) return seg_workspace_bytes(uint64_t(c.rows) * c.cols);
    const uint64_t tiles = tiles_for(c.rows, c.cols);
    return totals_by_scan(c) ? nested_offset(tiles) + nested_bytes(tiles) : record_bytes(tiles);
}

// Host-side checks of a call; nothing has been queued on the stream when this returns an error.
tcu_status_t check_call(const Call &c) {
    if (!valid_dtype(c.dt) || !valid_s(c.s)) return (c.s > 0 && valid_dtype(c.dt)) ? TCU_ERR_UNSUPPORTED : TCU_ERR_INVALID_ARG;
    if (c.rows == 0 || c.cols == 0) return TCU_OK;
    if (!c.d_in || !c.d_out) return TCU_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(c.d_in) & 15) || (reinterpret_cast<uintptr_t>(c.d_out) & 15)) return TCU_ERR_INVALID_ARG;
    const int eb = elem_bytes(c.dt);
    // dense rows: the row pitch must keep every row 16-byte aligned on both sides (TMA boxes, vector stores)
    if (c.rows > 1 && ((c.cols * eb) % 16 != 0 || (c.cols * 4) % 16 != 0)) return TCU_ERR_UNSUPPORTED;
    if (c.level0 && (c.cols % kTileCols) != 0) return TCU_ERR_UNSUPPORTED;
    // (a scan is addressed by TMA as rows of 128 elements with a 32-bit signed row coordinate)
    if (c.rows > (1ull << 31) || c.cols > kMaxScanElements) return TCU_ERR_UNSUPPORTED;
    if (c.rows > 1 && (c.d_carry_in || c.d_carry_out)) return TCU_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(c.d_carry_in) & 7) || (reinterpret_cast<uintptr_t>(c.d_carry_out) & 7)) return TCU_ERR_INVALID_ARG;
    if (c.two_sweep && (c.rows > 1 || c.d_carry_in || c.d_carry_out)) return TCU_ERR_UNSUPPORTED;
    const uint64_t total = uint64_t(c.rows) * c.cols;
    if (overlaps(c.d_in, total * eb, c.d_out, total * 4)) return TCU_ERR_INVALID_ARG;
    if (!c.d_ws) return TCU_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(c.d_ws) & 255) return TCU_ERR_INVALID_ARG;
    if (c.ws_bytes < needed_workspace(c)) return TCU_ERR_WORKSPACE;
    if (c.segmented) {
        if (c.rows != 1 || c.level0 || c.two_sweep || c.d_carry_in || c.d_carry_out) return TCU_ERR_UNSUPPORTED;
        if (c.num_segments == 0 || c.num_segments > (1ull << 34)) return TCU_ERR_INVALID_ARG;
        if (!c.d_offsets && c.seg_pitch == 0) return TCU_ERR_INVALID_ARG;
        if (reinterpret_cast<uintptr_t>(c.d_offsets) & 7) return TCU_ERR_INVALID_ARG;
    }
    const uint64_t tiles = tiles_for(c.rows, c.cols);
    if (tiles >= (1ull << 31)) return TCU_ERR_UNSUPPORTED;
    if (c.max_ctas < 0 || c.upper_path < 0 || c.upper_path > 2 || c.down_path < 0 || c.down_path > 1) return TCU_ERR_INVALID_ARG;
    return TCU_OK;
}

bool totals_by_scan(const Call &c) { return c.two_sweep && c.upper_path >= 1 && !c.nested; }

tcu_status_t scan_impl(const Call &c);
Call make_call(const void *d_in, void *d_out, size_t rows, size_t cols, tcu_dtype_t dt, int s, bool exclusive, void *d_ws,
               size_t ws_bytes, cudaStream_t stream);

// Sweep 1.5 of the two-sweep variant when the upper levels are asked for as products: the tile totals (already in the
// records) are split into narrow terms, every term array is scanned by an ordinary call of this library, and the
// scanned terms are recombined into the inclusive records that sweep 2 expects.
tcu_status_t scan_totals_by_scan(const Call &c, uint64_t tiles, uint64_t *inner_mma) {
    uint8_t *base = reinterpret_cast<uint8_t *>(c.d_ws) + nested_offset(tiles);
    const bool is_int = c.dt == TCU_I8_I32;
    const int terms = is_int ? kSplitTermsInt : kSplitTermsFloat;
    const size_t in_stride = nested_in_stride(tiles), out_stride = nested_out_stride(tiles);
    uint8_t *planes = base, *sums = base + 4 * in_stride, *inner_ws = sums + 4 * out_stride;
    const unsigned blocks = unsigned((tiles + 255) / 256);
    // The inner scans' header and records lie where an earlier, larger scan on the same workspace may have kept its
    // records: they are cleared before use.
    if (cudaMemsetAsync(inner_ws, 0, nested_ws_bytes(tiles), c.stream) != cudaSuccess) return TCU_ERR_CUDA;
    if (is_int) tcu_totals_split_kernel<true><<<blocks, 256, 0, c.stream>>>(c.d_ws, uint32_t(tiles), planes, uint32_t(in_stride));
    else tcu_totals_split_kernel<false><<<blocks, 256, 0, c.stream>>>(c.d_ws, uint32_t(tiles), planes, uint32_t(in_stride));
    if (cudaGetLastError() != cudaSuccess) return TCU_ERR_CUDA;
    for (int b = 0; b < terms; ++b) {
        Call in = make_call(planes + size_t(b) * in_stride, sums + size_t(b) * out_stride, 1, size_t(tiles),
                            is_int ? TCU_I8_I32 : TCU_BF16_F32, c.s, false, inner_ws, nested_ws_bytes(tiles), c.stream);
        in.nested = true;
        in.upper_path = c.upper_path;            // the inner scans take the same optional product levels
        in.spin_limit = c.spin_limit;
        tcu_scan_stats_t inner;
        in.stats_out = &inner;
        const tcu_status_t st = scan_impl(in);
        if (st != TCU_OK) return st;
        *inner_mma += inner.mma_instructions;
    }
    if (is_int) tcu_totals_combine_kernel<true><<<blocks, 256, 0, c.stream>>>(c.d_ws, uint32_t(tiles), sums, uint32_t(out_stride));
    else tcu_totals_combine_kernel<false><<<blocks, 256, 0, c.stream>>>(c.d_ws, uint32_t(tiles), sums, uint32_t(out_stride));
    if (cudaGetLastError() != cudaSuccess) return TCU_ERR_CUDA;
    // Whatever is not a record is wiped before the call returns the workspace: a later, larger scan keeps its records
    // here, and a left-over word must never read as a record of its epoch (zero is the epoch of no launch).
    return cudaMemsetAsync(base, 0, nested_bytes(tiles), c.stream) == cudaSuccess ? TCU_OK : TCU_ERR_CUDA;
}

tcu_status_t scan_impl(const Call &c) {
    const tcu_status_t chk = check_call(c);
    if (chk != TCU_OK || c.rows == 0 || c.cols == 0) return chk;
    const void *d_in = c.d_in;
    void *d_out = c.d_out;
    const size_t rows = c.rows, cols = c.cols;
    const tcu_dtype_t dt = c.dt;
    const int s = c.s;
    const bool exclusive = c.exclusive, level0 = c.level0, two_sweep = c.two_sweep;
    void *d_ws = c.d_ws;
    cudaStream_t stream = c.stream;
    const int eb = elem_bytes(dt);

    const uint64_t rows128 = cols / kTileCols;
    const uint64_t tiles_per_row = (rows128 + kTileRows - 1) / kTileRows;
    const uint64_t tiles = rows * tiles_per_row;
    const uint32_t tail = uint32_t(cols % kTileCols);
    const int per32 = 32 / eb;
    const int seff = s > per32 ? s : per32;
    const int b_atoms = (seff * eb + 127) / 128;
    const uint32_t b_bytes = b_atoms == 1 ? uint32_t(seff * 128) : uint32_t(b_atoms * kAtomBytes);
    const uint32_t stage_bytes = kTileElems * eb;
    const bool upper_tc = c.upper_path >= 1 && !c.segmented && !level0;
    const bool chunk_tc = c.upper_path == 2 && s < kTileCols && !c.segmented && !level0;
    // the carry add as a product: for s = 128 one carry per row; for s < 128 one per chunk, which needs the chunk totals
    // out of the accumulator first, i.e. the chunk-product variant (upper_level_path = 2)
    const bool chunk_down = chunk_tc && (dt != TCU_I8_I32) && c.down_path == 1;
    const bool down_tc = ((dt != TCU_I8_I32) && s == 128 && !level0 && c.down_path == 1 && !c.segmented) || chunk_down;
    const size_t fixed = kConstOffset + kOnesBytes + b_bytes + size_t(kOutRingBytes) + (upper_tc ? (dt == TCU_I8_I32 ? kUpperBytesInt : kUpperBytesFloat) : 0) +
                         (down_tc && !chunk_down ? kDownBytes : 0) + (chunk_tc ? kChunkBytes : 0) + (chunk_down ? kAtomBytes : 0) + (c.segmented ? kSegRingBytes : 0) + 1024;  // + alignment slack
    int in_stages = int((232448 - fixed) / stage_bytes);
    if (in_stages > kUseInStages) in_stages = kUseInStages;
    if (in_stages < 2) return TCU_ERR_UNSUPPORTED;
    const size_t smem = fixed + size_t(in_stages) * stage_bytes;

    tcu_scan_stats_t st;
    std::memset(&st, 0, sizeof(st));
    st.rows = rows;
    st.cols = cols;
    st.s = s;
    st.dtype = dt;
    st.exclusive = exclusive;
    st.variant = two_sweep ? 1 : 0;
    st.upper_level_path = upper_tc ? uint32_t(c.upper_path) : 0;
    st.down_sweep_path = down_tc ? 1 : 0;
    st.tiles = tiles;
    st.mma_instructions = tiles * uint64_t((kTileCols / seff) * (seff / per32) + kTileCols / per32 + (upper_tc ? (dt == TCU_I8_I32 ? 4 : 8) : 0) + (chunk_tc ? (dt == TCU_I8_I32 ? 1 : 2) : 0) + (chunk_down ? (3 * (kTileCols / s) + 15) / 16 : (down_tc ? 1 : 0)));  // U_s products + row-total products
    st.sxs_products = tiles * uint64_t(kTileElems / (s * s));
    // product level, chain over the chunks of a row (absent when s = 128), scan over the 128 rows,
    // scan over the tiles (absent for a single tile), carry add
    st.levels_used = 1 + (s < kTileCols ? 1 : 0) + 1 + (tiles_per_row > 1 ? 1 : 0) + 1;
    st.depth_bound = 2 * floor_log(cols, uint64_t(s));
    st.in_stages = in_stages;
    st.smem_bytes = uint32_t(smem);
    st.tail_elements = tail;
    st.segments_path = c.segmented ? 1 : 0;

    // segmented scan: note, for every row of 128 elements that holds a segment start, whether it starts the row
    // and what the row hands on (eight lanes per start), before the tile kernel runs
    uint8_t *seg_flag = nullptr;
    uint32_t *seg_val = nullptr;
    SegSource seg{c.d_offsets, c.seg_pitch, c.num_segments};
    const unsigned seg_blocks = unsigned((c.num_segments * kSegLanes + 255) / 256);
    if (c.segmented) {
        seg_flag = reinterpret_cast<uint8_t *>(d_ws) + seg_flag_offset(cols);
        seg_val = reinterpret_cast<uint32_t *>(reinterpret_cast<uint8_t *>(d_ws) + seg_val_offset(cols));
        if (rows128 > 0) {
            if (cudaMemsetAsync(seg_flag, 0, size_t(tiles) * kTileRows, stream) != cudaSuccess) return TCU_ERR_CUDA;
            if (dt == TCU_I8_I32)
                tcu_segment_rows_kernel<true, false, kSegPrepare><<<seg_blocks, 256, 0, stream>>>(d_in, d_out, cols, seg, d_ws, uint32_t(tiles), seg_flag, seg_val, dt);
            else
                tcu_segment_rows_kernel<false, false, kSegPrepare><<<seg_blocks, 256, 0, stream>>>(d_in, d_out, cols, seg, d_ws, uint32_t(tiles), seg_flag, seg_val, dt);
            if (cudaGetLastError() != cudaSuccess) return TCU_ERR_CUDA;
        }
    }

    if (tiles > 0) {
        EncodeTiledFn encode = get_encode_fn();
        if (!encode) return TCU_ERR_CUDA;
        int sms = sm_count();
        if (sms <= 0) return TCU_ERR_CUDA;
        ScanParams prm;
        std::memset(&prm, 0, sizeof(prm));
        // persistent grid: every CTA must be resident at once (the carry chain waits on
        // lower-numbered tiles), so never more CTAs than SMs; one CTA fills an SM's shared memory
        uint64_t ctas = uint64_t(sms);
        const int cap = c.max_ctas;
        if (cap > 0 && uint64_t(cap) < ctas) ctas = uint64_t(cap);

        const cuuint64_t dims[3] = {cuuint64_t(kTileCols), cuuint64_t(rows128), cuuint64_t(rows)};
        const cuuint32_t estr[3] = {1, 1, 1};
        // stride between scans: the row pitch for batched input; for a single array any multiple of
        // 16 bytes will do (the coordinate is always 0), and n itself need not be one
        const cuuint64_t pitch_elems = rows > 1 ? cuuint64_t(cols) : cuuint64_t(rows128) * kTileCols;
        {
            const cuuint64_t strides[2] = {cuuint64_t(kTileCols) * eb, pitch_elems * eb};
            const cuuint32_t box[3] = {cuuint32_t(128 / eb), cuuint32_t(kTileRows), 1};
            CUtensorMapDataType ty = dt == TCU_I8_I32 ? CU_TENSOR_MAP_DATA_TYPE_UINT8
                                     : dt == TCU_F16_F32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16
                                                         : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
            CUresult r = encode(&prm.tmap_in, ty, 3, const_cast<void *>(d_in), dims, strides, box, estr,
                                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (r != CUDA_SUCCESS) return TCU_ERR_CUDA;
        }
        prm.ws = d_ws;
        prm.out = d_out;
        prm.carry_in = c.d_carry_in;
        prm.carry_out = c.d_carry_out;
        prm.stamps = c.d_stamps;
        prm.spin_limit = c.spin_limit;
        prm.skip_publish_tile = c.skip_tile;
        prm.seg_rowflag = seg_flag;
        prm.seg_rowval = seg_val;
        prm.scan_pitch = cols;
        prm.rows128 = uint32_t(rows128);
        prm.tiles_total = uint32_t(tiles);
        prm.tiles_per_row = uint32_t(tiles_per_row);
        prm.in_stages = uint32_t(in_stages);
        prm.b_bytes = b_bytes;
        prm.dtype = uint32_t(dt);
        prm.level0_only = level0 ? 1u : 0u;
        prm.prefilled = two_sweep ? 1u : 0u;
        prm.upper_tc = upper_tc ? 1u : 0u;
        prm.down_tc = down_tc ? 1u : 0u;
        if (two_sweep) {
            // sweep 1: one total per tile; then their scan, written as the records sweep 2 looks back over
            const uint64_t valid = uint64_t(rows128) * kTileCols;
            if (dt == TCU_I8_I32) tcu_tile_totals_kernel<true><<<unsigned(tiles), 256, 0, stream>>>(d_in, d_ws, valid, dt);
            else tcu_tile_totals_kernel<false><<<unsigned(tiles), 256, 0, stream>>>(d_in, d_ws, valid, dt);
            if (cudaGetLastError() != cudaSuccess) return TCU_ERR_CUDA;
            if (totals_by_scan(c)) {
                uint64_t inner_mma = 0;
                const tcu_status_t ts = scan_totals_by_scan(c, tiles, &inner_mma);
                if (ts != TCU_OK) return ts;
                st.mma_instructions += inner_mma;
                st.levels_used += 1;             // (the totals go through a scan of their own)
            } else {
                if (dt == TCU_I8_I32) tcu_totals_scan_kernel<true><<<1, 1024, 0, stream>>>(d_ws, uint32_t(tiles));
                else tcu_totals_scan_kernel<false><<<1, 1024, 0, stream>>>(d_ws, uint32_t(tiles));
                if (cudaGetLastError() != cudaSuccess) return TCU_ERR_CUDA;
            }
        }
        dim3 grid(unsigned(tiles < ctas ? tiles : ctas));
        st.grid = grid.x;
        // the plain scan has a kernel of its own, with every option compiled out
        const bool plain = !upper_tc && !down_tc && !c.segmented && !level0 && !two_sweep && !c.d_stamps && !c.d_carry_out &&
                           c.skip_tile == kNoTile;
        const int variant = chunk_tc ? kChunk : (plain ? kLean : kFull);
        cudaError_t e;
        if (dt == TCU_I8_I32)
            e = exclusive ? dispatch_s<true, true>(s, variant, prm, grid, smem, stream) : dispatch_s<true, false>(s, variant, prm, grid, smem, stream);
        else
            e = exclusive ? dispatch_s<false, true>(s, variant, prm, grid, smem, stream) : dispatch_s<false, false>(s, variant, prm, grid, smem, stream);
        if (e != cudaSuccess) return TCU_ERR_CUDA;
    }
    if (c.segmented) {
        // rows that hold a start: rescan them from the first start on; then the incomplete last row, if any
        auto launch = [&](auto is_int, auto excl) {
            constexpr bool I = decltype(is_int)::value, E = decltype(excl)::value;
            if (rows128 > 0)
                tcu_segment_rows_kernel<I, E, kSegFixup><<<seg_blocks, 256, 0, stream>>>(d_in, d_out, cols, seg, d_ws, uint32_t(tiles), seg_flag, seg_val, dt);
            if (tail > 0)
                tcu_segment_rows_kernel<I, E, kSegTail><<<1, 32, 0, stream>>>(d_in, d_out, cols, seg, d_ws, uint32_t(tiles), seg_flag, seg_val, dt);
        };
        if (dt == TCU_I8_I32) {
            if (exclusive) launch(std::true_type{}, std::true_type{});
            else launch(std::true_type{}, std::false_type{});
        } else {
            if (exclusive) launch(std::false_type{}, std::true_type{});
            else launch(std::false_type{}, std::false_type{});
        }
        if (cudaGetLastError() != cudaSuccess) return TCU_ERR_CUDA;
        // The row notes are not records: they are wiped before the call returns the workspace, because a later, larger
        // scan keeps its records where they lie, and a left-over word must never read as a record of its epoch.
        if (rows128 > 0 && cudaMemsetAsync(seg_flag, 0, seg_workspace_bytes(cols) - seg_flag_offset(cols), stream) != cudaSuccess)
            return TCU_ERR_CUDA;
    } else if (tail > 0) {   // the last cols % 128 elements of every scan
        const size_t start = size_t(rows128) * kTileCols;
        if (dt == TCU_I8_I32) {
            if (exclusive) tcu_scan_tail_kernel<true, true><<<unsigned(rows), 128, 0, stream>>>(d_in, d_out, start, size_t(cols), tail, d_ws, uint32_t(tiles_per_row), dt, c.d_carry_in, c.d_carry_out);
            else tcu_scan_tail_kernel<true, false><<<unsigned(rows), 128, 0, stream>>>(d_in, d_out, start, size_t(cols), tail, d_ws, uint32_t(tiles_per_row), dt, c.d_carry_in, c.d_carry_out);
        } else {
            if (exclusive) tcu_scan_tail_kernel<false, true><<<unsigned(rows), 128, 0, stream>>>(d_in, d_out, start, size_t(cols), tail, d_ws, uint32_t(tiles_per_row), dt, c.d_carry_in, c.d_carry_out);
            else tcu_scan_tail_kernel<false, false><<<unsigned(rows), 128, 0, stream>>>(d_in, d_out, start, size_t(cols), tail, d_ws, uint32_t(tiles_per_row), dt, c.d_carry_in, c.d_carry_out);
        }
        if (cudaGetLastError() != cudaSuccess) return TCU_ERR_CUDA;
    }
    t_stats = st;
    t_have_stats = true;
    if (c.stats_out) *c.stats_out = st;
    return TCU_OK;
}

Call make_call(const void *d_in, void *d_out, size_t rows, size_t cols, tcu_dtype_t dt, int s, bool exclusive, void *d_ws,
               size_t ws_bytes, cudaStream_t stream) {
    Call c;
    c.d_in = d_in;
    c.d_out = d_out;
    c.rows = rows;
    c.cols = cols;
    c.dt = dt;
    c.s = s;
    c.exclusive = exclusive;
    c.d_ws = d_ws;
    c.ws_bytes = ws_bytes;
    c.stream = stream;
    return c;
}

// Built-in scratch of tcu_scan_inclusive_noalloc: the tile records of the cross-tile carry scan for
// at most TCU_SCAN_NOALLOC_MAX_ELEMENTS elements.  One copy per GPU that loads this library, held
// until the process exits.  In host code this name is only a handle for the runtime: the address the
// kernels need comes from cudaGetSymbolAddress (see noalloc_scratch below).
constexpr size_t kNoAllocScratchBytes =
    size_t(kHeaderBytes) + 16 * (size_t(TCU_SCAN_NOALLOC_MAX_ELEMENTS) / kTileElems) + 16;
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

// Device address of the built-in scratch on the current device, looked up once per device.
tcu_status_t noalloc_scratch(void **out) {
    constexpr int kMaxDevices = 64;
    static std::mutex mu;
    static void *addr[kMaxDevices] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return TCU_ERR_CUDA;
    std::lock_guard<std::mutex> lk(mu);
    if (!addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return TCU_ERR_CUDA;
        addr[dev] = p;
    }
    *out = addr[dev];
    return TCU_OK;
}

// Streams and events of the pipelined host-buffer entry point: created on first use, per device, kept
// for the life of the process (host-side objects; no device memory).
struct HostPipe {
    static constexpr int kEvents = 64;      // far more than the pieces that can be in flight at once
    cudaStream_t up = nullptr, down = nullptr;
    cudaEvent_t start = nullptr, finish = nullptr;
    cudaEvent_t ev[kEvents] = {};
    bool ok = false;
};

HostPipe *host_pipe() {
    constexpr int kMaxDevices = 64;
    static std::mutex mu;
    static HostPipe pipes[kMaxDevices];
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lk(mu);
    HostPipe &p = pipes[dev];
    if (!p.ok) {
        bool good = cudaStreamCreateWithFlags(&p.up, cudaStreamNonBlocking) == cudaSuccess &&
                    cudaStreamCreateWithFlags(&p.down, cudaStreamNonBlocking) == cudaSuccess &&
                    cudaEventCreateWithFlags(&p.start, cudaEventDisableTiming) == cudaSuccess &&
                    cudaEventCreateWithFlags(&p.finish, cudaEventDisableTiming) == cudaSuccess;
        for (int i = 0; good && i < HostPipe::kEvents; ++i)
            good = cudaEventCreateWithFlags(&p.ev[i], cudaEventDisableTiming) == cudaSuccess;
        if (!good) return nullptr;
        p.ok = true;
    }
    return &p;
}

}  // namespace

extern "C" {

size_t tcu_scan_workspace_bytes(size_t rows, size_t cols, tcu_dtype_t dt, int s) {
    (void)dt;
    (void)s;
    if (rows > 1 && cols % 16 != 0) return seg_workspace_bytes(uint64_t(rows) * cols);   // rows become segments of one array
    const uint64_t tiles = tiles_for(rows, cols);
    // (room for every option: the two-sweep variant with the totals scanned by this library's own scan needs the most)
    return rows > 1 ? record_bytes(tiles) : nested_offset(tiles) + nested_bytes(tiles);
}

tcu_status_t tcu_scan_workspace_init(void *d_ws, size_t ws_bytes, cudaStream_t stream) {
    if (!d_ws || ws_bytes < size_t(kHeaderBytes)) return TCU_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(d_ws) & 255) return TCU_ERR_INVALID_ARG;
    return cudaMemsetAsync(d_ws, 0, ws_bytes, stream) == cudaSuccess ? TCU_OK : TCU_ERR_CUDA;
}

tcu_status_t tcu_scan_inclusive(const void *d_in, void *d_out, size_t n, tcu_dtype_t dt, int s, void *d_ws,
                                size_t ws_bytes, cudaStream_t stream) {
    return scan_impl(make_call(d_in, d_out, 1, n, dt, s, false, d_ws, ws_bytes, stream));
}

tcu_status_t tcu_scan_exclusive(const void *d_in, void *d_out, size_t n, tcu_dtype_t dt, int s, void *d_ws,
                                size_t ws_bytes, cudaStream_t stream) {
    return scan_impl(make_call(d_in, d_out, 1, n, dt, s, true, d_ws, ws_bytes, stream));
}

tcu_status_t tcu_scan_batched(const void *d_in, void *d_out, size_t rows, size_t cols, tcu_dtype_t dt, int s,
                              int exclusive, void *d_ws, size_t ws_bytes, cudaStream_t stream) {
    if (rows > 1 && cols % 16 != 0) {
        // rows that do not start 16-byte aligned cannot be tiled one by one: tile the array as a whole and treat
        // the row starts as segment starts
        if (cols > kMaxScanElements / rows) return TCU_ERR_UNSUPPORTED;
        Call c = make_call(d_in, d_out, 1, rows * cols, dt, s, exclusive != 0, d_ws, ws_bytes, stream);
        c.segmented = true;
        c.seg_pitch = cols;
        c.num_segments = rows;
        const tcu_status_t st = scan_impl(c);
        if (st == TCU_OK) {          // report the shape the caller asked for
            t_stats.rows = rows;
            t_stats.cols = cols;
        }
        return st;
    }
    return scan_impl(make_call(d_in, d_out, rows, cols, dt, s, exclusive != 0, d_ws, ws_bytes, stream));
}

size_t tcu_scan_segmented_workspace_bytes(size_t n, tcu_dtype_t dt, int s) {
    (void)dt;
    (void)s;
    return seg_workspace_bytes(n);
}

tcu_status_t tcu_scan_segmented(const void *d_in, void *d_out, size_t n, const uint64_t *d_offsets, size_t num_segments,
                                tcu_dtype_t dt, int s, int exclusive, void *d_ws, size_t ws_bytes, cudaStream_t stream) {
    if (n > 0 && (num_segments == 0 || !d_offsets)) return TCU_ERR_INVALID_ARG;
    Call c = make_call(d_in, d_out, 1, n, dt, s, exclusive != 0, d_ws, ws_bytes, stream);
    c.segmented = true;
    c.d_offsets = d_offsets;
    c.num_segments = num_segments;
    return scan_impl(c);
}

tcu_status_t tcu_scan_ex(const void *d_in, void *d_out, size_t rows, size_t cols, tcu_dtype_t dt, int s,
                         const tcu_scan_options_t *opt, tcu_scan_stats_t *stats_out, void *d_ws, size_t ws_bytes,
                         cudaStream_t stream) {
    Call c = make_call(d_in, d_out, rows, cols, dt, s, false, d_ws, ws_bytes, stream);
    c.stats_out = stats_out;
    if (opt) {
        if (opt->struct_bytes != sizeof(tcu_scan_options_t)) return TCU_ERR_INVALID_ARG;
        if (opt->variant > 1 || opt->max_ctas > (1u << 20)) return TCU_ERR_INVALID_ARG;
        if (opt->upper_level_path > 2 || opt->down_sweep_path > 1) return TCU_ERR_INVALID_ARG;
        c.exclusive = opt->exclusive != 0;
        c.two_sweep = opt->variant == 1;
        c.upper_path = int(opt->upper_level_path);
        c.down_path = int(opt->down_sweep_path);
        c.max_ctas = int(opt->max_ctas);
        c.d_carry_in = opt->d_carry_in;
        c.d_carry_out = opt->d_carry_out;
        c.d_stamps = reinterpret_cast<unsigned long long *>(opt->d_stamps);
    }
    return scan_impl(c);
}

tcu_status_t tcu_scan_inclusive_noalloc(const void *d_in, void *d_out, size_t n, tcu_dtype_t dt, int s,
                                        cudaStream_t stream) {
    if (n > size_t(TCU_SCAN_NOALLOC_MAX_ELEMENTS)) return TCU_ERR_TOO_LARGE;
    // every argument is checked before anything is queued on the stream (the scratch pointer is filled in below;
    // a placeholder with the right alignment stands in for it during the check)
    Call c = make_call(d_in, d_out, 1, n, dt, s, false, reinterpret_cast<void *>(uintptr_t(256)), kNoAllocScratchBytes, stream);
    const tcu_status_t chk = check_call(c);
    if (chk != TCU_OK || n == 0) return chk;
    void *scratch = nullptr;
    tcu_status_t st = noalloc_scratch(&scratch);
    if (st != TCU_OK) return st;
    // The scratch still holds the records of whatever call used it last.  Everything the kernels
    // expect to find at zero (header counters, the records of this call's tiles) is cleared here.
    const size_t used = record_bytes(tiles_for(1, n));           // (never more than the array: n was checked above)
    static_assert(kNoAllocScratchBytes >= size_t(kHeaderBytes) + 16 * (size_t(TCU_SCAN_NOALLOC_MAX_ELEMENTS) / kTileElems) + 16,
                  "the built-in scratch holds the records of the largest scan it accepts");
    if (used > kNoAllocScratchBytes) return TCU_ERR_TOO_LARGE;
    if (cudaMemsetAsync(scratch, 0, used, stream) != cudaSuccess) return TCU_ERR_CUDA;
    c.d_ws = scratch;
    return scan_impl(c);
}

tcu_status_t tcu_scan_noalloc_status(cudaStream_t stream) {
    void *scratch = nullptr;
    tcu_status_t st = noalloc_scratch(&scratch);
    if (st != TCU_OK) return st;
    return tcu_scan_device_status(scratch, stream);
}

tcu_status_t tcu_scan_level0_debug(const void *d_in, void *d_out, size_t n, tcu_dtype_t dt, int s, void *d_ws,
                                   size_t ws_bytes, cudaStream_t stream) {
    Call c = make_call(d_in, d_out, 1, n, dt, s, false, d_ws, ws_bytes, stream);
    c.level0 = true;
    return scan_impl(c);
}

tcu_status_t tcu_scan_host(const void *h_in, void *h_out, size_t n, tcu_dtype_t dt, int s, int exclusive, void *d_in,
                           void *d_out, void *d_ws, size_t ws_bytes, cudaStream_t stream) {
    if (!valid_dtype(dt)) return TCU_ERR_INVALID_ARG;
    if (n == 0) return TCU_OK;
    if (!h_in || !h_out || !d_in || !d_out) return TCU_ERR_INVALID_ARG;
    const size_t eb = size_t(elem_bytes(dt));
    constexpr size_t kChunk = size_t(1) << 24;                 // elements per piece (a multiple of the tile)
    Call whole = make_call(d_in, d_out, 1, n, dt, s, exclusive != 0, d_ws, ws_bytes, stream);
    const tcu_status_t chk = check_call(whole);
    if (chk != TCU_OK) return chk;
    HostPipe *pipe = (exclusive || n <= 2 * kChunk) ? nullptr : host_pipe();
    if (!pipe) {                                               // short or exclusive: one copy in, one scan, one copy out
        if (cudaMemcpyAsync(d_in, h_in, n * eb, cudaMemcpyHostToDevice, stream) != cudaSuccess) return TCU_ERR_CUDA;
        tcu_status_t st = scan_impl(whole);
        if (st != TCU_OK) return st;
        if (cudaMemcpyAsync(h_out, d_out, n * 4, cudaMemcpyDeviceToHost, stream) != cudaSuccess) return TCU_ERR_CUDA;
        return TCU_OK;
    }
    // Long inclusive scans are cut into pieces: the upload of piece i+1, the scan of piece i (continuing from the
    // total of the pieces before it) and the download of piece i-1 overlap, each on its own stream.  The total
    // travels as an 8-byte carry through two slots of the workspace header, used in turn.
    const uint8_t *hi = reinterpret_cast<const uint8_t *>(h_in);
    uint8_t *ho = reinterpret_cast<uint8_t *>(h_out);
    uint8_t *di = reinterpret_cast<uint8_t *>(d_in), *dout = reinterpret_cast<uint8_t *>(d_out);
    uint64_t *slots = reinterpret_cast<WsHeader *>(d_ws)->carry_slot;      // (address arithmetic only)
    if (cudaEventRecord(pipe->start, stream) != cudaSuccess) return TCU_ERR_CUDA;    // the caller's earlier work comes first
    cudaStreamWaitEvent(pipe->up, pipe->start, 0);
    cudaStreamWaitEvent(pipe->down, pipe->start, 0);
    const size_t pieces = (n + kChunk - 1) / kChunk;
    for (size_t i = 0; i < pieces; ++i) {
        const size_t lo = i * kChunk, len = (lo + kChunk <= n) ? kChunk : n - lo;
        cudaEvent_t up_done = pipe->ev[(2 * i) % HostPipe::kEvents], scan_done = pipe->ev[(2 * i + 1) % HostPipe::kEvents];
        if (cudaMemcpyAsync(di + lo * eb, hi + lo * eb, len * eb, cudaMemcpyHostToDevice, pipe->up) != cudaSuccess) return TCU_ERR_CUDA;
        cudaEventRecord(up_done, pipe->up);
        cudaStreamWaitEvent(stream, up_done, 0);
        Call c = make_call(di + lo * eb, dout + lo * 4, 1, len, dt, s, false, d_ws, ws_bytes, stream);
        c.d_carry_in = i == 0 ? nullptr : &slots[(i - 1) & 1];
        c.d_carry_out = &slots[i & 1];
        tcu_status_t st = scan_impl(c);
        if (st != TCU_OK) return st;
        cudaEventRecord(scan_done, stream);
        cudaStreamWaitEvent(pipe->down, scan_done, 0);
        if (cudaMemcpyAsync(ho + lo * 4, dout + lo * 4, len * 4, cudaMemcpyDeviceToHost, pipe->down) != cudaSuccess) return TCU_ERR_CUDA;
    }
    if (cudaEventRecord(pipe->finish, pipe->down) != cudaSuccess) return TCU_ERR_CUDA;
    cudaStreamWaitEvent(stream, pipe->finish, 0);              // synchronising `stream` now covers the downloads too
    return cudaGetLastError() == cudaSuccess ? TCU_OK : TCU_ERR_CUDA;
}

tcu_status_t tcu_scan_device_status(const void *d_ws, cudaStream_t stream) {
    if (!d_ws) return TCU_ERR_WORKSPACE;
    WsHeader h;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return TCU_ERR_CUDA;
    if (cudaMemcpy(&h, d_ws, sizeof(h), cudaMemcpyDeviceToHost) != cudaSuccess) return TCU_ERR_CUDA;
    return h.error == 0 ? TCU_OK : TCU_ERR_TIMEOUT;
}

tcu_status_t tcu_scan_selftest_timeout(const void *d_in, void *d_out, size_t n, tcu_dtype_t dt, int s, size_t skip_tile,
                                       unsigned limit_ms, int upper_level_path, int down_sweep_path, void *d_ws,
                                       size_t ws_bytes, cudaStream_t stream) {
    if (limit_ms == 0 || limit_ms > 1000) return TCU_ERR_INVALID_ARG;
    if (n == 0 || n % kTileCols != 0 || skip_tile >= tiles_for(1, n)) return TCU_ERR_INVALID_ARG;
    Call c = make_call(d_in, d_out, 1, n, dt, s, false, d_ws, ws_bytes, stream);
    c.upper_path = upper_level_path;           // (range-checked with the other arguments)
    c.down_path = down_sweep_path;
    c.skip_tile = uint32_t(skip_tile);
    c.spin_limit = (long long)limit_ms * 2000000LL;            // about 2 cycles per nanosecond
    return scan_impl(c);
}

tcu_status_t tcu_reduce_total(const void *d_in, size_t n, tcu_dtype_t dt, void *d_total, void *d_ws, size_t ws_bytes,
                              cudaStream_t stream) {
    if (!valid_dtype(dt)) return TCU_ERR_INVALID_ARG;
    if (!d_total || (reinterpret_cast<uintptr_t>(d_total) & 7)) return TCU_ERR_INVALID_ARG;
    if (n > 0 && (!d_in || (reinterpret_cast<uintptr_t>(d_in) & 15))) return TCU_ERR_INVALID_ARG;
    if (n > kMaxScanElements) return TCU_ERR_UNSUPPORTED;
    if (!d_ws) return TCU_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(d_ws) & 255) return TCU_ERR_INVALID_ARG;
    if (ws_bytes < tcu_scan_workspace_bytes(1, n + kTileElems, dt, 16)) return TCU_ERR_WORKSPACE;
    // one total per 128 x 128-element tile over the whole 16-byte pieces, then one block adds them and the
    // few elements that are left
    const size_t per_piece = 16 / size_t(elem_bytes(dt));
    const uint64_t whole = uint64_t(n / per_piece) * per_piece;
    const uint32_t tiles = uint32_t((whole + kTileElems - 1) / kTileElems);
    if (dt == TCU_I8_I32) {
        if (tiles) tcu_tile_totals_kernel<true><<<tiles, 256, 0, stream>>>(d_in, d_ws, whole, dt);
        tcu_sum_totals_kernel<true><<<1, 1024, 0, stream>>>(d_ws, tiles, d_in, whole, uint32_t(n - whole), dt, d_total);
    } else {
        if (tiles) tcu_tile_totals_kernel<false><<<tiles, 256, 0, stream>>>(d_in, d_ws, whole, dt);
        tcu_sum_totals_kernel<false><<<1, 1024, 0, stream>>>(d_ws, tiles, d_in, whole, uint32_t(n - whole), dt, d_total);
    }
    return cudaGetLastError() == cudaSuccess ? TCU_OK : TCU_ERR_CUDA;
}

tcu_status_t tcu_carry_exclusive_prefix(const void *d_totals, size_t count, size_t index, tcu_dtype_t dt, void *d_carry,
                                        cudaStream_t stream) {
    if (!valid_dtype(dt)) return TCU_ERR_INVALID_ARG;
    if (!d_carry || (reinterpret_cast<uintptr_t>(d_carry) & 7) || index > count || count > (1u << 20)) return TCU_ERR_INVALID_ARG;
    if (count > 0 && (!d_totals || (reinterpret_cast<uintptr_t>(d_totals) & 7))) return TCU_ERR_INVALID_ARG;
    if (dt == TCU_I8_I32)
        tcu_carry_prefix_kernel<true><<<1, 32, 0, stream>>>(reinterpret_cast<const uint64_t *>(d_totals), uint32_t(index),
                                                          reinterpret_cast<uint64_t *>(d_carry));
    else
        tcu_carry_prefix_kernel<false><<<1, 32, 0, stream>>>(reinterpret_cast<const uint64_t *>(d_totals), uint32_t(index),
                                                           reinterpret_cast<uint64_t *>(d_carry));
    return cudaGetLastError() == cudaSuccess ? TCU_OK : TCU_ERR_CUDA;
}

size_t tcu_sort_tmp_bytes(size_t n) {
    // flags (n bytes, padded), scanned flags (4 n), second key buffer (4 n); each part 256-byte aligned
    const size_t a = (n + 255) & ~size_t(255), b = (4 * n + 255) & ~size_t(255);
    return a + 2 * b + 256;
}

tcu_status_t tcu_sort_u32(const uint32_t *d_keys_in, uint32_t *d_keys_out, size_t n, void *d_tmp, size_t tmp_bytes,
                          void *d_ws, size_t ws_bytes, cudaStream_t stream) {
    if (n == 0) return TCU_OK;
    if (!d_keys_in || !d_keys_out || !d_tmp) return TCU_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(d_keys_in) & 15) || (reinterpret_cast<uintptr_t>(d_keys_out) & 15) ||
        (reinterpret_cast<uintptr_t>(d_tmp) & 255))
        return TCU_ERR_INVALID_ARG;
    if (n >= (size_t(1) << 31)) return TCU_ERR_UNSUPPORTED;          // positions are int32 scan results
    if (tmp_bytes < tcu_sort_tmp_bytes(n)) return TCU_ERR_WORKSPACE;
    const size_t a = (n + 255) & ~size_t(255), b = (4 * n + 255) & ~size_t(255);
    int8_t *flags = reinterpret_cast<int8_t *>(d_tmp);
    int32_t *f = reinterpret_cast<int32_t *>(reinterpret_cast<uint8_t *>(d_tmp) + a);
    uint32_t *other = reinterpret_cast<uint32_t *>(reinterpret_cast<uint8_t *>(d_tmp) + a + b);
    const tcu_status_t chk = check_call(make_call(flags, f, 1, n, TCU_I8_I32, 16, true, d_ws, ws_bytes, stream));
    if (chk != TCU_OK) return chk;
    // 32 passes ping-pong between `other` and d_keys_out so that the last pass lands in d_keys_out
    const uint32_t *src = d_keys_in;
    for (int bit = 0; bit < 32; ++bit) {
        uint32_t *dst = (bit & 1) ? d_keys_out : other;
        const unsigned blocks4 = unsigned((n + 4 * 256 - 1) / (4 * 256));
        split_flags_kernel<<<blocks4, 256, 0, stream>>>(src, flags, n, bit);
        tcu_status_t st = scan_impl(make_call(flags, f, 1, n, TCU_I8_I32, 16, true, d_ws, ws_bytes, stream));
        if (st != TCU_OK) return st;
        split_scatter_kernel<<<unsigned((n + 255) / 256), 256, 0, stream>>>(src, flags, f, dst, n);
        if (cudaGetLastError() != cudaSuccess) return TCU_ERR_CUDA;
        src = dst;
    }
    return TCU_OK;
}

tcu_status_t tcu_widen_copy(const void *d_in, void *d_out, size_t n, tcu_dtype_t dt, cudaStream_t stream) {
    if (dt != TCU_I8_I32 && dt != TCU_F16_F32 && dt != TCU_BF16_F32) return TCU_ERR_INVALID_ARG;
    if (n == 0) return TCU_OK;
    if (!d_in || !d_out || (n % 4) != 0) return TCU_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(d_in) & 15) || (reinterpret_cast<uintptr_t>(d_out) & 15)) return TCU_ERR_INVALID_ARG;
    const uint64_t pieces = n / 4, per_block = uint64_t(kWidenThreads) * kWidenPerThread;
    const uint64_t blocks = (pieces + per_block - 1) / per_block;
    if (blocks >= (1ull << 31)) return TCU_ERR_UNSUPPORTED;
    if (dt == TCU_I8_I32) tcu_widen_copy_kernel<0><<<unsigned(blocks), kWidenThreads, 0, stream>>>(d_in, d_out, pieces);
    else if (dt == TCU_F16_F32) tcu_widen_copy_kernel<1><<<unsigned(blocks), kWidenThreads, 0, stream>>>(d_in, d_out, pieces);
    else tcu_widen_copy_kernel<2><<<unsigned(blocks), kWidenThreads, 0, stream>>>(d_in, d_out, pieces);
    return cudaGetLastError() == cudaSuccess ? TCU_OK : TCU_ERR_CUDA;
}

tcu_status_t tcu_scan_last_stats(tcu_scan_stats_t *out) {
    if (!out) return TCU_ERR_INVALID_ARG;
    if (!t_have_stats) return TCU_ERR_INVALID_ARG;
    *out = t_stats;
    return TCU_OK;
}

#ifdef TCU_PROFILE
// Debug build only (see the debug section of tcu_scan_kernel.cuh): point the kernels at a device buffer of
// 64 wait counters per CTA, or of 8 time stamps per tile.
int tcu_scan_debug_set_profile_buffer(void *d_buf) {
    unsigned long long *p = reinterpret_cast<unsigned long long *>(d_buf);
    return cudaMemcpyToSymbol(tcu::g_prof, &p, sizeof(p)) == cudaSuccess ? 0 : 4;
}
int tcu_scan_debug_set_trace_buffer(void *d_buf) {
    unsigned long long *p = reinterpret_cast<unsigned long long *>(d_buf);
    return cudaMemcpyToSymbol(tcu::g_trace, &p, sizeof(p)) == cudaSuccess ? 0 : 4;
}
#endif

const char *tcu_status_string(tcu_status_t st) {
    switch (st) {
        case TCU_OK: return "ok";
        case TCU_ERR_INVALID_ARG: return "invalid argument";
        case TCU_ERR_UNSUPPORTED: return "unsupported request";
        case TCU_ERR_WORKSPACE: return "workspace missing or too small";
        case TCU_ERR_CUDA: return "CUDA call failed";
        case TCU_ERR_TIMEOUT: return "device-side wait timed out";
        case TCU_ERR_TOO_LARGE: return "problem larger than the built-in scratch allows";
        default: return "unknown status";
    }
}

}  // extern "C"
