/*
 * tcu_scan.h - C ABI of the B200 (sm_100a) tensor-core-unit prefix-sum library.
 *
 * The library computes the inclusive / exclusive prefix sum ("scan") of the paper
 * "A Parallel Scan Algorithm in the Tensor Core Unit Model" in its (s^2, l)-TCU
 * formulation: the input is viewed as s x s tiles, every length-s chunk is scanned
 * by a dense product with the triangular all-ones matrix on the tensor cores
 * (Algorithm 1, up-sweep round t = 0), chunk / row / tile totals are scanned above
 * that (up-sweep rounds t >= 1 and Section 2.2 steps 2-3), and the carries are added
 * back (down-sweep and Section 2.2 step 4) - all in one pass over HBM.
 *
 * General conventions
 * -------------------
 *  - Every `d_*` pointer is a DEVICE pointer owned by the caller; the library never
 *    allocates or frees device memory and keeps no pointer after a call returns.
 *    Every `h_*` pointer is a HOST pointer.
 *  - All scan calls are asynchronous on `stream`.  Argument errors are detected on
 *    the host and returned before anything is queued on the stream.  A device-side wait
 *    that gave up (it never spins forever) is reported by tcu_scan_device_status().
 *  - Input and output must not overlap (element widths differ, so the paper's
 *    in-place form is not offered).  `d_in` and `d_out` must be 16-byte aligned.
 *  - Integer output is the exact sum modulo 2^32 (two's complement int32).
 *    Floating-point output is fp32; the association order of the additions is not
 *    specified and may differ between calls in the last bits.
 *  - `s` is the paper's tile size: chunks of `s` consecutive elements are scanned by
 *    one U_s product.  Supported: 16, 64, 128.
 *  - The workspace must have been cleared once by tcu_scan_workspace_init() before
 *    its first use; it may then be reused by any number of calls, of any shape whose
 *    requirement fits, as long as calls that share it do not overlap in time.
 *  - The library keeps no state between calls except the bookkeeping of the calling
 *    thread's last scan (tcu_scan_last_stats); every choice is an argument of the call.
 *  - A "carry" that travels between calls (tcu_scan_options_t.d_carry_in / d_carry_out,
 *    tcu_reduce_total, tcu_carry_exclusive_prefix) is an 8-byte device value: a double
 *    for the floating-point types, a zero-extended uint32 for TCU_I8_I32.
 */
#ifndef TCU_SCAN_H_
#define TCU_SCAN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#ifndef __DRIVER_TYPES_H__
typedef struct CUstream_st *cudaStream_t; /* same declaration as the CUDA runtime's */
#endif

typedef enum {
    TCU_OK = 0,
    TCU_ERR_INVALID_ARG = 1, /* NULL pointer, misaligned pointer, s or dtype out of range, overlap */
    TCU_ERR_UNSUPPORTED = 2, /* valid request the library does not implement (see each call)      */
    TCU_ERR_WORKSPACE = 3,   /* workspace missing or smaller than tcu_scan_workspace_bytes()       */
    TCU_ERR_CUDA = 4,        /* a CUDA runtime / driver call failed (no device, launch failure...) */
    TCU_ERR_TIMEOUT = 5,     /* a bounded device-side wait ran out; the output is not valid        */
    TCU_ERR_TOO_LARGE = 6    /* tcu_scan_inclusive_noalloc: n exceeds TCU_SCAN_NOALLOC_MAX_ELEMENTS */
} tcu_status_t;

/* input element type -> output element type */
typedef enum {
    TCU_I8_I32 = 0,  /* int8  -> int32, exact (tcgen05 kind::i8)  */
    TCU_F16_F32 = 1, /* fp16  -> fp32         (tcgen05 kind::f16) */
    TCU_BF16_F32 = 2 /* bf16  -> fp32         (tcgen05 kind::f16) */
} tcu_dtype_t;

/* What one scan call did (host-side bookkeeping, filled at launch). */
typedef struct {
    uint64_t rows, cols;        /* problem shape (rows = 1 for the single-array calls)               */
    uint32_t s, dtype, exclusive;
    uint32_t variant;           /* 0 = single pass, decoupled look-back; 1 = two sweeps                 */
    uint32_t upper_level_path;  /* where the levels above the U_s products ran: see tcu_scan_options_t */
    uint64_t tiles;             /* 128 x 128-element tiles processed                                  */
    uint64_t mma_instructions;  /* tcgen05.mma instructions issued                                    */
    uint64_t sxs_products;      /* s x s-equivalent U_s products they amount to ( = padded n / s^2 )  */
    uint32_t levels_used;       /* depth of the GPU hierarchy (product, in-row, cross-row, cross-tile,
                                   carry add), to be compared with the paper's 2 floor(log_s n)        */
    uint32_t depth_bound;       /* 2 floor(log_s cols), Corollary 1                                   */
    uint32_t grid, smem_bytes, in_stages, tail_elements;
    uint32_t down_sweep_path;   /* 0 = carries added on the vector ALUs; 1 = by a tensor-core product        */
    uint32_t segments_path;     /* 0 = dense rows; 1 = segment boundaries inside the array (segmented call, or
                                   batched rows whose length is not a multiple of 16)                    */
} tcu_scan_stats_t;

/* Per-call choices of tcu_scan_ex().  Zero-initialise, set struct_bytes = sizeof(tcu_scan_options_t),
 * then set what differs from the defaults. */
typedef struct {
    uint32_t struct_bytes;
    uint32_t exclusive;         /* 0 = inclusive, 1 = exclusive */
    uint32_t variant;           /* 0 = single pass with decoupled look-back (default); 1 = two sweeps:
                                   reduce every tile, scan the totals, then scan with every carry known
                                   (reads the input twice; exists so that the choice can be measured)  */
    uint32_t upper_level_path;  /* Paper Section 2 keeps every level of the up-sweep a product of two square
                                   matrices; the totals that the upper levels work on are int32 / fp32,
                                   which are not tensor-core input types.
                                   0 (default) = upper levels on the CUDA cores (register chain along a
                                       row, warp shuffles across the 128 rows of a tile);
                                   1 = the scan over the 128 row totals of a tile is a tcgen05 product of
                                       a strictly lower triangular all-ones matrix with the totals split
                                       into exact narrow terms (two signed 8-bit limbs for int8 input,
                                       three bf16 terms for fp16 / bf16 input), recombined afterwards.
                                   2 = in addition, for s < 128, the carries of the 128 / s chunks of a row are
                                       the product of the chunk totals (split the same way) with a strictly
                                       upper triangular ones matrix, instead of a chain of additions along
                                       the row (for s = 128 a row is one chunk and 2 means 1).
                                   Integer results are identical, floating-point results satisfy the
                                   same tolerance.  In the single-pass variant the level across tiles stays a
                                   look-back on CUDA cores; in the two-sweep variant (variant = 1) a value >= 1
                                   also sends the scan of the tile totals (Section 2.2 step 3) through the
                                   tensor-core scan: each total is split exactly into narrow terms (four signed
                                   base-256 digits; the fp32-rounded total in three bf16 terms), every term
                                   array is scanned by an inner call of this library with the same s and the
                                   same value of this option, and the scanned terms are recombined (shifts
                                   and adds mod 2^32; three fp32 sums added in fp64). */
    uint32_t down_sweep_path;   /* Paper Section 2, matrix B_s, and the discussion's remark that the tensor
                                   unit is used at O(1/s) in the down-sweep.  1 = fp16 / bf16 scans add the
                                   carries by a tcgen05 product instead of one vector add per element:
                                   with s = 128, each row's carry to the whole row (accumulator += C * ones,
                                   C holding the carry split exactly into three bf16 terms); with s < 128
                                   and upper_level_path = 2 (which provides the carries of the chunks), each
                                   chunk's carry to the s elements of the chunk (accumulator += C * E, C
                                   holding the 128 / s carries of a row in three bf16 terms each, E a 0 / 1
                                   matrix that selects the chunk of every column).  Ignored otherwise
                                   (integer scans: no pair of 8-bit operands adds a 32-bit carry). */
    uint32_t max_ctas;          /* 0 = one persistent CTA per SM; otherwise at most this many.  One CTA owns
                                   one SM's tensor core, so this is the p of the paper's p-TCU time bound
                                   O(n(1 + l/s^2)/p + (s^2 + l) log_s n) (Section 2.2, last paragraph).
                                   Results do not depend on it. */
    const void *d_carry_in;     /* single array only: carry (8 bytes, see above) that precedes x[0], or NULL */
    void *d_carry_out;          /* single array only: receives carry_in + x[0] + ... + x[n-1] (8 bytes), or NULL;
                                   not written when n = 0 */
    uint64_t *d_stamps;         /* NULL, or TCU_SCAN_STAMPS_PER_CTA values per CTA of the launch (at most one
                                   CTA per SM): %globaltimer nanoseconds at fixed points of the kernel, for
                                   taking the fixed cost of a launch apart (index meanings: entry, set-up
                                   done, previous kernel done, first tile claimed, landed, published, carry
                                   known, stored, role loops done, all warps done, exit, tiles by group 0/1) */
} tcu_scan_options_t;
#define TCU_SCAN_STAMPS_PER_CTA 16

/* Bytes of device workspace needed to scan `rows` independent rows of `cols` elements
 * (rows = 1 for the single-array calls).  Holds the per-tile {flag, aggregate / inclusive
 * prefix} records of the cross-tile carry scan (Section 2.2 steps 2-3: segment totals and
 * their scan); when cols is not a multiple of 16 and rows > 1, also the per-row boundary
 * notes of the segmented path; for a single array, also the scratch of the two-sweep variant
 * when it scans the tile totals with the library's own scan (tcu_scan_options_t: variant = 1
 * with upper_level_path >= 1) - the size covers every option of tcu_scan_ex, about 40 bytes
 * per 128 x 128-element tile in all.  Never fails; returns a small non-zero size even for
 * empty problems.
 * One workspace may serve calls of different sizes, types and kinds, one after the other on a
 * stream, if it is large enough for each: records are tagged with the number of the launch that
 * wrote them, and everything else a call keeps in the workspace (row notes, the two-sweep
 * scratch) is wiped before the call's work on the stream ends.  Two calls that could run at the
 * same time on the GPU (different streams, no dependency between them) need a workspace each.
 * The launch number is a 32-bit count kept in the workspace: clear the workspace again
 * (tcu_scan_workspace_init) before it has served 2^32 launches.
 * The scan calls that take a workspace only queue kernels and memsets on `stream` (no
 * synchronisation, no allocation), so a sequence of them can be captured into a CUDA graph and
 * replayed (tested for tcu_scan_inclusive). */
size_t tcu_scan_workspace_bytes(size_t rows, size_t cols, tcu_dtype_t dt, int s);

/* Clear a workspace (asynchronous memset on `stream`).  Must run once before the first
 * scan that uses `d_ws`, and again if a call ever reported TCU_ERR_TIMEOUT. */
tcu_status_t tcu_scan_workspace_init(void *d_ws, size_t ws_bytes, cudaStream_t stream);

/* Inclusive scan, y[i] = x[0] + ... + x[i]  (paper Section 1: the default meaning of
 * "prefix sum"; Algorithm 1 + Section 2.2 for arbitrary n).
 *   d_in   device, n elements of the input type, 16-byte aligned
 *   d_out  device, n elements of the output type (4 bytes each), 16-byte aligned
 *   n      any value from 0 to 2^37 (n = 0 returns TCU_OK without a launch; more: TCU_ERR_UNSUPPORTED)
 *   d_ws   device workspace of at least tcu_scan_workspace_bytes(1, n, dt, s) bytes */
tcu_status_t tcu_scan_inclusive(const void *d_in, void *d_out, size_t n, tcu_dtype_t dt, int s,
                                void *d_ws, size_t ws_bytes, cudaStream_t stream);

/* Exclusive scan, y[0] = 0, y[i] = x[0] + ... + x[i-1]  (the paper names the exclusive
 * form only in Table 1; this is the standard reading: shifted by one, identity 0 in front).
 * Arguments as for tcu_scan_inclusive. */
tcu_status_t tcu_scan_exclusive(const void *d_in, void *d_out, size_t n, tcu_dtype_t dt, int s,
                                void *d_ws, size_t ws_bytes, cudaStream_t stream);

/* `rows` independent scans of `cols` elements each, dense row-major (row stride = cols)
 * (Section 2.2 step 1: the algorithm run on each contiguous segment, no stitching).
 * Any cols >= 1.  When cols is a multiple of 16 every row starts 16-byte aligned and the rows
 * are tiled one by one; otherwise the array is tiled as a whole and the row starts are
 * segment boundaries inside it (the path of tcu_scan_segmented; rows * cols <= 2^37).
 *   d_ws   at least tcu_scan_workspace_bytes(rows, cols, dt, s) bytes */
tcu_status_t tcu_scan_batched(const void *d_in, void *d_out, size_t rows, size_t cols,
                              tcu_dtype_t dt, int s, int exclusive,
                              void *d_ws, size_t ws_bytes, cudaStream_t stream);

/* Segmented scan: the array is cut into `num_segments` consecutive segments and every segment
 * is scanned on its own (Section 2.2, steps 1-4, with the segments given by the caller instead
 * of the base-s digits of n: scan each segment, take the segment totals, scan them, add them
 * back - here with the chain of carries cut at every segment start).
 *   d_offsets  device, num_segments + 1 values of uint64: segment k is [offsets[k], offsets[k+1]);
 *              non-decreasing, offsets[0] = 0, offsets[num_segments] = n (the caller's promise:
 *              the values live on the device and are not checked); empty segments are allowed
 *   d_ws       at least tcu_scan_segmented_workspace_bytes(n, dt, s) bytes, cleared once like any
 *              workspace
 * Elements of a segment whose 128-element row (rows are counted from the start of the array)
 * holds no segment start go through the tensor-core path; rows that hold a start are rescanned
 * from that start on by CUDA cores. */
size_t tcu_scan_segmented_workspace_bytes(size_t n, tcu_dtype_t dt, int s);
tcu_status_t tcu_scan_segmented(const void *d_in, void *d_out, size_t n, const uint64_t *d_offsets,
                                size_t num_segments, tcu_dtype_t dt, int s, int exclusive,
                                void *d_ws, size_t ws_bytes, cudaStream_t stream);

/* The general form: rows = 1 for a single array.  `opt` may be NULL (all defaults); `stats_out`
 * may be NULL, otherwise it receives what tcu_scan_last_stats() would return after this call. */
tcu_status_t tcu_scan_ex(const void *d_in, void *d_out, size_t rows, size_t cols, tcu_dtype_t dt, int s,
                         const tcu_scan_options_t *opt, tcu_scan_stats_t *stats_out,
                         void *d_ws, size_t ws_bytes, cudaStream_t stream);

/* Inclusive scan for callers that cannot hand the library a workspace.  (The paper has no
 * counterpart for this entry point; it exists for integration reasons only.)
 *
 * Some callers have no way to allocate device memory at the moment they need a scan: a plug-in
 * that lives inside a host program which carved up the GPU's memory at start-up and forbids
 * cudaMalloc afterwards (it would stall the device and may fail under a fixed budget), or a
 * routine on a hot path that must not take the allocator's lock.  For them the tile records of
 * the cross-tile carry scan live in a fixed array that is part of the library image itself.
 * The caller still passes the input and the output; the call allocates and frees nothing.
 *
 *   n       at most TCU_SCAN_NOALLOC_MAX_ELEMENTS, else TCU_ERR_TOO_LARGE (nothing is launched)
 *   others  as for tcu_scan_inclusive; they are checked before anything is queued on the stream
 *
 * Cost: every GPU on which the library is loaded holds about 64 KiB for the array until the
 * process ends, whether this entry point is used or not.
 * First use: the first call on each device looks up the array's device address (that device
 * must be current); make that first call before starting any stream capture.
 * Sharing: there is one array per device and every call uses it, so two calls whose kernels
 * could overlap on the GPU (different streams, no dependency between them) corrupt each
 * other's carries; serialise them.  Each call clears the part of the array it needs, on
 * `stream`, before its kernel runs - which also wipes the record of an earlier time-out, so
 * ask tcu_scan_noalloc_status() after a call whose result matters, before the next call. */
#define TCU_SCAN_NOALLOC_MAX_ELEMENTS (1u << 26)
tcu_status_t tcu_scan_inclusive_noalloc(const void *d_in, void *d_out, size_t n, tcu_dtype_t dt, int s,
                                        cudaStream_t stream);

/* What tcu_scan_device_status() is for a workspace, for the built-in array of
 * tcu_scan_inclusive_noalloc on the current device: synchronises `stream`, then returns TCU_OK,
 * or TCU_ERR_TIMEOUT if the most recent noalloc call gave up a bounded wait.  (No counterpart
 * in the paper.)  Allocates nothing. */
tcu_status_t tcu_scan_noalloc_status(cudaStream_t stream);

/* Debug / teaching entry: only up-sweep round t = 0 of Algorithm 1, i.e. every chunk of
 * s consecutive elements replaced by its own inclusive scan (W = L_s T), no carries.
 * n must be a multiple of 128.  Same arguments otherwise. */
tcu_status_t tcu_scan_level0_debug(const void *d_in, void *d_out, size_t n, tcu_dtype_t dt, int s,
                                   void *d_ws, size_t ws_bytes, cudaStream_t stream);

/* Host-buffer form: uploads h_in to d_in, scans, downloads d_out to h_out.  Everything is
 * asynchronous; the caller synchronises `stream` before reading h_out (that also covers the
 * copies, which long inclusive scans run on two internal streams so that upload, scan and
 * download of successive 2^24-element pieces overlap; each piece continues from the total of
 * the pieces before it, handed over as an 8-byte carry inside the workspace).  h_in / h_out
 * should be pinned, otherwise the copies serialise.
 * d_in / d_out are caller-owned device staging buffers of n input / n output elements; they and
 * the workspace are in use until `stream` has drained. */
tcu_status_t tcu_scan_host(const void *h_in, void *h_out, size_t n, tcu_dtype_t dt, int s, int exclusive,
                           void *d_in, void *d_out, void *d_ws, size_t ws_bytes, cudaStream_t stream);

/* Synchronises `stream`, then returns TCU_OK, or TCU_ERR_TIMEOUT if any kernel that used
 * `d_ws` since its last init gave up a bounded wait (its output is then not valid). */
tcu_status_t tcu_scan_device_status(const void *d_ws, cudaStream_t stream);

/* Self-test of the failure path (no counterpart in the paper): runs the ordinary inclusive scan
 * kernel on the given input, except that the records of tile `skip_tile` (128 x 128 elements per
 * tile) are never published and every device-side wait gives up after `limit_ms` milliseconds
 * (1..1000) instead of about a second.  Tiles after `skip_tile` therefore wait in vain, the
 * kernel records the time-out, winds down (drains its copies, frees its tensor memory) and
 * returns.  After the stream has drained, tcu_scan_device_status(d_ws) returns TCU_ERR_TIMEOUT,
 * the output is not valid, and the context is still usable; tcu_scan_workspace_init() clears
 * the condition.  Nothing faults or hangs.  skip_tile must be below the number of tiles, and
 * n a multiple of 128.  upper_level_path / down_sweep_path select the same optional tensor-core
 * branches as in tcu_scan_options_t (0 / 0: the ordinary path), whose store and totals warps meet
 * at barriers inside their loops and must therefore give up together. */
tcu_status_t tcu_scan_selftest_timeout(const void *d_in, void *d_out, size_t n, tcu_dtype_t dt, int s,
                                       size_t skip_tile, unsigned limit_ms, int upper_level_path,
                                       int down_sweep_path, void *d_ws, size_t ws_bytes, cudaStream_t stream);

/* One array split over several devices (paper Section 2.2 steps 2-4 with one segment per device,
 * and the p-TCU bound of its last paragraph): each device computes the total of its shard
 * (tcu_reduce_total), the totals are exchanged by the caller (8 bytes per device, e.g. an NCCL
 * all-gather into local memory), each device sums the totals of the shards before its own
 * (tcu_carry_exclusive_prefix) and scans its shard with that carry (tcu_scan_ex, d_carry_in).
 *
 * tcu_reduce_total: *d_total = x[0] + ... + x[n-1] as an 8-byte carry.  d_in 16-byte aligned;
 *   d_ws as for a scan of n elements (its tile records are used as scratch).
 * tcu_carry_exclusive_prefix: *d_carry = totals[0] + ... + totals[index-1] (8-byte carries,
 *   count >= index values at d_totals). */
tcu_status_t tcu_reduce_total(const void *d_in, size_t n, tcu_dtype_t dt, void *d_total,
                              void *d_ws, size_t ws_bytes, cudaStream_t stream);
tcu_status_t tcu_carry_exclusive_prefix(const void *d_totals, size_t count, size_t index, tcu_dtype_t dt,
                                        void *d_carry, cudaStream_t stream);

/* Radix sort of 32-bit unsigned keys by 32 stable one-bit splits, each split an exclusive
 * tcu scan of int8 flags (the paper's introduction asks whether a tensor-core-unit machine
 * can sort; with Blelloch's reduction of radix sort to prefix sums it can).  An application
 * of the scan, not a tuned sort.
 *   d_keys_in / d_keys_out   device, n keys each, 16-byte aligned, must not overlap
 *   d_tmp                    device scratch of tcu_sort_tmp_bytes(n) bytes, 256-byte aligned
 *   d_ws                     scan workspace of tcu_scan_workspace_bytes(1, n, TCU_I8_I32, 16) bytes
 *   n < 2^31 */
size_t tcu_sort_tmp_bytes(size_t n);
tcu_status_t tcu_sort_u32(const uint32_t *d_keys_in, uint32_t *d_keys_out, size_t n, void *d_tmp, size_t tmp_bytes,
                          void *d_ws, size_t ws_bytes, cudaStream_t stream);

/* Measuring aid (no counterpart in the paper): out[i] = in[i] widened to the output type of `dt` (int8 -> int32,
 * fp16 / bf16 -> fp32, all exact), a plain copy kernel with the traffic mix of the scan of that type (1 or 2 bytes
 * read, 4 bytes written per element) and no dependence between elements.  The benchmark times it beside the scan to
 * show what that mix reaches on the machine's memory system.
 *   d_in, d_out   device pointers, 16-byte aligned, not overlapping; n elements, n a multiple of 4
 * Errors: TCU_ERR_INVALID_ARG (null or misaligned pointer, n not a multiple of 4, unknown dt), TCU_ERR_UNSUPPORTED
 * (n >= 2^42), TCU_ERR_CUDA (the launch failed).  Asynchronous on `stream`. */
tcu_status_t tcu_widen_copy(const void *d_in, void *d_out, size_t n, tcu_dtype_t dt, cudaStream_t stream);

/* Copies the bookkeeping of the most recent scan call made by the calling thread. */
tcu_status_t tcu_scan_last_stats(tcu_scan_stats_t *out);

const char *tcu_status_string(tcu_status_t st);

#ifdef __cplusplus
}
#endif
#endif /* TCU_SCAN_H_ */
