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
 *    the host and returned before anything is launched.  A device-side wait that
 *    gave up (it never spins forever) is reported by tcu_scan_device_status().
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

/* What the last scan call of this process did (host-side bookkeeping, filled at launch). */
typedef struct {
    uint64_t rows, cols;        /* problem shape (rows = 1 for the single-array calls)               */
    uint32_t s, dtype, exclusive;
    uint32_t variant;           /* 0 = single pass, decoupled look-back; 1 = two sweeps                 */
    uint32_t upper_level_path;  /* 0 = levels above the products run on CUDA cores (warp shuffles);
                                   1 = the scan over the 128 row totals is a tensor-core product on 8-bit limbs */
    uint64_t tiles;             /* 128 x 128-element tiles processed                                  */
    uint64_t mma_instructions;  /* tcgen05.mma instructions issued                                    */
    uint64_t sxs_products;      /* s x s-equivalent U_s products they amount to ( = padded n / s^2 )  */
    uint32_t levels_used;       /* depth of the GPU hierarchy (product, in-row, cross-row, cross-tile,
                                   carry add), to be compared with the paper's 2 floor(log_s n)        */
    uint32_t depth_bound;       /* 2 floor(log_s cols), Corollary 1                                   */
    uint32_t grid, smem_bytes, in_stages, tail_elements;
    uint32_t down_sweep_path;   /* 0 = carries added on the vector ALUs; 1 = by a tensor-core product        */
} tcu_scan_stats_t;

/* Bytes of device workspace needed to scan `rows` independent rows of `cols` elements
 * (rows = 1 for the single-array calls).  Holds the per-tile {flag, aggregate / inclusive
 * prefix} records of the cross-tile carry scan (Section 2.2 steps 2-3: segment totals and
 * their scan).  Never fails; returns a small non-zero size even for empty problems. */
size_t tcu_scan_workspace_bytes(size_t rows, size_t cols, tcu_dtype_t dt, int s);

/* Clear a workspace (asynchronous memset on `stream`).  Must run once before the first
 * scan that uses `d_ws`, and again if a call ever reported TCU_ERR_TIMEOUT. */
tcu_status_t tcu_scan_workspace_init(void *d_ws, size_t ws_bytes, cudaStream_t stream);

/* Inclusive scan, y[i] = x[0] + ... + x[i]  (paper Section 1: the default meaning of
 * "prefix sum"; Algorithm 1 + Section 2.2 for arbitrary n).
 *   d_in   device, n elements of the input type, 16-byte aligned
 *   d_out  device, n elements of the output type (4 bytes each), 16-byte aligned
 *   n      any value >= 0 (n = 0 returns TCU_OK without a launch)
 *   d_ws   device workspace of at least tcu_scan_workspace_bytes(1, n, dt, s) bytes */
tcu_status_t tcu_scan_inclusive(const void *d_in, void *d_out, size_t n, tcu_dtype_t dt, int s,
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
 *   others  as for tcu_scan_inclusive
 *
 * Cost: every GPU on which the library is loaded holds about 64 KiB for the array until the
 * process ends, whether this entry point is used or not.
 * First use: the first call on each device looks up the array's device address (that device
 * must be current); make that first call before starting any stream capture.
 * Sharing: there is one array per device and every call uses it, so two calls whose kernels
 * could overlap on the GPU (different streams, no dependency between them) corrupt each
 * other's carries; serialise them.  Each call clears the part of the array it needs, on
 * `stream`, before its kernel runs. */
#define TCU_SCAN_NOALLOC_MAX_ELEMENTS (1u << 26)
tcu_status_t tcu_scan_inclusive_noalloc(const void *d_in, void *d_out, size_t n, tcu_dtype_t dt, int s,
                                        cudaStream_t stream);

/* Exclusive scan, y[0] = 0, y[i] = x[0] + ... + x[i-1]  (the paper names the exclusive
 * form only in Table 1; this is the standard reading: shifted by one, identity 0 in front).
 * Arguments as for tcu_scan_inclusive. */
tcu_status_t tcu_scan_exclusive(const void *d_in, void *d_out, size_t n, tcu_dtype_t dt, int s,
                                void *d_ws, size_t ws_bytes, cudaStream_t stream);

/* The same inclusive scan in the two-sweep structure of classical work-efficient scans (the
 * paper's up-sweep / down-sweep split across kernels): sweep 1 reads the input and reduces every
 * tile to its total, a one-block kernel scans the totals, sweep 2 is the single-pass kernel with
 * every carry already known.  It reads the input twice and exists so that the choice between
 * the two structures can be measured; results satisfy the same parity bars.  Arguments as for
 * tcu_scan_inclusive. */
tcu_status_t tcu_scan_inclusive_twosweep(const void *d_in, void *d_out, size_t n, tcu_dtype_t dt, int s,
                                         void *d_ws, size_t ws_bytes, cudaStream_t stream);

/* `rows` independent scans of `cols` elements each, dense row-major (row stride = cols)
 * (Section 2.2 step 1: the algorithm run on each contiguous segment, no stitching).
 * cols must be a multiple of 16 (so that every row starts 16-byte aligned in both arrays), else
 * TCU_ERR_UNSUPPORTED.
 *   d_ws   at least tcu_scan_workspace_bytes(rows, cols, dt, s) bytes */
tcu_status_t tcu_scan_batched(const void *d_in, void *d_out, size_t rows, size_t cols,
                              tcu_dtype_t dt, int s, int exclusive,
                              void *d_ws, size_t ws_bytes, cudaStream_t stream);

/* Debug / teaching entry: only up-sweep round t = 0 of Algorithm 1, i.e. every chunk of
 * s consecutive elements replaced by its own inclusive scan (W = L_s T), no carries.
 * n must be a multiple of 128.  Same arguments otherwise. */
tcu_status_t tcu_scan_level0_debug(const void *d_in, void *d_out, size_t n, tcu_dtype_t dt, int s,
                                   void *d_ws, size_t ws_bytes, cudaStream_t stream);

/* Host-buffer form: uploads h_in to d_in, scans, downloads d_out to h_out.  Everything is
 * asynchronous; the caller synchronises `stream` before reading h_out (that also covers the
 * copies, which long inclusive scans run on two internal streams so that upload, scan and
 * download of successive 2^24-element pieces overlap; each piece continues from the last output
 * of the piece before it).  h_in / h_out should be pinned, otherwise the copies serialise.
 * d_in / d_out are caller-owned device staging buffers of n input / n output elements; they and
 * the workspace are in use until `stream` has drained. */
tcu_status_t tcu_scan_host(const void *h_in, void *h_out, size_t n, tcu_dtype_t dt, int s, int exclusive,
                           void *d_in, void *d_out, void *d_ws, size_t ws_bytes, cudaStream_t stream);

/* Synchronises `stream`, then returns TCU_OK, or TCU_ERR_TIMEOUT if any kernel that used
 * `d_ws` since its last init gave up a bounded wait (its output is then not valid). */
tcu_status_t tcu_scan_device_status(const void *d_ws, cudaStream_t stream);

/* Self-test of the failure path (no counterpart in the paper): launches one warp that waits,
 * for at most `limit_ms` milliseconds (1..1000), on a tile record that nothing publishes, and
 * then records the time-out in the workspace header the way the scan kernels do.  After the
 * stream has drained, tcu_scan_device_status(d_ws) returns TCU_ERR_TIMEOUT and the context is
 * still usable; tcu_scan_workspace_init() clears the condition.  Nothing faults or hangs. */
tcu_status_t tcu_scan_selftest_timeout(void *d_ws, size_t ws_bytes, unsigned limit_ms, cudaStream_t stream);

/* Radix sort of 32-bit unsigned keys by 32 stable one-bit splits, each split an exclusive
 * tcu scan of int8 flags (the paper's introduction: with Blelloch's reduction of radix sort to
 * prefix sums, a tensor-core-unit machine can sort).  An application of the scan, not a tuned
 * sort.
 *   d_keys_in / d_keys_out   device, n keys each, 16-byte aligned, must not overlap
 *   d_tmp                    device scratch of tcu_sort_tmp_bytes(n) bytes, 256-byte aligned
 *   d_ws                     scan workspace of tcu_scan_workspace_bytes(1, n, TCU_I8_I32, 16) bytes
 *   n < 2^31 */
size_t tcu_sort_tmp_bytes(size_t n);
tcu_status_t tcu_sort_u32(const uint32_t *d_keys_in, uint32_t *d_keys_out, size_t n, void *d_tmp, size_t tmp_bytes,
                          void *d_ws, size_t ws_bytes, cudaStream_t stream);

/* Experiment knob (paper Section 2: "all numerical operations are multiplications between two
 * square matrices"): path = 1 makes the following int8 scans of this process compute the scan over
 * the 128 row totals of a tile - an upper level of the up-sweep, whose int32 operands are not a
 * tensor-core input type - as a tcgen05 kind::i8 product of a strictly lower triangular all-ones
 * matrix with the totals split into two signed 8-bit limbs, recombined exactly.  path = 0 (default)
 * uses warp shuffles.  Results are identical; tcu_scan_stats_t.upper_level_path records the choice.
 * Floating-point inputs always use path 0. */
tcu_status_t tcu_scan_set_upper_level_path(int path);

/* Experiment knob (paper Section 2, matrix B_s, and the discussion's remark that the tensor unit is
 * used at O(1/s) in the down-sweep): path = 1 makes the following fp16 / bf16 scans with s = 128
 * add each row's carry to the whole row by a tcgen05 product - accumulator += C * ones, C holding
 * the carry split exactly into three bf16 terms - instead of one vector add per element.  Other
 * dtypes and tile sizes ignore it.  Results satisfy the same tolerance;
 * tcu_scan_stats_t.down_sweep_path records the choice. */
tcu_status_t tcu_scan_set_down_sweep_path(int path);

/* Experiment knob: run the following scans of this process on at most `max_ctas` persistent CTAs,
 * i.e. on that many SMs (0 restores the default, one CTA per SM).  One CTA owns one SM's tensor
 * core, so this is the p of the paper's p-TCU time bound O(n(1 + l/s^2)/p + (s^2 + l) log_s n)
 * (Section 2.2, last paragraph, and the abstract).  Results do not depend on it. */
tcu_status_t tcu_scan_set_max_ctas(int max_ctas);

/* Copies the bookkeeping of the most recent scan call made by this process. */
tcu_status_t tcu_scan_last_stats(tcu_scan_stats_t *out);

const char *tcu_status_string(tcu_status_t st);

#ifdef __cplusplus
}
#endif
#endif /* TCU_SCAN_H_ */
