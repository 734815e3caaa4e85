/*
 * Result oracle for the prefix sum ("scan"): the definition, written out.
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing in the product path may call, link or
 * import this file; it exists so that the tests, the smoke check and the
 * benchmark's CPU-baseline leg have something slow and obviously correct to
 * compare the GPU library against.  It shares no code with the CUDA path.
 *
 * What it computes (paper, Section 1, notation paragraph: "prefix sum" means
 * the inclusive prefix sum unless stated otherwise; the operator is +):
 *
 *     inclusive:  y[i] = init + x[0] + x[1] + ... + x[i]
 *     exclusive:  y[i] = init + x[0] + ... + x[i-1],   y[0] = init
 *
 * evaluated strictly left to right, one running accumulator, no blocking, no
 * reordering.  Integer input is accumulated in int64 (exact for every size
 * this library accepts); floating-point input has already been widened
 * exactly to fp64 by the caller and is accumulated in fp64.
 *
 * For the floating-point tolerance the same pass also produces
 *     a[i] = sum of |x[j]| over the same index range as y[i] (without init),
 * so that a test can check  |y_gpu[i] - y[i]| <= 1e-5 * a[i] + 1e-6.
 *
 * The exclusive scan is not defined by the paper beyond the word itself
 * (Table 1 lists Blelloch's scan as "exclusive"); the reading used is the
 * standard one: shift right by one, identity element 0 in front.
 */
#include <stddef.h>
#include <stdint.h>
#include <math.h>

void oracle_scan_i8_i64(const int8_t *x, size_t n, int exclusive, int64_t init, int64_t *y)
{
    int64_t acc = init;
    for (size_t i = 0; i < n; ++i) {
        if (exclusive) {
            y[i] = acc;
            acc += (int64_t)x[i];
        } else {
            acc += (int64_t)x[i];
            y[i] = acc;
        }
    }
}

void oracle_scan_f64(const double *x, size_t n, int exclusive, double init, double *y, double *a)
{
    double acc = init;
    double abs_acc = 0.0;
    for (size_t i = 0; i < n; ++i) {
        if (exclusive) {
            y[i] = acc;
            if (a) a[i] = abs_acc;
            acc += x[i];
            abs_acc += fabs(x[i]);
        } else {
            acc += x[i];
            abs_acc += fabs(x[i]);
            y[i] = acc;
            if (a) a[i] = abs_acc;
        }
    }
}

/* Row-wise form: `rows` independent scans of length `cols`, dense row-major
 * (paper, Section 2.2 step 1: the same algorithm run on each contiguous
 * segment, here without the stitching steps because rows are independent). */
void oracle_scan_rows_i8_i64(const int8_t *x, size_t rows, size_t cols, int exclusive, int64_t *y)
{
    for (size_t r = 0; r < rows; ++r)
        oracle_scan_i8_i64(x + r * cols, cols, exclusive, 0, y + r * cols);
}

void oracle_scan_rows_f64(const double *x, size_t rows, size_t cols, int exclusive, double *y, double *a)
{
    for (size_t r = 0; r < rows; ++r)
        oracle_scan_f64(x + r * cols, cols, exclusive, 0.0, y + r * cols, a ? a + r * cols : (double *)0);
}

/* Segmented form: the array is cut at offsets[0] = 0 <= offsets[1] <= ... <= offsets[num_segments] = n and
 * every piece [offsets[k], offsets[k+1]) is scanned on its own, from zero (paper, Section 2.2 steps 1-4 build
 * the scan of a long array out of independent scans of consecutive segments plus their totals; here the
 * totals are not carried over, because the segments are separate problems).  Empty pieces are allowed. */
void oracle_scan_segments_i8_i64(const int8_t *x, const uint64_t *offsets, size_t num_segments, int exclusive, int64_t *y)
{
    for (size_t k = 0; k < num_segments; ++k)
        oracle_scan_i8_i64(x + offsets[k], (size_t)(offsets[k + 1] - offsets[k]), exclusive, 0, y + offsets[k]);
}

void oracle_scan_segments_f64(const double *x, const uint64_t *offsets, size_t num_segments, int exclusive, double *y, double *a)
{
    for (size_t k = 0; k < num_segments; ++k)
        oracle_scan_f64(x + offsets[k], (size_t)(offsets[k + 1] - offsets[k]), exclusive, 0.0, y + offsets[k],
                        a ? a + offsets[k] : (double *)0);
}
