/*
 * CPU oracle for the mask statistics of CAST (arxiv 2509.25996, App. C):
 *
 *   numerator of r_t / i_t   ||M - M_ref||_0     (M_ref = the previous mask for r_t, the initial mask for i_t)
 *   sparse weight ratio S_t  ||W (.) M||_1 / ||W||_1, returned as its two sums
 *
 * THIS FILE IS TEST INFRASTRUCTURE: a plain serial loop in fp64, written from the definitions so that it
 * can be checked against them by eye.  It shares no code with the CUDA library; only tests, the smoke
 * check and the CPU-baseline leg of the benchmark run it.
 *
 * Pins (tests/test_oracle_pins.py): numpy sums over a mask decoded independently in the tests; closed
 * forms (full density gives S = 1 and equal masks give 0 flips; complementary 2:4 masks flip every entry).
 *
 * Masks are stored as the library-neutral metadata of the AdamS oracle: M bits per group, packed LSB
 * first into row-major 32-bit words, cols/32 words per row; either a keep bitmask per group or, for 2:4,
 * the two kept positions lo | hi << 2.
 */
#include <math.h>
#include <stdint.h>

static uint32_t stats_field(const uint32_t *meta, int64_t r, int64_t cols, int64_t i, int M)
{
    int64_t bit = i * M;
    uint32_t word = meta[r * (cols / 32) + bit / 32];
    uint32_t field_mask = (M == 32) ? 0xFFFFFFFFu : ((1u << M) - 1u);
    return (word >> (bit % 32)) & field_mask;
}

static uint32_t stats_keep(uint32_t field, int bitmask_encoding)
{
    if (bitmask_encoding) return field;
    return (1u << (field & 3u)) | (1u << ((field >> 2) & 3u));
}

/* out[0] += ||M - M_ref||_0 (0 when meta_ref is NULL); out_sums[0] += ||W (.) M||_1; out_sums[1] += ||W||_1 */
int oracle_mask_stats(const float *w, const uint32_t *meta, const uint32_t *meta_ref,
                      int64_t rows, int64_t cols, int M, int bitmask_encoding,
                      uint64_t *out_flips, double *out_sums)
{
    if (!w || !meta || !out_flips || !out_sums) return -1;
    if (rows < 0 || cols < 0 || M < 1 || M > 32 || 32 % M != 0 || cols % 32 != 0) return -1;
    if (!bitmask_encoding && M != 4) return -1;
    uint64_t flips = 0;
    double kept_abs = 0.0, total_abs = 0.0;
    for (int64_t r = 0; r < rows; ++r) {
        for (int64_t i = 0; i < cols / M; ++i) {
            uint32_t keep = stats_keep(stats_field(meta, r, cols, i, M), bitmask_encoding);
            if (meta_ref) {
                uint32_t ref = stats_keep(stats_field(meta_ref, r, cols, i, M), bitmask_encoding);
                for (int j = 0; j < M; ++j)
                    flips += ((keep >> j) & 1u) != ((ref >> j) & 1u);          /* ||M - M_ref||_0 */
            }
            for (int j = 0; j < M; ++j) {
                double a = fabs((double)w[r * cols + i * M + j]);
                total_abs += a;                                                  /* ||W||_1        */
                if ((keep >> j) & 1u) kept_abs += a;                             /* ||W (.) M||_1  */
            }
        }
    }
    *out_flips += flips;
    out_sums[0] += kept_abs;
    out_sums[1] += total_abs;
    return 0;
}
