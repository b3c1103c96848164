/*
 * CPU oracle for the final pruning of CAST (arxiv 2509.25996, Alg. 2, final loop; Alg. 1, last lines):
 *
 *     W^ = W (.) M ,  then the scale is folded in:  W^ <- Diag(A~) W^    (Eq. 12 applied to the pruned matrix)
 *
 * with M either chosen now by magnitude (Eq. 6 with exactly N kept per group, Eq. 4; ties to the lower
 * column) or read from stored metadata.  No optimizer state is touched.
 *
 * THIS FILE IS TEST INFRASTRUCTURE: a plain serial loop in fp64, shared with nothing in the CUDA library.
 * Pins (tests/test_oracle_pins.py): numpy's stable argsort for the kept set, torch's bf16 conversion for the
 * values, gather/scatter through an independently decoded mask for the two output layouts.
 *
 * Output layouts: dense (rows x cols, pruned slots +0.0) or compressed (rows x cols*N/M, the N kept values
 * of each group in column order).  Metadata as in the AdamS oracle: M bits per group packed LSB first into
 * row-major 32-bit words, either a keep bitmask or, for 2:4, lo | hi << 2.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

#define PF_RESELECT   1u
#define PF_BITMASK    4u
#define PF_COMPRESSED 32u

static uint16_t pf_bf16_rne(double x)      /* round to nearest even, from the format's definition */
{
    uint16_t sign = (uint16_t)(signbit(x) ? 0x8000u : 0u);
    double a = fabs(x);
    if (isnan(x)) return (uint16_t)(sign | 0x7FC0u);
    if (isinf(x)) return (uint16_t)(sign | 0x7F80u);
    if (a == 0.0) return sign;
    int e;
    (void)frexp(a, &e);
    int binade = e - 1;
    if (binade < -126) binade = -126;
    double q = ldexp(1.0, binade - 7);
    double r = nearbyint(a / q) * q;
    if (r >= ldexp(1.0, 128)) return (uint16_t)(sign | 0x7F80u);
    float rf = (float)r;
    uint32_t bits;
    memcpy(&bits, &rf, sizeof bits);
    return (uint16_t)(sign | (uint16_t)(bits >> 16));
}

int oracle_prune_fold(const float *w, const float *scale, int n_seg, uint32_t *meta, uint16_t *out,
                      int64_t rows, int64_t cols, int N, int M, uint32_t flags)
{
    if (!w || !meta || !out) return -1;
    if (rows < 0 || cols < 0 || M < 1 || M > 32 || 32 % M != 0 || N < 1 || N > M || cols % 32 != 0) return -1;
    const int bitmask = (flags & PF_BITMASK) != 0;
    if (!bitmask && !(N == 2 && M == 4)) return -1;
    if (scale && (n_seg < 1 || cols % n_seg != 0 || (cols / n_seg) % M != 0)) return -1;
    const uint32_t field_mask = (M == 32) ? 0xFFFFFFFFu : ((1u << M) - 1u);
    for (int64_t r = 0; r < rows; ++r) {
        for (int64_t i = 0; i < cols / M; ++i) {
            const int64_t base = r * cols + i * M;
            const int64_t bit = i * M;
            uint32_t *word = &meta[r * (cols / 32) + bit / 32];
            uint32_t keep = 0;
            if (flags & PF_RESELECT) {
                for (int j = 0; j < M; ++j) {            /* kept iff fewer than N entries come before it */
                    float aj = fabsf(w[base + j]);
                    int before = 0;
                    for (int k = 0; k < M; ++k) {
                        float ak = fabsf(w[base + k]);
                        if (k != j && (ak > aj || (ak == aj && k < j))) ++before;
                    }
                    if (before < N) keep |= 1u << j;
                }
            } else {
                uint32_t field = (*word >> (bit % 32)) & field_mask;
                keep = bitmask ? field : ((1u << (field & 3u)) | (1u << ((field >> 2) & 3u)));
            }
            int emitted = 0;
            for (int j = 0; j < M; ++j) {
                const int kept = (keep >> j) & 1u;
                const int64_t col = i * M + j;
                const double a = scale ? (double)scale[r * n_seg + col / (cols / n_seg)] : 1.0;
                const uint16_t val = pf_bf16_rne(a * (double)w[base + j]);        /* Diag(A~) (W (.) M) */
                if (flags & PF_COMPRESSED) {
                    if (kept && emitted < N) out[(r * (cols / M) + i) * N + emitted++] = val;
                } else {
                    out[base + j] = kept ? val : 0;
                }
            }
            uint32_t field = keep;
            if (!bitmask) {
                int lo = -1, hi = -1;
                for (int j = 0; j < 4; ++j)
                    if (keep & (1u << j)) { if (lo < 0) lo = j; else hi = j; }
                field = (uint32_t)lo | ((uint32_t)hi << 2);
            }
            *word = (*word & ~(field_mask << (bit % 32))) | ((field & field_mask) << (bit % 32));
        }
    }
    return 0;
}
