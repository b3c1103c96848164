/*
 * CPU oracle for one AdamS step with N:M selection, proportional L1 decay,
 * weight scaling and mask metadata (CAST, arxiv 2509.25996).
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It is a plain, slow, serial loop written
 * from the paper so that a reader can check it against the paper by eye.  It
 * shares no code with the CUDA library, is never linked into it, and only the
 * tests, the smoke check and the CPU-baseline leg of the benchmark may run it.
 *
 * The file is compiled twice (see build_oracle.py): once with -DREAL=double
 * (entry point oracle_adams_step_f64: every operation in fp64, each stored
 * result rounded once to its storage type) and once with -DREAL=float (entry
 * point oracle_adams_step_f32: every operation in fp32 in the order written
 * here; compiled with -ffp-contract=off so nothing is fused).
 *
 * What is pinned, and by what (tests/test_oracle_pins.py):
 *   selection            brute force over all C(M,N) masks; the paper's 1:2
 *                        worked example (Sec. 5.1); Eq. 4 group counts
 *   Adam core            torch.optim.Adam on CPU (beta1 = 0 literal reading;
 *                        any beta1 under ORACLE_F_V_KEPT_FROM_G), closed forms
 *   L1 decay             closed forms at alpha = 1 and at Sign(0)
 *   scaling / emission   power-of-two scales, library bf16 conversion
 *   metadata, flips      hand-decoded masks, hand-counted flips
 * Multi-step trajectories have no printed values in the paper: the long-run
 * behaviour test is a smoke test only (parity unpinned for trajectories).
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

#ifndef REAL
#error "compile with -DREAL=double or -DREAL=float"
#endif
#ifndef ENTRY
#error "compile with -DENTRY=oracle_adams_step_f64 or _f32"
#endif

typedef REAL real;

/* flag bits of this oracle (its own numbering is kept equal to the library's
 * public header so a test can pass one integer to both; nothing is shared) */
#define ORACLE_F_RESELECT       1u   /* choose the kept set from |w_{t-1}| (Eq. 6)      */
#define ORACLE_F_COUNT_FLIPS    2u   /* add |mask_t xor mask_{t-1}| to *flip_count       */
#define ORACLE_F_META_BITMASK   4u   /* metadata = M-bit keep mask per group             */
#define ORACLE_F_V_KEPT_FROM_G  8u   /* alternate reading: kept entries feed g^2 into v  */
#define ORACLE_F_EMIT_DENSE    16u   /* forward weight is Diag(A) W without the mask     */
#define ORACLE_F_GRAD_OF_SCALED 64u  /* g is the gradient with respect to the scaled weight Diag(A~) W~ of
                                        Eq. 12; the chain rule gives dL/dW = A (.) g, and
                                        dL/dA[r, s] = sum over segment s of g[r, c] W_{t-1}[r, c]         */
#define ORACLE_F_EMIT_COMPRESSED 32u /* forward weight holds only the kept entries: rows x cols*N/M,
                                        the N kept values of each group in column order (the pruned
                                        matrix of Alg. 2's final loop without its zeros)               */

enum { ORACLE_OK = 0, ORACLE_BAD_ARGS = -1 };

static real real_sqrt(real x) { return (real)sqrt((double)x); } /* sqrt is correctly rounded, so
                                                                   rounding the fp64 root of an fp32
                                                                   value to fp32 equals sqrtf */

/* bf16 -> real: a bf16 is the upper half of an IEEE binary32 (exact). */
static real bf16_to_real(uint16_t h)
{
    uint32_t bits = (uint32_t)h << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (real)f;
}

/* real -> bf16, round to nearest, ties to even, written from the format's
 * definition: 1 sign bit, 8 exponent bits (bias 127), 7 fraction bits.  The
 * value is rounded to an integer multiple of the spacing 2^(e-7) of its binade
 * (e clamped at -126 for subnormals); nearbyint() rounds half to even in the
 * default rounding mode; the scalings by powers of two are exact. */
static uint16_t real_to_bf16_rne(real xr)
{
    double x = (double)xr;
    uint16_t sign = (uint16_t)(signbit(x) ? 0x8000u : 0u);
    double a = fabs(x);
    if (isnan(x)) return (uint16_t)(sign | 0x7FC0u);
    if (isinf(x)) return (uint16_t)(sign | 0x7F80u);
    if (a == 0.0) return sign;
    int e;
    (void)frexp(a, &e);            /* a = f * 2^e, f in [0.5, 1)  =>  floor(log2 a) = e - 1 */
    int binade = e - 1;
    if (binade < -126) binade = -126;
    double q = ldexp(1.0, binade - 7);          /* spacing of bf16 numbers in this binade  */
    double r = nearbyint(a / q) * q;            /* nearest multiple, ties to even           */
    if (r >= ldexp(1.0, 128)) return (uint16_t)(sign | 0x7F80u);   /* overflow -> inf      */
    float rf = (float)r;                        /* exact: r has at most 8 significant bits  */
    uint32_t bits;
    memcpy(&bits, &rf, sizeof bits);
    return (uint16_t)(sign | (uint16_t)(bits >> 16));
}

static int popcount32(uint32_t x)
{
    int c = 0;
    while (x) { c += (int)(x & 1u); x >>= 1; }
    return c;
}

/* Metadata field of group i of row r (M bits wide, packed LSB first into
 * row-major 32-bit words, cols/32 words per row; a word always describes 32
 * consecutive columns of one row).  The paper fixes only the size, one bit per
 * parameter (Remark in Sec. 4.1); the layout is defined here. */
static uint32_t meta_get_field(const uint32_t *meta, int64_t r, int64_t cols, int64_t i, int M)
{
    int64_t bit = i * M;
    uint32_t word = meta[r * (cols / 32) + bit / 32];
    uint32_t field_mask = (M == 32) ? 0xFFFFFFFFu : ((1u << M) - 1u);
    return (word >> (bit % 32)) & field_mask;
}

static void meta_set_field(uint32_t *meta, int64_t r, int64_t cols, int64_t i, int M, uint32_t field)
{
    int64_t bit = i * M;
    uint32_t *word = &meta[r * (cols / 32) + bit / 32];
    uint32_t field_mask = (M == 32) ? 0xFFFFFFFFu : ((1u << M) - 1u);
    *word = (*word & ~(field_mask << (bit % 32))) | ((field & field_mask) << (bit % 32));
}

/* keep mask (bit j set = column iM+j kept) <-> stored field */
static uint32_t field_from_keep(uint32_t keep, int bitmask_encoding)
{
    if (bitmask_encoding) return keep;
    /* 2:4 index form: positions of the two kept entries, lower one in bits 0-1 */
    int lo = -1, hi = -1;
    for (int j = 0; j < 4; ++j)
        if (keep & (1u << j)) { if (lo < 0) lo = j; else hi = j; }
    return (uint32_t)lo | ((uint32_t)hi << 2);
}

static uint32_t keep_from_field(uint32_t field, int bitmask_encoding)
{
    if (bitmask_encoding) return field;
    return (1u << (field & 3u)) | (1u << ((field >> 2) & 3u));
}

/*
 * One AdamS step over one row-major matrix W (rows x cols, cols = input
 * dimension).  w, m, v are updated in place.  g is bf16.  scale is A[rows][n_seg]
 * or NULL (all ones).  meta is read when the kept set is reused or flips are
 * counted, and always written.  step = t >= 1, total_steps = T >= t.
 */
int ENTRY(float *w, float *m, float *v, const uint16_t *g,
          uint16_t *w_fwd, uint32_t *meta,
          const float *scale, int n_seg,
          int64_t rows, int64_t cols, int N, int M,
          double lr_d, double beta1_d, double beta2_d, double eps_d, double l1_coeff_d,
          int64_t step, int64_t total_steps,
          uint32_t flags, uint64_t *flip_count,
          double *scale_grad,   /* [rows][n_seg], added to; may be NULL; used with ORACLE_F_GRAD_OF_SCALED */
          const float *scale_chain) /* [rows][n_seg]: the scale the forward pass that produced g was emitted with, where
                                       it differs from `scale` (which scales THIS step's emission); NULL = `scale`.
                                       Only the chain rule dL/dW = A (.) g of ORACLE_F_GRAD_OF_SCALED reads it. */
{
    if (!w || !m || !v || !g || !w_fwd || !meta) return ORACLE_BAD_ARGS;
    if (rows < 0 || cols < 0 || M < 1 || M > 32 || N < 1 || N > M) return ORACLE_BAD_ARGS;
    if (cols % M != 0 || cols % 32 != 0 || 32 % M != 0) return ORACLE_BAD_ARGS;
    if (step < 1 || total_steps < step) return ORACLE_BAD_ARGS;
    if (scale && (n_seg < 1 || cols % n_seg != 0 || (cols / n_seg) % M != 0)) return ORACLE_BAD_ARGS;
    const int bitmask_encoding = (flags & ORACLE_F_META_BITMASK) != 0;
    if (!bitmask_encoding && !(N == 2 && M == 4)) return ORACLE_BAD_ARGS;
    if ((flags & ORACLE_F_COUNT_FLIPS) && !flip_count) return ORACLE_BAD_ARGS;
    if ((flags & ORACLE_F_EMIT_COMPRESSED) && (flags & ORACLE_F_EMIT_DENSE)) return ORACLE_BAD_ARGS;
    if (scale_grad && !(flags & ORACLE_F_GRAD_OF_SCALED)) return ORACLE_BAD_ARGS;
    if (scale_chain && (!scale || !(flags & ORACLE_F_GRAD_OF_SCALED))) return ORACLE_BAD_ARGS;

    /* scalars of the step, formed in double and rounded once to the working type */
    const real alpha = (real)((double)step / (double)total_steps);   /* alpha_t = t/T   (Alg. 1) */
    const real bc1   = (real)(1.0 - pow(beta1_d, (double)step));     /* 1 - beta1^t               */
    const real bc2   = (real)(1.0 - pow(beta2_d, (double)step));     /* 1 - beta2^t               */
    const real lr = (real)lr_d, beta1 = (real)beta1_d, beta2 = (real)beta2_d;
    const real eps = (real)eps_d, lambda = (real)l1_coeff_d;
    const real one = (real)1;

    uint64_t flips = 0;

    for (int64_t r = 0; r < rows; ++r) {
        for (int64_t i = 0; i < cols / M; ++i) {               /* group g_r^(i), Eq. 3 */
            const int64_t base = r * cols + i * M;

            /* ---- kept set of the group (Eq. 6 with exactly N kept, Eq. 4) ---- */
            uint32_t keep = 0;
            if (flags & ORACLE_F_RESELECT) {
                for (int j = 0; j < M; ++j) {
                    /* rank of entry j = how many entries of the group come before it in the
                     * order "larger |w| first, lower column first among equals" */
                    float aj = fabsf(w[base + j]);
                    int rank = 0;
                    for (int k = 0; k < M; ++k) {
                        if (k == j) continue;
                        float ak = fabsf(w[base + k]);
                        if (ak > aj || (ak == aj && k < j)) ++rank;
                    }
                    if (rank < N) keep |= 1u << j;
                }
            } else {
                keep = keep_from_field(meta_get_field(meta, r, cols, i, M), bitmask_encoding);
            }

            if (flags & ORACLE_F_COUNT_FLIPS) {
                uint32_t prev = keep_from_field(meta_get_field(meta, r, cols, i, M), bitmask_encoding);
                flips += (uint64_t)popcount32(keep ^ prev);       /* ||M_t - M_{t-1}||_0, App. C */
            }

            int n_emitted = 0;      /* kept entries of this group written so far (compressed form) */
            for (int j = 0; j < M; ++j) {
                const int64_t idx = base + j;
                const int kept = (keep >> j) & 1u;
                const real theta_prev = (real)w[idx];
                real grad = bf16_to_real(g[idx]);
                if (flags & ORACLE_F_GRAD_OF_SCALED) {
                    /* W_scale[r, c] = A[r, s(c)] W[r, c]  (Eq. 12)  =>  dL/dA[r, s] += g W,  dL/dW = A g */
                    const int64_t col_g = i * M + j;
                    const int64_t seg = scale ? col_g / (cols / n_seg) : 0;
                    if (scale_grad) scale_grad[r * (scale ? n_seg : 1) + seg] += (double)grad * (double)w[idx];
                    if (scale) grad = (real)(scale_chain ? scale_chain : scale)[r * n_seg + seg] * grad;
                }

                /* first moment (Alg. 1: mu_t = beta1 mu_{t-1} + (1 - beta1) g_t); stored undecayed */
                const real mu = beta1 * (real)m[idx] + (one - beta1) * grad;
                m[idx] = (float)mu;

                /* proportional L1 decay on entries outside the kept set (Eq. 7) */
                real mu_tilde;
                if (!kept) {
                    real sgn = (real)((theta_prev > 0) - (theta_prev < 0));    /* Sign(0) = 0 */
                    mu_tilde = (one - alpha) * mu + alpha * lambda * sgn;
                } else {
                    mu_tilde = mu;
                }

                /* second moment from the decayed first moment (Eq. 8) */
                real second_src = mu_tilde;
                if ((flags & ORACLE_F_V_KEPT_FROM_G) && kept) second_src = grad;
                const real v_new = beta2 * (real)v[idx] + (one - beta2) * second_src * second_src;
                v[idx] = (float)v_new;

                /* bias correction and parameter update (Alg. 1, last three lines of the loop).
                 * The stored, rounded v is what the next step sees; this step uses v_new. */
                const real mu_hat = mu_tilde / bc1;
                const real v_hat = v_new / bc2;
                const real theta = theta_prev - lr * mu_hat / (real_sqrt(v_hat) + eps);
                w[idx] = (float)theta;

                /* forward weight: Diag(A~) W~ (Eq. 12), pruned by the mask (Alg. 2, final loop).
                 * The scale multiplies the stored (rounded) master weight. */
                const int64_t col = i * M + j;
                const real a = scale ? (real)scale[r * n_seg + col / (cols / n_seg)] : one;
                if (flags & ORACLE_F_EMIT_COMPRESSED) {
                    /* group i of row r owns slots (r * cols/M + i) * N ... + N - 1 */
                    if (kept && n_emitted < N) {
                        w_fwd[(r * (cols / M) + i) * N + n_emitted] = real_to_bf16_rne(a * (real)w[idx]);
                        ++n_emitted;
                    }
                } else if (kept || (flags & ORACLE_F_EMIT_DENSE))
                    w_fwd[idx] = real_to_bf16_rne(a * (real)w[idx]);
                else
                    w_fwd[idx] = 0;                                             /* +0.0 */
            }

            meta_set_field(meta, r, cols, i, M, field_from_keep(keep, bitmask_encoding));
        }
    }
    if (flags & ORACLE_F_COUNT_FLIPS) *flip_count += flips;
    return ORACLE_OK;
}
