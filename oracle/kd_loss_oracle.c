/*
 * CPU oracle for the training loss of CAST (arxiv 2509.25996, Sec. 4.3, Eq. 13), per token:
 *
 *     L = eta * D_KL(P_t || P_s) + (1 - eta) * L_ce ,     D_KL(P_t || P_s) = sum_x P_t(x) log(P_t(x) / P_s(x)),
 *
 * with P_s = softmax(student logits), P_t = softmax(teacher logits), L_ce = -log P_s(label), and its
 * gradient with respect to the student logits,
 *
 *     dL/ds_x = grad_scale * ( P_s(x) - eta P_t(x) - (1 - eta) [x == label] )
 *
 * (from d D_KL / d s = P_s - P_t and d L_ce / d s = P_s - onehot).  A negative label means "no target": the
 * cross-entropy term and its gradient are left out for that token (the paper does not discuss padding; this is
 * the usual convention).  The paper does not say how tokens are reduced: the per-token losses are returned and
 * grad_scale carries whatever reduction the caller uses (1/tokens for a mean).
 *
 * THIS FILE IS TEST INFRASTRUCTURE: a plain serial loop in fp64 written from the definitions (max-shifted
 * softmax, nothing fused), shared with nothing in the CUDA library.
 * Pins (tests/test_oracle_pins.py): torch's kl_div / cross_entropy / autograd in fp64; closed forms (equal
 * logits give D_KL = 0; uniform student gives L_ce = log V).
 *
 * Logits are bf16 (upper half of an IEEE binary32), row-major [tokens][vocab].
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

static double kd_bf16(uint16_t h)
{
    uint32_t bits = (uint32_t)h << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

/* loss[tokens]; grad (may be NULL) [tokens][vocab] in fp64, unrounded */
int oracle_kd_loss(const uint16_t *student, const uint16_t *teacher, const int32_t *labels,
                   int64_t tokens, int64_t vocab, double eta, double grad_scale,
                   double *loss, double *grad)
{
    if (!student || !teacher || !labels || !loss || tokens < 0 || vocab < 1) return -1;
    for (int64_t t = 0; t < tokens; ++t) {
        const uint16_t *s = student + t * vocab, *q = teacher + t * vocab;
        const int64_t y = labels[t];
        if (y >= vocab) return -1;
        double ms = -INFINITY, mq = -INFINITY;
        for (int64_t x = 0; x < vocab; ++x) {
            if (kd_bf16(s[x]) > ms) ms = kd_bf16(s[x]);
            if (kd_bf16(q[x]) > mq) mq = kd_bf16(q[x]);
        }
        double zs = 0.0, zq = 0.0;
        for (int64_t x = 0; x < vocab; ++x) {
            zs += exp(kd_bf16(s[x]) - ms);
            zq += exp(kd_bf16(q[x]) - mq);
        }
        const double log_zs = log(zs), log_zq = log(zq);
        double kl = 0.0;
        for (int64_t x = 0; x < vocab; ++x) {
            const double log_ps = kd_bf16(s[x]) - ms - log_zs;       /* log P_s(x) */
            const double log_pt = kd_bf16(q[x]) - mq - log_zq;       /* log P_t(x) */
            const double pt = exp(log_pt);
            if (pt > 0.0) kl += pt * (log_pt - log_ps);              /* P_t log(P_t / P_s) */
            if (grad) {
                double g = exp(log_ps) - eta * pt;
                if (y >= 0) g -= (1.0 - eta) * (x == y ? 1.0 : 0.0);
                else g -= (1.0 - eta) * exp(log_ps);                 /* no target: the CE share of P_s drops out too */
                grad[t * vocab + x] = grad_scale * g;
            }
        }
        double ce = 0.0;
        if (y >= 0) ce = -(kd_bf16(s[y]) - ms - log_zs);             /* -log P_s(label) */
        loss[t] = eta * kl + (1.0 - eta) * ce;
    }
    return 0;
}
