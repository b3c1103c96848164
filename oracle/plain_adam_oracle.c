/*
 * CPU oracle for the plain Adam step that trains the scale matrix A of CAST's weight scaling (Sec. 4.2: A is
 * "learned jointly"; the paper does not say with which optimizer -- the reading taken is Adam with bias
 * correction, no decay and no mask, i.e. Alg. 1 without its sparsity-specific lines).
 *
 * THIS FILE IS TEST INFRASTRUCTURE: a serial fp64 loop, shared with nothing in the CUDA library.
 * Pin (tests/test_oracle_pins.py): torch.optim.Adam over several steps.
 */
#include <math.h>
#include <stdint.h>

int oracle_plain_adam(float *theta, float *m, float *v, const float *grad, int64_t n,
                      double lr, double beta1, double beta2, double eps, int64_t step)
{
    if (!theta || !m || !v || !grad || n < 0 || step < 1) return -1;
    const double bc1 = 1.0 - pow(beta1, (double)step);
    const double bc2 = 1.0 - pow(beta2, (double)step);
    for (int64_t i = 0; i < n; ++i) {
        const double g = (double)grad[i];
        const double mu = beta1 * (double)m[i] + (1.0 - beta1) * g;
        const double nu = beta2 * (double)v[i] + (1.0 - beta2) * g * g;
        m[i] = (float)mu;
        v[i] = (float)nu;
        theta[i] = (float)((double)theta[i] - lr * (mu / bc1) / (sqrt(nu / bc2) + eps));
    }
    return 0;
}
