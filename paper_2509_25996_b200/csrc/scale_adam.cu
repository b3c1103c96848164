// Plain Adam step on the scale matrix A of Eq. 12 (the paper learns A jointly with the weights, Sec. 4.2, and
// does not name its optimizer; the reading taken is Alg. 1 without its mask and decay lines).  A has
// rows * n entries (n = 2 in the paper's experiments), thousands of times fewer than the weights: the kernel
// is latency-sized, one thread per entry, arithmetic in fp64.
#include <cmath>

#include "cast_internal.h"

namespace cast {
namespace {

__global__ void scale_adam_kernel(float* __restrict__ a, float* __restrict__ m, float* __restrict__ v, float* __restrict__ grad,
                                  long long n, double lr_bc1, double beta1, double beta2, double inv_bc2, double eps, int clear_grad)
{
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const double g = (double)grad[i];
    const double mu = beta1 * (double)m[i] + (1.0 - beta1) * g;
    const double nu = beta2 * (double)v[i] + (1.0 - beta2) * g * g;
    m[i] = (float)mu;
    v[i] = (float)nu;
    a[i] = (float)((double)a[i] - lr_bc1 * mu / (sqrt(nu * inv_bc2) + eps));
    if (clear_grad) grad[i] = 0.0f;
}

}  // namespace
}  // namespace cast

using namespace cast;

extern "C" int cast_scale_adam_step(float* a, float* m_a, float* v_a, float* grad, int64_t n,
                                    float lr, float beta1, float beta2, float eps, int64_t step,
                                    int clear_grad, cast_stream_t stream)
{
    if (!a || !m_a || !v_a || !grad) return CAST_ERR_NULL;
    if (n < 1 || n > 0x7FFFFFFF) return CAST_ERR_SHAPE;
    if (!std::isfinite(lr) || !(beta1 >= 0.0f && beta1 < 1.0f) || !(beta2 >= 0.0f && beta2 < 1.0f)) return CAST_ERR_HYPER;
    if (!(eps > 0.0f) || !std::isfinite(eps) || step < 1) return CAST_ERR_HYPER;
    const void* ptrs[4] = {a, m_a, v_a, grad};
    for (const void* p : ptrs)
        if ((uintptr_t)p & 3u) return CAST_ERR_ALIGN;
    for (int i = 0; i < 4; ++i)
        for (int j = i + 1; j < 4; ++j) {
            const uintptr_t x = (uintptr_t)ptrs[i], y = (uintptr_t)ptrs[j];
            if (x < y + 4ull * (uint64_t)n && y < x + 4ull * (uint64_t)n) return CAST_ERR_ALIAS;
        }
    int rc;
    if ((rc = check_device_memory(ptrs, 4)) != CAST_OK) return rc;
    const double bc1 = 1.0 - std::pow((double)beta1, (double)step);
    const double bc2 = 1.0 - std::pow((double)beta2, (double)step);
    const int threads = 256;
    const unsigned blocks = (unsigned)((n + threads - 1) / threads);
    scale_adam_kernel<<<blocks, threads, 0, (cudaStream_t)stream>>>(a, m_a, v_a, grad, (long long)n, (double)lr / bc1, (double)beta1,
                                                                    (double)beta2, 1.0 / bc2, (double)eps, clear_grad);
    CAST_CUDA_TRY(cudaGetLastError());
    count_launch();
    return CAST_OK;
}
