// Plain Adam step on the scale matrix A of Eq. 12 (the paper learns A jointly with the weights, Sec. 4.2, and
// does not name its optimizer; the reading taken is Alg. 1 without its mask and decay lines).  A has
// rows * n entries (n = 2 in the paper's experiments), thousands of times fewer than the weights: the kernel
// is latency-sized, one thread per entry, arithmetic in fp64.
#include <cmath>
#include <cstring>

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

// All scale matrices of a plan in one grid (each is a few thousand entries: one launch per matrix would be
// hundreds of launches of a microsecond each).  Tables in kernel parameter space, like the step's.
constexpr int kScaleTile = 256;
struct ScaleDesc { float* a; float* m; float* v; float* grad; float* keep_old; uint32_t n; uint32_t pad_; };   // keep_old: receives a before the update, or nullptr
struct ScaleParams {
    uint32_t n_tensors;
    uint32_t hint_shift;
    uint16_t hint[kHintEntries];
    uint32_t tile_start[kMaxLaunchTensors + 1];
    ScaleDesc desc[kMaxLaunchTensors];
};

__global__ void __launch_bounds__(kScaleTile)
scale_adam_multi_kernel(const __grid_constant__ ScaleParams p, double lr_bc1, double beta1, double beta2, double inv_bc2,
                        double eps, int clear_grad)
{
    const uint32_t tile = blockIdx.x;
    uint32_t k = p.hint[tile >> p.hint_shift];
    while (tile >= p.tile_start[k + 1]) ++k;
    const ScaleDesc& t = p.desc[k];
    const uint32_t i = (tile - p.tile_start[k]) * kScaleTile + threadIdx.x;
    if (i >= t.n) return;
    const double g = (double)t.grad[i];
    if (t.keep_old != nullptr) t.keep_old[i] = t.a[i];      // the scale the last emission used: the next step's chain-rule factor
    const double mu = beta1 * (double)t.m[i] + (1.0 - beta1) * g;
    const double nu = beta2 * (double)t.v[i] + (1.0 - beta2) * g * g;
    t.m[i] = (float)mu;
    t.v[i] = (float)nu;
    t.a[i] = (float)((double)t.a[i] - lr_bc1 * mu / (sqrt(nu * inv_bc2) + eps));
    if (clear_grad) t.grad[i] = 0.0f;
}

int check_adam_hyper(float lr, float beta1, float beta2, float eps, int64_t step)
{
    if (!std::isfinite(lr) || !(beta1 >= 0.0f && beta1 < 1.0f) || !(beta2 >= 0.0f && beta2 < 1.0f)) return CAST_ERR_HYPER;
    if (!(eps > 0.0f) || !std::isfinite(eps) || step < 1) return CAST_ERR_HYPER;
    return CAST_OK;
}

}  // namespace
}  // namespace cast

using namespace cast;

extern "C" int cast_plan_scale_adam_step(void* plan, float* const* m_a, float* const* v_a,
                                         float lr, float beta1, float beta2, float eps, int64_t step,
                                         int clear_grad, cast_stream_t stream)
{
    const int n = plan_tensor_count(plan);
    if (n < 0) return CAST_ERR_PLAN;
    if (!m_a || !v_a) return CAST_ERR_NULL;
    int rc;
    if ((rc = check_adam_hyper(lr, beta1, beta2, eps, step)) != CAST_OK) return rc;
    int N = 0, M = 0;
    TensorDesc d;
    for (int i = 0; i < n; ++i) {
        plan_tensor_desc(plan, i, &N, &M, &d);
        if (!d.scale || !d.scale_grad || !m_a[i] || !v_a[i]) return CAST_ERR_NULL;      // every matrix needs a scale and its gradient
        if (((uintptr_t)m_a[i] & 3u) || ((uintptr_t)v_a[i] & 3u)) return CAST_ERR_ALIGN;
        const void* ptrs[2] = {m_a[i], v_a[i]};
        if ((rc = check_device_memory(ptrs, 2)) != CAST_OK) return rc;
    }
    const double bc1 = 1.0 - std::pow((double)beta1, (double)step);
    const double bc2 = 1.0 - std::pow((double)beta2, (double)step);
    int i = 0;
    while (i < n) {
        ScaleParams p;
        std::memset(&p, 0, sizeof p);
        uint64_t tiles = 0;
        while (i < n && p.n_tensors < (uint32_t)kMaxLaunchTensors) {
            plan_tensor_desc(plan, i, &N, &M, &d);
            // entries of A: rows * n = units / (units per segment); recovered from the descriptor's segment divisor
            const uint32_t n_entries = (uint32_t)(((uint64_t)(d.n_units - 1) * d.seg_magic) >> d.seg_shift) + 1;
            // a descriptor without a second scale names `scale` itself there: nothing to keep
            p.desc[p.n_tensors] = ScaleDesc{const_cast<float*>(d.scale), m_a[i], v_a[i], d.scale_grad,
                                            d.scale_chain != d.scale ? const_cast<float*>(d.scale_chain) : nullptr, n_entries, 0};
            p.tile_start[p.n_tensors] = (uint32_t)tiles;
            tiles += (n_entries + kScaleTile - 1) / kScaleTile;
            ++p.n_tensors;
            ++i;
        }
        p.tile_start[p.n_tensors] = (uint32_t)tiles;
        fill_hint_table(p.n_tensors, p.tile_start, p.hint, &p.hint_shift);
        scale_adam_multi_kernel<<<(unsigned)tiles, kScaleTile, 0, (cudaStream_t)stream>>>(p, (double)lr / bc1, (double)beta1, (double)beta2,
                                                                                          1.0 / bc2, (double)eps, clear_grad);
        CAST_CUDA_TRY(cudaGetLastError());
        count_launch();
    }
    return CAST_OK;
}

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
