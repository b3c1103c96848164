// cast_host_step_static: the AdamS N:M step for a matrix held in HOST memory, staged through a device
// area that is part of the library image instead of being allocated at run time.
//
// Who needs this.  cast_host_ctx_create reserves its staging slots with cudaMalloc.  Some callers
// cannot do that: a training process whose framework allocator has already taken all device memory
// (a further cudaMalloc fails or forces the pool to shrink), a step that runs where the implicit
// device-wide synchronisation of cudaMalloc / cudaFree is not acceptable, or a process that is simply
// not allowed to grow its device footprint after start-up.  For them the staging area below is a
// file-scope __device__ array: it belongs to the library image, every GPU on which the process uses
// it holds these ~16.6 MiB until the process exits, and this entry point calls no allocation or
// release routine of CUDA or of any other library.
//
// When the memory is actually taken.  The CUDA runtime loads a library's device code lazily by
// default: the image that holds the array is placed in device memory by the FIRST call of this
// entry point on a device (its cudaGetSymbolAddress), not when the shared library is opened.  That
// first call therefore needs ~16.6 MiB of free device memory and may synchronise the device: make
// it once per device at start-up, before a framework allocator takes the memory and outside any
// stream capture (or run the process with CUDA_MODULE_LOADING=EAGER, which moves the loading to
// context creation).  Every later call finds the address cached and touches no memory management.
//
// The array's name is only a host-side handle here: its device address is looked up once per device
// with cudaGetSymbolAddress (with that device current) and that address is what kernels and copies get.
#include <mutex>

#include "cast_internal.h"

namespace cast {
namespace {

constexpr int64_t kStaticMaxParams = CAST_STATIC_MAX_PARAMS;          // parameters per call
constexpr size_t kP = (size_t)kStaticMaxParams;
// fixed layout, sized for the maximum: w | m | v | g | w_fwd | meta | scale | flip counter
constexpr size_t kOffW = 0;
constexpr size_t kOffM = kOffW + 4 * kP;
constexpr size_t kOffV = kOffM + 4 * kP;
constexpr size_t kOffG = kOffV + 4 * kP;
constexpr size_t kOffFwd = kOffG + 2 * kP;
constexpr size_t kOffMeta = kOffFwd + 2 * kP;
constexpr size_t kOffScale = kOffMeta + kP / 8;          // at most rows * n <= P / 8 scale entries
constexpr size_t kOffFlips = kOffScale + 4 * (kP / 8);
constexpr size_t kStaticBytes = kOffFlips + 256;
static_assert(kOffM % 256 == 0 && kOffG % 256 == 0 && kOffMeta % 256 == 0 && kOffScale % 256 == 0 && kOffFlips % 256 == 0,
              "every part of the staging area starts on a 256-byte boundary");

static __device__ __align__(256) unsigned char g_static_stage[kStaticBytes];

std::mutex g_setup_mu;
unsigned char* g_stage_addr[64];          // device address of g_static_stage, per device (nullptr = not looked up)

// Device address of the staging area on the current device; looked up on the first call per device.
int stage_address(unsigned char** out)
{
    int dev = 0;
    CAST_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return CAST_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_setup_mu);
    if (g_stage_addr[dev] == nullptr) {
        void* p = nullptr;
        CAST_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_stage));
        if (p == nullptr) return CAST_ERR_CUDA;
        g_stage_addr[dev] = static_cast<unsigned char*>(p);
    }
    *out = g_stage_addr[dev];
    return CAST_OK;
}

}  // namespace
}  // namespace cast

using namespace cast;

extern "C" int cast_host_step_static(float* w, float* m, float* v, const cast_bf16* g,
                                     cast_bf16* w_fwd_bf16, uint32_t* meta,
                                     const float* scale, int scale_groups,
                                     int64_t rows, int64_t cols, int N, int M,
                                     float lr, float beta1, float beta2, float eps, float l1_coeff,
                                     int64_t step, int64_t total_steps,
                                     uint32_t flags, unsigned long long* flip_count,
                                     cast_stream_t stream)
{
    int rc;
    if ((rc = check_nm_flags(N, M, flags, flip_count)) != CAST_OK) return rc;
    if (flags & CAST_F_MASK_STATS) return CAST_ERR_PLAN;      // the statistics epilogue needs a plan
    StepConsts k;
    if ((rc = make_step_consts(lr, beta1, beta2, eps, l1_coeff, step, total_steps, N, flags, &k)) != CAST_OK) return rc;
    if (!w || !m || !v || !g || !w_fwd_bf16 || !meta) return CAST_ERR_NULL;
    if ((rc = check_shape(rows, cols, M, scale != nullptr, scale_groups)) != CAST_OK) return rc;
    if (rows * cols > kStaticMaxParams) return CAST_ERR_PLAN;          // larger than the built-in staging area
    const uint64_t fwd_total = fwd_elems_of(rows, cols, N, M, flags);
    if ((rc = check_pointers(w, m, v, g, w_fwd_bf16, meta, scale, scale_groups, rows, cols, fwd_total)) != CAST_OK) return rc;
    const void* host_ptrs[7] = {w, m, v, g, w_fwd_bf16, meta, scale};
    for (const void* p : host_ptrs) {
        if (!p) continue;
        cudaPointerAttributes attr;
        CAST_CUDA_TRY(cudaPointerGetAttributes(&attr, p));
        if (attr.type == cudaMemoryTypeDevice) return CAST_ERR_MEMORY;
    }

    unsigned char* base = nullptr;
    if ((rc = stage_address(&base)) != CAST_OK) return rc;
    float* d_w = reinterpret_cast<float*>(base + kOffW);
    float* d_m = reinterpret_cast<float*>(base + kOffM);
    float* d_v = reinterpret_cast<float*>(base + kOffV);
    uint16_t* d_g = reinterpret_cast<uint16_t*>(base + kOffG);
    uint16_t* d_fwd = reinterpret_cast<uint16_t*>(base + kOffFwd);
    uint32_t* d_meta = reinterpret_cast<uint32_t*>(base + kOffMeta);
    float* d_scale = reinterpret_cast<float*>(base + kOffScale);
    unsigned long long* d_flips = reinterpret_cast<unsigned long long*>(base + kOffFlips);

    cudaStream_t s = (cudaStream_t)stream;
    const size_t P = (size_t)rows * (size_t)cols;
    const bool count = (flags & CAST_F_COUNT_FLIPS) != 0;
    const bool need_prev = !(flags & CAST_F_RESELECT) || count;
    unsigned long long flips = 0;
    // Everything is queued by this lambda; whatever it returns, the stream is drained before the call returns, so that
    // no copy into or out of the caller's host buffers is still in flight when the caller gets control back.
    auto queue_all = [&]() -> int {
        CAST_CUDA_TRY(cudaMemcpyAsync(d_w, w, 4 * P, cudaMemcpyHostToDevice, s));
        CAST_CUDA_TRY(cudaMemcpyAsync(d_m, m, 4 * P, cudaMemcpyHostToDevice, s));
        CAST_CUDA_TRY(cudaMemcpyAsync(d_v, v, 4 * P, cudaMemcpyHostToDevice, s));
        CAST_CUDA_TRY(cudaMemcpyAsync(d_g, g, 2 * P, cudaMemcpyHostToDevice, s));
        if (need_prev) CAST_CUDA_TRY(cudaMemcpyAsync(d_meta, meta, P / 8, cudaMemcpyHostToDevice, s));
        if (scale)
            CAST_CUDA_TRY(cudaMemcpyAsync(d_scale, scale, 4 * (size_t)rows * (size_t)scale_groups, cudaMemcpyHostToDevice, s));
        // the area keeps whatever the previous call left: the counter is the one part that must start at zero
        if (count) CAST_CUDA_TRY(cudaMemsetAsync(d_flips, 0, sizeof(unsigned long long), s));
        const TensorDesc d = make_desc(d_w, d_m, d_v, d_g, d_fwd, d_meta, scale ? d_scale : nullptr, scale_groups, rows, cols);
        const int launch_rc = launch_single(d, M, k, count ? d_flips : nullptr, s);
        if (launch_rc != CAST_OK) return launch_rc;
        CAST_CUDA_TRY(cudaMemcpyAsync(w, d_w, 4 * P, cudaMemcpyDeviceToHost, s));
        CAST_CUDA_TRY(cudaMemcpyAsync(m, d_m, 4 * P, cudaMemcpyDeviceToHost, s));
        CAST_CUDA_TRY(cudaMemcpyAsync(v, d_v, 4 * P, cudaMemcpyDeviceToHost, s));
        CAST_CUDA_TRY(cudaMemcpyAsync(w_fwd_bf16, d_fwd, 2 * (size_t)fwd_total, cudaMemcpyDeviceToHost, s));
        CAST_CUDA_TRY(cudaMemcpyAsync(meta, d_meta, P / 8, cudaMemcpyDeviceToHost, s));
        if (count) CAST_CUDA_TRY(cudaMemcpyAsync(&flips, d_flips, sizeof flips, cudaMemcpyDeviceToHost, s));
        return CAST_OK;
    };
    rc = queue_all();
    const cudaError_t drained = cudaStreamSynchronize(s);
    if (rc != CAST_OK) return rc;             // the host buffers may hold a partly updated state: see the header
    if (drained != cudaSuccess) return cuda_failed(drained);
    if (count) *flip_count += flips;
    return CAST_OK;
}
