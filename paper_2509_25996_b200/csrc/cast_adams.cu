// Entry points of the AdamS N:M library: argument checks, per-iteration scalars, launches, plans.
// Everything that can be wrong is detected on the host before a launch; no device-side waits exist.
#include <atomic>
#include <cmath>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "cast_internal.h"

namespace cast {

static thread_local int g_last_cuda_error = 0;
static std::atomic<unsigned long long> g_launches{0};

int cuda_failed(cudaError_t e)
{
    g_last_cuda_error = (int)e;
    (void)cudaGetLastError();   // clear the sticky-free error state of the runtime
    return CAST_ERR_CUDA;
}

int check_nm_flags(int N, int M, uint32_t flags, const void* flip_count)
{
    if (!(M == 2 || M == 4 || M == 8 || M == 16 || M == 32)) return CAST_ERR_NM;
    if (N < 1 || N > M) return CAST_ERR_NM;
    if (!(flags & CAST_F_META_BITMASK) && !(N == 2 && M == 4)) return CAST_ERR_NM;
    const uint32_t known = CAST_F_RESELECT | CAST_F_COUNT_FLIPS | CAST_F_META_BITMASK |
                           CAST_F_V_KEPT_FROM_G | CAST_F_EMIT_DENSE;
    if (flags & ~known) return CAST_ERR_HYPER;
    if ((flags & CAST_F_COUNT_FLIPS) && flip_count == nullptr) return CAST_ERR_NULL;
    return CAST_OK;
}

int make_step_consts(float lr, float beta1, float beta2, float eps, float l1_coeff,
                     int64_t step, int64_t total_steps, int N, uint32_t flags, StepConsts* out)
{
    if (!std::isfinite(lr) || !std::isfinite(l1_coeff)) return CAST_ERR_HYPER;
    if (!(beta1 >= 0.0f && beta1 < 1.0f) || !(beta2 >= 0.0f && beta2 < 1.0f)) return CAST_ERR_HYPER;
    if (!(eps > 0.0f) || !std::isfinite(eps)) return CAST_ERR_HYPER;
    if (step < 1 || total_steps < step) return CAST_ERR_HYPER;
    // Folded in double, rounded once: alpha_t = t/T (Alg. 1), 1 - beta^t (bias corrections).
    const double alpha = (double)step / (double)total_steps;
    const double bc1 = 1.0 - std::pow((double)beta1, (double)step);
    const double bc2 = 1.0 - std::pow((double)beta2, (double)step);
    StepConsts c;
    c.beta1 = (double)beta1;
    c.omb1 = 1.0 - (double)beta1;
    c.c_mu = 1.0 - alpha;
    c.c_sign = alpha * (double)l1_coeff;
    c.beta2 = beta2;
    c.omb2 = (float)(1.0 - (double)beta2);
    c.inv_bc2 = (float)(1.0 / bc2);
    c.lr_bc1 = (float)((double)lr / bc1);
    c.eps = eps;
    c.n_keep = N;
    c.flags = flags;
    *out = c;
    return CAST_OK;
}

int check_shape(int64_t rows, int64_t cols, int M, bool has_scale, int scale_groups)
{
    if (rows < 1 || cols < 1) return CAST_ERR_SHAPE;
    if (cols % 32 != 0 || cols % M != 0) return CAST_ERR_SHAPE;
    if (rows > (int64_t)0x7FFFFFFF / cols) return CAST_ERR_SHAPE;          // rows*cols < 2^31
    if (has_scale) {
        if (scale_groups < 1 || cols % scale_groups != 0) return CAST_ERR_SHAPE;
        const int64_t seg = cols / scale_groups;
        const int64_t q = M > kUnitElems ? M : kUnitElems;
        if (seg % q != 0) return CAST_ERR_SHAPE;     // no group and no 8-column unit straddles a segment
    }
    return CAST_OK;
}

namespace {
struct Range { uintptr_t lo, hi; };
inline bool overlap(const Range& a, const Range& b) { return a.lo < b.hi && b.lo < a.hi; }
}  // namespace

int check_pointers(const void* w, const void* m, const void* v, const void* g, const void* w_fwd,
                   const void* meta, const void* scale, int scale_groups, int64_t rows, int64_t cols)
{
    if (!w || !m || !v || !g || !w_fwd || !meta) return CAST_ERR_NULL;
    const void* all[7] = {w, m, v, g, w_fwd, meta, scale};
    for (const void* p : all)
        if (p && ((uintptr_t)p & 15u)) return CAST_ERR_ALIGN;
    const uint64_t P = (uint64_t)rows * (uint64_t)cols;
    Range r[7] = {
        {(uintptr_t)w, (uintptr_t)w + 4 * P},         {(uintptr_t)m, (uintptr_t)m + 4 * P},
        {(uintptr_t)v, (uintptr_t)v + 4 * P},         {(uintptr_t)g, (uintptr_t)g + 2 * P},
        {(uintptr_t)w_fwd, (uintptr_t)w_fwd + 2 * P}, {(uintptr_t)meta, (uintptr_t)meta + P / 8},
        {(uintptr_t)scale, (uintptr_t)scale + (scale ? 4ull * (uint64_t)rows * (uint64_t)scale_groups : 0)}};
    const int n = scale ? 7 : 6;
    for (int i = 0; i < n; ++i)
        for (int j = i + 1; j < n; ++j)
            if (overlap(r[i], r[j])) return CAST_ERR_ALIAS;
    return CAST_OK;
}

int check_device_memory(const void* const* ptrs, int n)
{
    for (int i = 0; i < n; ++i) {
        if (!ptrs[i]) continue;
        cudaPointerAttributes attr;
        CAST_CUDA_TRY(cudaPointerGetAttributes(&attr, ptrs[i]));
        if (attr.type != cudaMemoryTypeDevice && attr.type != cudaMemoryTypeManaged) return CAST_ERR_MEMORY;
    }
    return CAST_OK;
}

// unit / d for every unit < 2^31 as (uint64(unit) * magic) >> shift:
// with l = ceil(log2 d), shift = 31 + l and magic = floor(2^shift / d) + 1 (which fits 32 bits),
// unit * magic / 2^shift exceeds unit / d by less than 1/d while unit < 2^31, so the floors agree.
static void fast_div(uint32_t d, uint32_t* magic, uint32_t* shift)
{
    uint32_t l = 0;
    while ((1ull << l) < d) ++l;
    *shift = 31 + l;
    *magic = (uint32_t)(((1ull << (31 + l)) / d) + 1ull);
}

TensorDesc make_desc(float* w, float* m, float* v, const uint16_t* g, uint16_t* w_fwd, uint32_t* meta,
                     const float* scale, int scale_groups, int64_t rows, int64_t cols)
{
    TensorDesc d;
    std::memset(&d, 0, sizeof d);
    d.w = w; d.m = m; d.v = v; d.g = g; d.w_fwd = w_fwd; d.meta = meta; d.scale = scale;
    d.n_units = (uint32_t)((uint64_t)rows * (uint64_t)cols / kUnitElems);
    if (scale) {
        const uint32_t seg_units = (uint32_t)(cols / scale_groups / kUnitElems);
        fast_div(seg_units, &d.seg_magic, &d.seg_shift);
    }
    return d;
}

// ---------------------------------------------------------------------------------------------
// launches

namespace {

struct DeviceInfo { int sm_count = 0; };
std::mutex g_mu;
DeviceInfo g_dev[64];
int g_blocks_per_sm[64][6][2];   // [device][log2 M][multi], 0 = unknown

int device_info(int* dev_out, DeviceInfo* info)
{
    int dev = 0;
    CAST_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return CAST_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mu);
    if (g_dev[dev].sm_count == 0) {
        int sms = 0;
        CAST_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        g_dev[dev].sm_count = sms;
    }
    *dev_out = dev;
    *info = g_dev[dev];
    return CAST_OK;
}

template <int M, bool MULTI>
int launch_t(const TensorDesc& single, const TensorDesc* descs, const uint32_t* tile_start,
             uint32_t total_tiles, const StepConsts& c, unsigned long long* flip_count, cudaStream_t stream,
             int log2m)
{
    if (total_tiles == 0) return CAST_OK;
    int dev = 0;
    DeviceInfo info;
    int rc = device_info(&dev, &info);
    if (rc != CAST_OK) return rc;
    int per_sm;
    {
        std::lock_guard<std::mutex> lock(g_mu);
        per_sm = g_blocks_per_sm[dev][log2m][MULTI ? 1 : 0];
    }
    if (per_sm == 0) {
        CAST_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, adams_nm_kernel<M, MULTI>, kThreads, 0));
        if (per_sm < 1) per_sm = 1;
        std::lock_guard<std::mutex> lock(g_mu);
        g_blocks_per_sm[dev][log2m][MULTI ? 1 : 0] = per_sm;
    }
    // persistent grid: a whole number of CTAs per SM
    uint64_t grid = (uint64_t)info.sm_count * (uint64_t)per_sm;
    if (grid > total_tiles) grid = total_tiles;
    adams_nm_kernel<M, MULTI><<<(unsigned)grid, kThreads, 0, stream>>>(single, descs, tile_start, total_tiles, c, flip_count);
    CAST_CUDA_TRY(cudaGetLastError());
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return CAST_OK;
}

template <bool MULTI>
int launch_m(int M, const TensorDesc& single, const TensorDesc* descs, const uint32_t* tile_start,
             uint32_t total_tiles, const StepConsts& c, unsigned long long* flip_count, cudaStream_t stream)
{
    switch (M) {
        case 2:  return launch_t<2, MULTI>(single, descs, tile_start, total_tiles, c, flip_count, stream, 1);
        case 4:  return launch_t<4, MULTI>(single, descs, tile_start, total_tiles, c, flip_count, stream, 2);
        case 8:  return launch_t<8, MULTI>(single, descs, tile_start, total_tiles, c, flip_count, stream, 3);
        case 16: return launch_t<16, MULTI>(single, descs, tile_start, total_tiles, c, flip_count, stream, 4);
        case 32: return launch_t<32, MULTI>(single, descs, tile_start, total_tiles, c, flip_count, stream, 5);
    }
    return CAST_ERR_NM;
}

}  // namespace

int launch_single(const TensorDesc& d, int M, const StepConsts& c, unsigned long long* flip_count, cudaStream_t stream)
{
    return launch_m<false>(M, d, nullptr, nullptr, tiles_of(d), c, flip_count, stream);
}

int launch_multi(const TensorDesc* d_descs, const uint32_t* d_tile_start, uint32_t total_tiles, int M,
                 const StepConsts& c, unsigned long long* flip_count, cudaStream_t stream)
{
    TensorDesc none;
    std::memset(&none, 0, sizeof none);
    return launch_m<true>(M, none, d_descs, d_tile_start, total_tiles, c, flip_count, stream);
}

// ---------------------------------------------------------------------------------------------
// plans

namespace {
constexpr uint64_t kPlanMagic = 0x43415354504C414Eull;   // "CASTPLAN"
struct Plan {
    uint64_t magic;
    int device;
    int N, M;
    int n_tensors;
    uint32_t total_tiles;
    void* d_table;                // [n_tensors] TensorDesc, then [n_tensors + 1] uint32 tile starts
    const TensorDesc* d_descs;
    const uint32_t* d_tile_start;
};
}  // namespace

}  // namespace cast

using namespace cast;

extern "C" int cast_adams_step(float* w, float* m, float* v, const cast_bf16* g,
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
    StepConsts c;
    if ((rc = make_step_consts(lr, beta1, beta2, eps, l1_coeff, step, total_steps, N, flags, &c)) != CAST_OK) return rc;
    if (!w || !m || !v || !g || !w_fwd_bf16 || !meta) return CAST_ERR_NULL;
    if ((rc = check_shape(rows, cols, M, scale != nullptr, scale_groups)) != CAST_OK) return rc;
    if ((rc = check_pointers(w, m, v, g, w_fwd_bf16, meta, scale, scale_groups, rows, cols)) != CAST_OK) return rc;
    const void* ptrs[8] = {w, m, v, g, w_fwd_bf16, meta, scale, (flags & CAST_F_COUNT_FLIPS) ? flip_count : nullptr};
    if ((rc = check_device_memory(ptrs, 8)) != CAST_OK) return rc;
    const TensorDesc d = make_desc(w, m, v, g, w_fwd_bf16, meta, scale, scale_groups, rows, cols);
    return launch_single(d, M, c, flip_count, (cudaStream_t)stream);
}

extern "C" int cast_plan_create(const cast_tensor_t* tensors, int n_tensors, int N, int M, void** plan_out)
{
    if (!plan_out) return CAST_ERR_NULL;
    *plan_out = nullptr;
    if (!tensors) return CAST_ERR_NULL;
    if (n_tensors < 1) return CAST_ERR_SHAPE;
    int rc;
    // the encoding flag is a per-step choice; here only N:M itself is checked
    if ((rc = check_nm_flags(N, M, CAST_F_META_BITMASK, nullptr)) != CAST_OK) return rc;

    std::vector<TensorDesc> descs((size_t)n_tensors);
    std::vector<uint32_t> tile_start((size_t)n_tensors + 1);
    uint64_t tiles = 0;
    for (int i = 0; i < n_tensors; ++i) {
        const cast_tensor_t& t = tensors[i];
        if (!t.w || !t.m || !t.v || !t.g || !t.w_fwd || !t.meta) return CAST_ERR_NULL;
        if ((rc = check_shape(t.rows, t.cols, M, t.scale != nullptr, t.scale_groups)) != CAST_OK) return rc;
        if ((rc = check_pointers(t.w, t.m, t.v, t.g, t.w_fwd, t.meta, t.scale, t.scale_groups, t.rows, t.cols)) != CAST_OK) return rc;
        descs[(size_t)i] = make_desc(t.w, t.m, t.v, t.g, t.w_fwd, t.meta, t.scale, t.scale_groups, t.rows, t.cols);
        tile_start[(size_t)i] = (uint32_t)tiles;
        tiles += tiles_of(descs[(size_t)i]);
        if (tiles >= 0xFFFFFFFFull) return CAST_ERR_SHAPE;
    }
    tile_start[(size_t)n_tensors] = (uint32_t)tiles;
    for (int i = 0; i < n_tensors; ++i) {
        const cast_tensor_t& t = tensors[i];
        const void* ptrs[7] = {t.w, t.m, t.v, t.g, t.w_fwd, t.meta, t.scale};
        if ((rc = check_device_memory(ptrs, 7)) != CAST_OK) return rc;
    }

    Plan* p = new (std::nothrow) Plan;
    if (!p) return CAST_ERR_PLAN;
    std::memset(p, 0, sizeof *p);
    cudaError_t e = cudaGetDevice(&p->device);
    if (e != cudaSuccess) { delete p; return cuda_failed(e); }
    const size_t desc_bytes = sizeof(TensorDesc) * (size_t)n_tensors;
    const size_t start_bytes = sizeof(uint32_t) * ((size_t)n_tensors + 1);
    e = cudaMalloc(&p->d_table, desc_bytes + start_bytes);
    if (e != cudaSuccess) { delete p; return cuda_failed(e); }
    e = cudaMemcpy(p->d_table, descs.data(), desc_bytes, cudaMemcpyHostToDevice);
    if (e == cudaSuccess)
        e = cudaMemcpy((char*)p->d_table + desc_bytes, tile_start.data(), start_bytes, cudaMemcpyHostToDevice);
    if (e != cudaSuccess) { cudaFree(p->d_table); delete p; return cuda_failed(e); }
    p->magic = kPlanMagic;
    p->N = N; p->M = M; p->n_tensors = n_tensors;
    p->total_tiles = (uint32_t)tiles;
    p->d_descs = (const TensorDesc*)p->d_table;
    p->d_tile_start = (const uint32_t*)((char*)p->d_table + desc_bytes);
    *plan_out = p;
    return CAST_OK;
}

extern "C" int cast_plan_step(void* plan, const cast_hyper_t* h, unsigned long long* flip_count, cast_stream_t stream)
{
    Plan* p = (Plan*)plan;
    if (!p || p->magic != kPlanMagic) return CAST_ERR_PLAN;
    if (!h) return CAST_ERR_NULL;
    int rc;
    if ((rc = check_nm_flags(p->N, p->M, h->flags, flip_count)) != CAST_OK) return rc;
    StepConsts c;
    if ((rc = make_step_consts(h->lr, h->beta1, h->beta2, h->eps, h->l1_coeff, h->step, h->total_steps,
                               p->N, h->flags, &c)) != CAST_OK) return rc;
    int dev = -1;
    CAST_CUDA_TRY(cudaGetDevice(&dev));
    if (dev != p->device) return CAST_ERR_PLAN;
    if (h->flags & CAST_F_COUNT_FLIPS) {
        const void* fp[1] = {flip_count};
        if ((rc = check_device_memory(fp, 1)) != CAST_OK) return rc;
    }
    return launch_multi(p->d_descs, p->d_tile_start, p->total_tiles, p->M, c, flip_count, (cudaStream_t)stream);
}

extern "C" int cast_plan_destroy(void* plan)
{
    Plan* p = (Plan*)plan;
    if (!p || p->magic != kPlanMagic) return CAST_ERR_PLAN;
    p->magic = 0;
    cudaError_t e = cudaFree(p->d_table);
    delete p;
    if (e != cudaSuccess) return cuda_failed(e);
    return CAST_OK;
}

extern "C" const char* cast_strerror(int status)
{
    switch (status) {
        case CAST_OK:         return "ok";
        case CAST_ERR_NULL:   return "a required pointer is NULL";
        case CAST_ERR_SHAPE:  return "shape rule violated (cols % 32, cols % M, rows*cols < 2^31, scale segments)";
        case CAST_ERR_ALIGN:  return "a pointer is not 16-byte aligned";
        case CAST_ERR_NM:     return "unsupported N:M or metadata form";
        case CAST_ERR_HYPER:  return "hyper-parameter or flag out of range";
        case CAST_ERR_CUDA:   return "a CUDA runtime call failed (see cast_last_cuda_error)";
        case CAST_ERR_PLAN:   return "invalid plan or context handle";
        case CAST_ERR_ALIAS:  return "buffers of one matrix overlap";
        case CAST_ERR_MEMORY: return "a pointer is not of the required memory kind";
    }
    return "unknown status";
}

extern "C" int cast_last_cuda_error(void) { return cast::g_last_cuda_error; }

extern "C" unsigned long long cast_kernel_launch_count(void)
{
    return cast::g_launches.load(std::memory_order_relaxed);
}
