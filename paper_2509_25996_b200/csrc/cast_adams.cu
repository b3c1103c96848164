// Entry points of the AdamS N:M library: argument checks, per-iteration scalars, launches, plans.
// Everything that can be wrong is detected on the host before a launch; no device-side waits exist.
#include <atomic>
#include <cmath>
#include <cstring>
#include <new>
#include <vector>

#include "cast_internal.h"

namespace cast {

static thread_local int g_last_cuda_error = 0;
static std::atomic<unsigned long long> g_launches{0};

void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

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
                           CAST_F_V_KEPT_FROM_G | CAST_F_EMIT_DENSE | CAST_F_EMIT_COMPRESSED |
                           CAST_F_GRAD_OF_SCALED | CAST_F_MASK_STATS | CAST_F_BULK_STAGING | CAST_F_PLAIN_ACCESS;
    if (flags & ~known) return CAST_ERR_HYPER;
    if ((flags & CAST_F_BULK_STAGING) && (flags & CAST_F_PLAIN_ACCESS)) return CAST_ERR_HYPER;
    if ((flags & CAST_F_EMIT_COMPRESSED) && (flags & CAST_F_EMIT_DENSE)) return CAST_ERR_HYPER;
    if ((flags & CAST_F_EMIT_COMPRESSED) && M > kUnitElems) return CAST_ERR_NM;
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
    c.inv_bc2_s = (float)(18446744073709551616.0 / bc2);             // 2^64 / bc2
    c.lr_bc1_s = (float)(4294967296.0 * (double)lr / bc1);            // 2^32 lr / bc1
    c.eps_s = (float)(4294967296.0 * (double)eps);                    // 2^32 eps
    if (!std::isfinite(c.lr_bc1_s) || !std::isfinite(c.eps_s) || !std::isfinite(c.inv_bc2_s)) return CAST_ERR_HYPER;
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
                   const void* meta, const void* scale, int scale_groups, int64_t rows, int64_t cols,
                   uint64_t fwd_elems)
{
    if (!w || !m || !v || !g || !w_fwd || !meta) return CAST_ERR_NULL;
    const void* all[7] = {w, m, v, g, w_fwd, meta, scale};
    for (const void* p : all)
        if (p && ((uintptr_t)p & 15u)) return CAST_ERR_ALIGN;
    const uint64_t P = (uint64_t)rows * (uint64_t)cols;
    Range r[7] = {
        {(uintptr_t)w, (uintptr_t)w + 4 * P},         {(uintptr_t)m, (uintptr_t)m + 4 * P},
        {(uintptr_t)v, (uintptr_t)v + 4 * P},         {(uintptr_t)g, (uintptr_t)g + 2 * P},
        {(uintptr_t)w_fwd, (uintptr_t)w_fwd + 2 * fwd_elems}, {(uintptr_t)meta, (uintptr_t)meta + P / 8},
        {(uintptr_t)scale, (uintptr_t)scale + (scale ? 4ull * (uint64_t)rows * (uint64_t)scale_groups : 0)}};
    const int n = scale ? 7 : 6;
    for (int i = 0; i < n; ++i)
        for (int j = i + 1; j < n; ++j)
            if (overlap(r[i], r[j])) return CAST_ERR_ALIAS;
    return CAST_OK;
}

int check_scale_grad(const float* scale_grad, const float* scale, int scale_groups, int64_t rows,
                     const void* const* others, const uint64_t* other_bytes, int n_others)
{
    if (!scale_grad) return CAST_OK;
    if (!scale) return CAST_ERR_NULL;
    if ((uintptr_t)scale_grad & 15u) return CAST_ERR_ALIGN;
    const Range r = {(uintptr_t)scale_grad, (uintptr_t)scale_grad + 4ull * (uint64_t)rows * (uint64_t)scale_groups};
    for (int i = 0; i < n_others; ++i) {
        if (!others[i]) continue;
        const Range o = {(uintptr_t)others[i], (uintptr_t)others[i] + other_bytes[i]};
        if (overlap(r, o)) return CAST_ERR_ALIAS;
    }
    const void* p[1] = {scale_grad};
    return check_device_memory(p, 1);
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
                     const float* scale, int scale_groups, int64_t rows, int64_t cols, float* scale_grad,
                     const uint32_t* meta_ref, const float* scale_chain)
{
    TensorDesc d;
    std::memset(&d, 0, sizeof d);
    d.w = w; d.m = m; d.v = v; d.g = g; d.w_fwd = w_fwd; d.meta = meta; d.scale = scale;
    d.scale_grad = scale ? scale_grad : nullptr;
    d.meta_ref = reinterpret_cast<const uint8_t*>(meta_ref);
    d.scale_chain = scale ? (scale_chain ? scale_chain : scale) : nullptr;
    d.n_units = (uint32_t)((uint64_t)rows * (uint64_t)cols / kUnitElems);
    if (scale) {
        const uint32_t seg_units = (uint32_t)(cols / scale_groups / kUnitElems);
        fast_div(seg_units, &d.seg_magic, &d.seg_shift);
    }
    return d;
}

// ---------------------------------------------------------------------------------------------
// launches

// The kernels are instantiated in step_inst.cu, compiled once per slice (M, two_four, statistics, reading of
// Eq. 8) with every valid compile-time flag word of that slice; each such object exports one launcher.
using StepLauncher = int (*)(uint32_t flag_word, const StepLaunch& a);
#define CAST_SLICE(M, TF, S, V) int launch_step_m##M##_tf##TF##_s##S##_v##V(uint32_t flag_word, const StepLaunch& a);
#define CAST_SLICES_OF(M, TF) CAST_SLICE(M, TF, 0, 0) CAST_SLICE(M, TF, 0, 1) CAST_SLICE(M, TF, 1, 0) CAST_SLICE(M, TF, 1, 1)
CAST_SLICES_OF(2, 0) CAST_SLICES_OF(4, 0) CAST_SLICES_OF(4, 1) CAST_SLICES_OF(8, 0) CAST_SLICES_OF(16, 0) CAST_SLICES_OF(32, 0)
#undef CAST_SLICE
#define CAST_SLICE(M, TF, S, V) launch_step_m##M##_tf##TF##_s##S##_v##V,
// indexed [group size: 2, 4, 4 as 2:4, 8, 16, 32][statistics * 2 + alternate reading]
static const StepLauncher kStepLaunchers[6][4] = {
    {CAST_SLICES_OF(2, 0)}, {CAST_SLICES_OF(4, 0)}, {CAST_SLICES_OF(4, 1)}, {CAST_SLICES_OF(8, 0)}, {CAST_SLICES_OF(16, 0)}, {CAST_SLICES_OF(32, 0)}};
#undef CAST_SLICE
#undef CAST_SLICES_OF

// bulk_step.cu: the headline step staged through shared memory by bulk copies
bool bulk_variant_exists(int M, int n_keep, uint32_t flag_word);
int launch_bulk(const StepLaunch& a, int M, uint32_t flag_word);

uint32_t kernel_flag_word(uint32_t flags)
{
    uint32_t f = flags & kCompileTimeFlags;
    if (!(f & kReselect)) f &= ~kCountFlips;       // a reused mask has no flips: the counter gets nothing added
    return f;
}

int launch_step(const StepLaunch& a, int M)
{
    const uint32_t f = kernel_flag_word(a.c->flags);
    const bool two_four = M == 4 && a.c->n_keep == 2;
    const bool st = (f & kMaskStats) != 0;
    if (!step_kernel_exists(M, two_four, f)) return CAST_ERR_NM;
    if (a.single ? tiles_of(*a.single) == 0 : a.multi->tile_start[a.multi->n_tensors] == 0) return CAST_OK;
    if (a.single && tiles_of(*a.single) > kMaxTiles) return CAST_ERR_SHAPE;
    const bool staged_built = bulk_variant_exists(M, a.c->n_keep, f);
    if ((a.c->flags & CAST_F_BULK_STAGING) && !staged_built) return CAST_ERR_NM;      // not a configuration the staged form is built for
    // Left to itself a plan stages launches of at least 16 Ki tiles (16.8 M parameters): below that a launch is over
    // before the device's power limit matters, and the staged form's extra latency per CTA shows instead (one
    // 3072 x 768 matrix, cold: 20.3 against 18.6 us).
    const uint64_t n_tiles = a.single ? tiles_of(*a.single) : a.multi->tile_start[a.multi->n_tensors];
    const bool by_default = a.prefer_staged && staged_built && n_tiles >= 16384u && !(a.c->flags & CAST_F_PLAIN_ACCESS);
    if ((a.c->flags & CAST_F_BULK_STAGING) || by_default) {
        const int brc = launch_bulk(a, M, f);
        if (brc == CAST_OK) g_launches.fetch_add(1, std::memory_order_relaxed);
        return brc;
    }
    int row = -1;
    switch (M) {
        case 2:  row = 0; break;
        case 4:  row = two_four ? 2 : 1; break;
        case 8:  row = 3; break;
        case 16: row = 4; break;
        case 32: row = 5; break;
    }
    if (row < 0) return CAST_ERR_NM;
    const int rc = kStepLaunchers[row][(st ? 2 : 0) + ((f & kVKeptFromG) ? 1 : 0)](f, a);
    if (rc == CAST_OK) g_launches.fetch_add(1, std::memory_order_relaxed);
    return rc;
}

int launch_single(const TensorDesc& d, int M, const StepConsts& c, unsigned long long* flip_count, cudaStream_t stream)
{
    const StepLaunch a = {&d, nullptr, &c, flip_count, nullptr, stream, nullptr, false};
    return launch_step(a, M);
}

int launch_multi(const MultiParams& p, int M, const StepConsts& c, unsigned long long* flip_count, cudaStream_t stream,
                 MaskStats* stat_slots, unsigned long long* fail_word)
{
    // a plan that owns a failure word lets the library choose the access path
    if (p.n_tensors == 1 && stat_slots == nullptr) {
        // one matrix: the single-matrix kernels take a 96-byte descriptor instead of the 32 KB table (a launch of a
        // few thousand CTAs is 2-3 us shorter: 3072 x 768, cold, 17.6 against 20.1 us)
        const StepLaunch one = {&p.desc[0], nullptr, &c, flip_count, nullptr, stream, fail_word, fail_word != nullptr};
        return launch_step(one, M);
    }
    const StepLaunch a = {nullptr, &p, &c, flip_count, stat_slots, stream, fail_word, fail_word != nullptr};
    return launch_step(a, M);
}

void fill_hint_table(uint32_t n_tensors, const uint32_t* tile_start, uint16_t* hint, uint32_t* hint_shift)
{
    const uint64_t tiles = tile_start[n_tensors];
    uint32_t shift = 0;
    while (((tiles + (1ull << shift) - 1) >> shift) > (uint64_t)kHintEntries) ++shift;
    *hint_shift = shift;
    const size_t n_hints = (size_t)((tiles + (1ull << shift) - 1) >> shift);
    size_t k = 0;
    for (size_t b = 0; b < (size_t)kHintEntries; ++b) {
        if (b < n_hints) {
            const uint64_t first = (uint64_t)b << shift;
            while (first >= tile_start[k + 1]) ++k;
        }
        hint[b] = (uint16_t)k;
    }
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
    uint32_t plan_flags;                 // CAST_F_EMIT_COMPRESSED fixes the size of the w_fwd buffers; CAST_F_MASK_STATS
                                         // says the plan owns the statistics slots
    MaskStats* stat_slots;               // device, kStatSlots accumulators (zero between steps), or nullptr
    unsigned long long* fail_word;       // page-locked host memory the staged kernels count abandoned copies in, or nullptr
    std::vector<MultiParams> launches;   // one table per launch of up to kMaxLaunchTensors matrices
};

// Adds the sum of the slots to the caller's accumulator and clears them (one CTA of kStatSlots threads).
__global__ void __launch_bounds__(kStatSlots)
fold_stat_slots_kernel(MaskStats* __restrict__ slots, MaskStats* __restrict__ out)
{
    MaskStats mine = slots[threadIdx.x];
    slots[threadIdx.x] = MaskStats{0ull, 0ull, 0.0, 0.0};
    unsigned long long d = mine.mask_diff;
    double k = mine.kept_abs_sum, t = mine.total_abs_sum;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        d += __shfl_down_sync(0xFFFFFFFFu, d, o);
        k += __shfl_down_sync(0xFFFFFFFFu, k, o);
        t += __shfl_down_sync(0xFFFFFFFFu, t, o);
    }
    __shared__ unsigned long long s_d[kStatSlots / 32];
    __shared__ double s_k[kStatSlots / 32], s_t[kStatSlots / 32];
    if ((threadIdx.x & 31) == 0) { s_d[threadIdx.x >> 5] = d; s_k[threadIdx.x >> 5] = k; s_t[threadIdx.x >> 5] = t; }
    __syncthreads();
    if (threadIdx.x < 32) {
        d = s_d[threadIdx.x]; k = s_k[threadIdx.x]; t = s_t[threadIdx.x];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            d += __shfl_down_sync(0xFFFFFFFFu, d, o);
            k += __shfl_down_sync(0xFFFFFFFFu, k, o);
            t += __shfl_down_sync(0xFFFFFFFFu, t, o);
        }
        if (threadIdx.x == 0) {
            atomicAdd(&out->mask_diff, d);
            atomicAdd(&out->kept_abs_sum, k);
            atomicAdd(&out->total_abs_sum, t);
        }
    }
}
static_assert(kStatSlots == 1024, "the fold kernel is one CTA with one thread per slot");
}  // namespace

int plan_tensor_count(const void* plan)
{
    const Plan* p = (const Plan*)plan;
    if (!p || p->magic != kPlanMagic) return -1;
    return p->n_tensors;
}

bool plan_tensor_desc(const void* plan, int i, int* N, int* M, TensorDesc* desc)
{
    const Plan* p = (const Plan*)plan;
    if (!p || p->magic != kPlanMagic || i < 0 || i >= p->n_tensors) return false;
    for (const MultiParams& mp : p->launches) {
        if (i < (int)mp.n_tensors) {
            *N = p->N;
            *M = p->M;
            *desc = mp.desc[i];
            return true;
        }
        i -= (int)mp.n_tensors;
    }
    return false;
}

bool plan_tensor(const void* plan, int i, int* M, const float** w, const uint32_t** meta, uint32_t* n_units)
{
    const Plan* p = (const Plan*)plan;
    if (!p || p->magic != kPlanMagic || i < 0 || i >= p->n_tensors) return false;
    for (const MultiParams& mp : p->launches) {
        if (i < (int)mp.n_tensors) {
            *M = p->M;
            *w = mp.desc[i].w;
            *meta = mp.desc[i].meta;
            *n_units = mp.desc[i].n_units;
            return true;
        }
        i -= (int)mp.n_tensors;
    }
    return false;
}

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
    if (flags & CAST_F_MASK_STATS) return CAST_ERR_PLAN;      // the statistics epilogue needs a plan (cast_plan_step_stats)
    StepConsts c;
    if ((rc = make_step_consts(lr, beta1, beta2, eps, l1_coeff, step, total_steps, N, flags, &c)) != CAST_OK) return rc;
    if (!w || !m || !v || !g || !w_fwd_bf16 || !meta) return CAST_ERR_NULL;
    if ((rc = check_shape(rows, cols, M, scale != nullptr, scale_groups)) != CAST_OK) return rc;
    if ((rc = check_pointers(w, m, v, g, w_fwd_bf16, meta, scale, scale_groups, rows, cols,
                             fwd_elems_of(rows, cols, N, M, flags))) != CAST_OK) return rc;
    const void* ptrs[8] = {w, m, v, g, w_fwd_bf16, meta, scale, (flags & CAST_F_COUNT_FLIPS) ? flip_count : nullptr};
    if ((rc = check_device_memory(ptrs, 8)) != CAST_OK) return rc;
    const TensorDesc d = make_desc(w, m, v, g, w_fwd_bf16, meta, scale, scale_groups, rows, cols);
    return launch_single(d, M, c, flip_count, (cudaStream_t)stream);
}

namespace {
// Checks of one matrix descriptor beyond what check_shape / check_pointers do: the scale-gradient buffer.
int check_tensor_scale_grad(const cast_tensor_t& t, int N, int M, uint32_t fwd_flags)
{
    const uint64_t P = (uint64_t)t.rows * (uint64_t)t.cols;
    const void* others[7] = {t.w, t.m, t.v, t.g, t.w_fwd, t.meta, t.scale};
    const uint64_t bytes[7] = {4 * P, 4 * P, 4 * P, 2 * P, 2 * fwd_elems_of(t.rows, t.cols, N, M, fwd_flags), P / 8,
                               t.scale ? 4ull * (uint64_t)t.rows * (uint64_t)t.scale_groups : 0};
    return check_scale_grad(t.scale_grad, t.scale, t.scale_groups, t.rows, others, bytes, 7);
}
}  // namespace

namespace {
// The accumulator of CAST_F_MASK_STATS: required with the flag, 8-byte aligned device memory.
int check_stats_ptr(uint32_t flags, const cast_mask_stats_t* stats)
{
    if (!(flags & CAST_F_MASK_STATS)) return CAST_OK;
    if (!stats) return CAST_ERR_NULL;
    if ((uintptr_t)stats & 7u) return CAST_ERR_ALIGN;
    const void* p[1] = {stats};
    return check_device_memory(p, 1);
}
// The optional second scale of one matrix (the forward pass's): needs `scale`, 16-byte aligned device memory of the
// same size that the step does not write.
int check_scale_chain(const cast_tensor_t& t)
{
    if (!t.scale_chain) return CAST_OK;
    if (!t.scale) return CAST_ERR_NULL;
    if ((uintptr_t)t.scale_chain & 15u) return CAST_ERR_ALIGN;
    const uint64_t P = (uint64_t)t.rows * (uint64_t)t.cols;
    const uintptr_t lo = (uintptr_t)t.scale_chain, hi = lo + 4ull * (uint64_t)t.rows * (uint64_t)t.scale_groups;
    const void* written[6] = {t.w, t.m, t.v, t.w_fwd, t.meta, t.scale_grad};
    const uint64_t bytes[6] = {4 * P, 4 * P, 4 * P, 2 * P, P / 8, t.scale_grad ? 4ull * (uint64_t)t.rows * (uint64_t)t.scale_groups : 0};
    for (int i = 0; i < 6; ++i)
        if (written[i] && lo < (uintptr_t)written[i] + bytes[i] && (uintptr_t)written[i] < hi) return CAST_ERR_ALIAS;
    const void* p[1] = {t.scale_chain};
    return check_device_memory(p, 1);
}
// The optional reference mask of one matrix: 16-byte aligned device memory that the step does not write.
int check_meta_ref(const cast_tensor_t& t)
{
    if (!t.meta_ref) return CAST_OK;
    if ((uintptr_t)t.meta_ref & 15u) return CAST_ERR_ALIGN;
    const uint64_t P = (uint64_t)t.rows * (uint64_t)t.cols;
    const uintptr_t lo = (uintptr_t)t.meta_ref, hi = lo + P / 8;
    const void* written[5] = {t.w, t.m, t.v, t.w_fwd, t.meta};
    const uint64_t bytes[5] = {4 * P, 4 * P, 4 * P, 2 * P, P / 8};
    for (int i = 0; i < 5; ++i)
        if (lo < (uintptr_t)written[i] + bytes[i] && (uintptr_t)written[i] < hi) return CAST_ERR_ALIAS;
    const void* p[1] = {t.meta_ref};
    return check_device_memory(p, 1);
}
}  // namespace

extern "C" int cast_adams_step_ex(const cast_tensor_t* t, int N, int M, const cast_hyper_t* h,
                                  unsigned long long* flip_count, cast_stream_t stream)
{
    if (!t || !h) return CAST_ERR_NULL;
    int rc;
    if ((rc = check_nm_flags(N, M, h->flags, flip_count)) != CAST_OK) return rc;
    if (h->flags & CAST_F_MASK_STATS) return CAST_ERR_PLAN;     // the statistics epilogue needs a plan (cast_plan_step_stats)
    StepConsts c;
    if ((rc = make_step_consts(h->lr, h->beta1, h->beta2, h->eps, h->l1_coeff, h->step, h->total_steps, N, h->flags, &c)) != CAST_OK) return rc;
    if (!t->w || !t->m || !t->v || !t->g || !t->w_fwd || !t->meta) return CAST_ERR_NULL;
    if ((rc = check_shape(t->rows, t->cols, M, t->scale != nullptr, t->scale_groups)) != CAST_OK) return rc;
    if ((rc = check_pointers(t->w, t->m, t->v, t->g, t->w_fwd, t->meta, t->scale, t->scale_groups, t->rows, t->cols,
                             fwd_elems_of(t->rows, t->cols, N, M, h->flags))) != CAST_OK) return rc;
    const void* ptrs[8] = {t->w, t->m, t->v, t->g, t->w_fwd, t->meta, t->scale, (h->flags & CAST_F_COUNT_FLIPS) ? flip_count : nullptr};
    if ((rc = check_device_memory(ptrs, 8)) != CAST_OK) return rc;
    if ((rc = check_tensor_scale_grad(*t, N, M, h->flags)) != CAST_OK) return rc;
    if ((rc = check_meta_ref(*t)) != CAST_OK) return rc;
    if ((rc = check_scale_chain(*t)) != CAST_OK) return rc;
    const TensorDesc d = make_desc(t->w, t->m, t->v, t->g, t->w_fwd, t->meta, t->scale, t->scale_groups, t->rows, t->cols,
                                   t->scale_grad, t->meta_ref, t->scale_chain);
    return launch_single(d, M, c, flip_count, (cudaStream_t)stream);
}

extern "C" int cast_plan_create(const cast_tensor_t* tensors, int n_tensors, int N, int M, void** plan_out)
{
    return cast_plan_create_ex(tensors, n_tensors, N, M, 0u, plan_out);
}

extern "C" int cast_plan_create_ex(const cast_tensor_t* tensors, int n_tensors, int N, int M, uint32_t plan_flags,
                                   void** plan_out)
{
    if (!plan_out) return CAST_ERR_NULL;
    *plan_out = nullptr;
    if (!tensors) return CAST_ERR_NULL;
    if (n_tensors < 1) return CAST_ERR_SHAPE;
    int rc;
    if (plan_flags & ~(uint32_t)(CAST_F_EMIT_COMPRESSED | CAST_F_MASK_STATS)) return CAST_ERR_HYPER;
    const uint32_t fwd_flags = plan_flags & CAST_F_EMIT_COMPRESSED;
    // the encoding flag is a per-step choice; here only N:M itself (and the compressed form's M <= 8) is checked
    if ((rc = check_nm_flags(N, M, CAST_F_META_BITMASK | fwd_flags, nullptr)) != CAST_OK) return rc;

    for (int i = 0; i < n_tensors; ++i) {
        const cast_tensor_t& t = tensors[i];
        if (!t.w || !t.m || !t.v || !t.g || !t.w_fwd || !t.meta) return CAST_ERR_NULL;
        if ((rc = check_shape(t.rows, t.cols, M, t.scale != nullptr, t.scale_groups)) != CAST_OK) return rc;
        if ((rc = check_pointers(t.w, t.m, t.v, t.g, t.w_fwd, t.meta, t.scale, t.scale_groups, t.rows, t.cols,
                                 fwd_elems_of(t.rows, t.cols, N, M, fwd_flags))) != CAST_OK) return rc;
    }
    for (int i = 0; i < n_tensors; ++i) {
        const cast_tensor_t& t = tensors[i];
        const void* ptrs[7] = {t.w, t.m, t.v, t.g, t.w_fwd, t.meta, t.scale};
        if ((rc = check_device_memory(ptrs, 7)) != CAST_OK) return rc;
        if ((rc = check_tensor_scale_grad(t, N, M, fwd_flags)) != CAST_OK) return rc;
        if ((rc = check_meta_ref(t)) != CAST_OK) return rc;
        if ((rc = check_scale_chain(t)) != CAST_OK) return rc;
    }

    Plan* p = new (std::nothrow) Plan;
    if (!p) return CAST_ERR_PLAN;
    p->magic = 0;
    p->stat_slots = nullptr;
    p->fail_word = nullptr;
    cudaError_t e = cudaGetDevice(&p->device);
    if (e == cudaSuccess) {
        // One word of page-locked host memory that the device can write: without it the plan simply keeps to the
        // plain access path (the staged one is only taken where a failure can be reported to the next call).
        void* hw = nullptr;
        if (cudaHostAlloc(&hw, sizeof(unsigned long long), cudaHostAllocPortable | cudaHostAllocMapped) == cudaSuccess) {
            p->fail_word = static_cast<unsigned long long*>(hw);
            *p->fail_word = 0ull;
        } else {
            (void)cudaGetLastError();
        }
    }
    if (e == cudaSuccess && (plan_flags & CAST_F_MASK_STATS)) {
        e = cudaMalloc(&p->stat_slots, sizeof(MaskStats) * kStatSlots);
        if (e == cudaSuccess) e = cudaMemset(p->stat_slots, 0, sizeof(MaskStats) * kStatSlots);
        if (e == cudaSuccess) e = cudaDeviceSynchronize();      // the slots are zero before any stream can use them
    }
    if (e != cudaSuccess) {
        if (p->stat_slots) cudaFree(p->stat_slots);
        if (p->fail_word) cudaFreeHost(p->fail_word);
        delete p;
        return cuda_failed(e);
    }
    // cut the list into launches: at most kMaxLaunchTensors matrices and kMaxTiles tiles each
    try {
        int i = 0;
        while (i < n_tensors) {
            p->launches.emplace_back();
            MultiParams& mp = p->launches.back();
            std::memset(&mp, 0, sizeof mp);
            uint64_t tiles = 0;
            while (i < n_tensors && mp.n_tensors < (uint32_t)kMaxLaunchTensors) {
                const cast_tensor_t& t = tensors[i];
                const TensorDesc d = make_desc(t.w, t.m, t.v, t.g, t.w_fwd, t.meta, t.scale, t.scale_groups, t.rows, t.cols, t.scale_grad,
                                               t.meta_ref, t.scale_chain);
                if (tiles + tiles_of(d) > kMaxTiles) break;      // a single matrix always fits (rows*cols < 2^31)
                mp.desc[mp.n_tensors] = d;
                mp.tile_start[mp.n_tensors] = (uint32_t)tiles;
                tiles += tiles_of(d);
                ++mp.n_tensors;
                ++i;
            }
            mp.tile_start[mp.n_tensors] = (uint32_t)tiles;
            fill_hints(&mp);
        }
    } catch (const std::bad_alloc&) {
        if (p->stat_slots) cudaFree(p->stat_slots);
        if (p->fail_word) cudaFreeHost(p->fail_word);
        delete p;
        return CAST_ERR_PLAN;
    }
    p->magic = kPlanMagic;
    p->N = N; p->M = M; p->n_tensors = n_tensors;
    p->plan_flags = plan_flags;
    *plan_out = p;
    return CAST_OK;
}

extern "C" int cast_plan_step(void* plan, const cast_hyper_t* h, unsigned long long* flip_count, cast_stream_t stream)
{
    return cast_plan_step_stats(plan, h, flip_count, nullptr, stream);
}

extern "C" int cast_plan_step_stats(void* plan, const cast_hyper_t* h, unsigned long long* flip_count,
                                    cast_mask_stats_t* stats, cast_stream_t stream)
{
    Plan* p = (Plan*)plan;
    if (!p || p->magic != kPlanMagic) return CAST_ERR_PLAN;
    if (!h) return CAST_ERR_NULL;
    int rc;
    if ((rc = check_nm_flags(p->N, p->M, h->flags, flip_count)) != CAST_OK) return rc;
    if ((rc = check_stats_ptr(h->flags, stats)) != CAST_OK) return rc;
    if ((h->flags & CAST_F_EMIT_COMPRESSED) != (p->plan_flags & CAST_F_EMIT_COMPRESSED)) return CAST_ERR_PLAN;
    // a staged step of this plan gave up on a copy earlier: some tile was not updated, and the caller must know
    if (p->fail_word && *static_cast<volatile unsigned long long*>(p->fail_word) != 0ull) return CAST_ERR_STAGING;
    const bool with_stats = (h->flags & CAST_F_MASK_STATS) != 0;
    if (with_stats && !p->stat_slots) return CAST_ERR_PLAN;      // the plan was not created for statistics
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
    for (const MultiParams& mp : p->launches)
        if ((rc = launch_multi(mp, p->M, c, flip_count, (cudaStream_t)stream, with_stats ? p->stat_slots : nullptr, p->fail_word)) != CAST_OK) {
            // what the launches so far left in the slots must not reach a later step
            if (with_stats) (void)cudaMemsetAsync(p->stat_slots, 0, sizeof(MaskStats) * kStatSlots, (cudaStream_t)stream);
            return rc;
        }
    if (with_stats) {
        fold_stat_slots_kernel<<<1, kStatSlots, 0, (cudaStream_t)stream>>>(p->stat_slots, reinterpret_cast<MaskStats*>(stats));
        CAST_CUDA_TRY(cudaGetLastError());
        g_launches.fetch_add(1, std::memory_order_relaxed);
    }
    return CAST_OK;
}

extern "C" int cast_plan_report_staging_failure(void* plan)
{
    Plan* p = (Plan*)plan;
    if (!p || p->magic != kPlanMagic) return CAST_ERR_PLAN;
    if (!p->fail_word) return CAST_ERR_PLAN;
    *static_cast<volatile unsigned long long*>(p->fail_word) += 1ull;      // what a staged kernel does when it gives up on a copy
    return CAST_OK;
}

extern "C" int cast_plan_destroy(void* plan)
{
    Plan* p = (Plan*)plan;
    if (!p || p->magic != kPlanMagic) return CAST_ERR_PLAN;
    p->magic = 0;
    int rc = CAST_OK;
    if (p->stat_slots) {
        const cudaError_t e = cudaFree(p->stat_slots);
        if (e != cudaSuccess) rc = cuda_failed(e);
    }
    if (p->fail_word) {
        const cudaError_t e = cudaFreeHost(p->fail_word);
        if (e != cudaSuccess) rc = cuda_failed(e);
    }
    delete p;
    return rc;
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
        case CAST_ERR_STAGING: return "an earlier staged step of this plan gave up waiting for a bulk copy: a tile was not updated";
    }
    return "unknown status";
}

extern "C" int cast_last_cuda_error(void) { return cast::g_last_cuda_error; }

extern "C" unsigned long long cast_kernel_launch_count(void)
{
    return cast::g_launches.load(std::memory_order_relaxed);
}
