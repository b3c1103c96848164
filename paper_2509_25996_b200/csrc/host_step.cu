// AdamS N:M step for optimizer state that lives in HOST memory: blocks of whole rows are staged
// through device buffers and updated by the same kernel as the device-resident entry points.
// Each staging slot has its own stream; a block's host->device copies, kernel and device->host
// copies are queued on its slot's stream, so reuse of a slot is ordered by the stream and blocks
// in different slots overlap (copy engines in both directions plus the kernel).
#include <cstring>
#include <new>
#include <vector>

#include "cast_internal.h"

namespace cast {
namespace {

constexpr uint64_t kCtxMagic = 0x43415354484F5354ull;   // "CASTHOST"
constexpr int kMaxSlots = 8;
constexpr int kFlipCounters = 256;

struct Slot {
    cudaStream_t stream = nullptr;
    char* base = nullptr;          // one allocation per slot
    float *w = nullptr, *m = nullptr, *v = nullptr, *scale = nullptr;
    uint16_t *g = nullptr, *fwd = nullptr;
    uint32_t* meta = nullptr;
};

struct HostCtx {
    uint64_t magic = 0;
    int device = 0;
    int64_t max_block = 0;
    int n_slots = 0;
    int next_slot = 0;
    Slot slot[kMaxSlots];
    unsigned long long* d_flips = nullptr;       // kFlipCounters device counters
    unsigned long long* h_flips = nullptr;       // page-locked mirror
    unsigned long long* flip_dst[kFlipCounters];
    int n_flip_pending = 0;
};

size_t align_up(size_t x) { return (x + 255) & ~(size_t)255; }

void free_ctx(HostCtx* c)
{
    for (int i = 0; i < c->n_slots; ++i) {
        if (c->slot[i].base) cudaFree(c->slot[i].base);
        if (c->slot[i].stream) cudaStreamDestroy(c->slot[i].stream);
    }
    if (c->d_flips) cudaFree(c->d_flips);
    if (c->h_flips) cudaFreeHost(c->h_flips);
    c->magic = 0;
    delete c;
}

int sync_ctx(HostCtx* c)
{
    for (int i = 0; i < c->n_slots; ++i) CAST_CUDA_TRY(cudaStreamSynchronize(c->slot[i].stream));
    if (c->n_flip_pending > 0) {
        CAST_CUDA_TRY(cudaMemcpy(c->h_flips, c->d_flips, sizeof(unsigned long long) * (size_t)c->n_flip_pending,
                                 cudaMemcpyDeviceToHost));
        for (int i = 0; i < c->n_flip_pending; ++i) *c->flip_dst[i] += c->h_flips[i];
        // cleared on a slot stream and waited for: the slot streams do not order against the legacy default stream,
        // so a plain cudaMemset could still be pending when the next counting step starts
        CAST_CUDA_TRY(cudaMemsetAsync(c->d_flips, 0, sizeof(unsigned long long) * (size_t)c->n_flip_pending, c->slot[0].stream));
        CAST_CUDA_TRY(cudaStreamSynchronize(c->slot[0].stream));
        c->n_flip_pending = 0;
    }
    return CAST_OK;
}

// A host pointer must not be device-only memory.
int check_host_memory(const void* const* ptrs, int n)
{
    for (int i = 0; i < n; ++i) {
        if (!ptrs[i]) continue;
        cudaPointerAttributes attr;
        CAST_CUDA_TRY(cudaPointerGetAttributes(&attr, ptrs[i]));
        if (attr.type == cudaMemoryTypeDevice) return CAST_ERR_MEMORY;
    }
    return CAST_OK;
}

}  // namespace
}  // namespace cast

using namespace cast;

extern "C" int cast_host_ctx_create(int64_t max_block_params, int n_slots, void** ctx_out)
{
    if (!ctx_out) return CAST_ERR_NULL;
    *ctx_out = nullptr;
    if (max_block_params < 1024 || max_block_params % 32 != 0 || max_block_params > 0x7FFFFFFF) return CAST_ERR_SHAPE;
    if (n_slots < 2 || n_slots > kMaxSlots) return CAST_ERR_SHAPE;
    HostCtx* c = new (std::nothrow) HostCtx;
    if (!c) return CAST_ERR_PLAN;
    c->max_block = max_block_params;
    c->n_slots = n_slots;
    cudaError_t e = cudaGetDevice(&c->device);
    const size_t P = (size_t)max_block_params;
    const size_t off_w = 0, off_m = off_w + align_up(4 * P), off_v = off_m + align_up(4 * P);
    const size_t off_g = off_v + align_up(4 * P), off_f = off_g + align_up(2 * P);
    const size_t off_meta = off_f + align_up(2 * P), off_scale = off_meta + align_up(P / 8);
    const size_t total = off_scale + align_up(4 * (P / 8));
    for (int i = 0; i < n_slots && e == cudaSuccess; ++i) {
        Slot& s = c->slot[i];
        e = cudaStreamCreateWithFlags(&s.stream, cudaStreamNonBlocking);
        if (e != cudaSuccess) break;
        e = cudaMalloc(&s.base, total);
        if (e != cudaSuccess) break;
        s.w = (float*)(s.base + off_w);
        s.m = (float*)(s.base + off_m);
        s.v = (float*)(s.base + off_v);
        s.g = (uint16_t*)(s.base + off_g);
        s.fwd = (uint16_t*)(s.base + off_f);
        s.meta = (uint32_t*)(s.base + off_meta);
        s.scale = (float*)(s.base + off_scale);
    }
    if (e == cudaSuccess) e = cudaMalloc(&c->d_flips, sizeof(unsigned long long) * kFlipCounters);
    if (e == cudaSuccess) e = cudaMemset(c->d_flips, 0, sizeof(unsigned long long) * kFlipCounters);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();      // the counters are zero before any slot stream can add to them
    if (e == cudaSuccess) e = cudaMallocHost(&c->h_flips, sizeof(unsigned long long) * kFlipCounters);
    if (e != cudaSuccess) {
        free_ctx(c);
        return cuda_failed(e);
    }
    c->magic = kCtxMagic;
    *ctx_out = c;
    return CAST_OK;
}

extern "C" int cast_host_step(void* ctx,
                              float* w, float* m, float* v, const cast_bf16* g,
                              cast_bf16* w_fwd_bf16, uint32_t* meta,
                              const float* scale, int scale_groups,
                              int64_t rows, int64_t cols, int N, int M,
                              float lr, float beta1, float beta2, float eps, float l1_coeff,
                              int64_t step, int64_t total_steps,
                              uint32_t flags, unsigned long long* flip_count)
{
    HostCtx* c = (HostCtx*)ctx;
    if (!c || c->magic != kCtxMagic) return CAST_ERR_PLAN;
    int rc;
    if ((rc = check_nm_flags(N, M, flags, flip_count)) != CAST_OK) return rc;
    if (flags & CAST_F_MASK_STATS) return CAST_ERR_PLAN;      // the statistics epilogue needs a plan
    StepConsts k;
    if ((rc = make_step_consts(lr, beta1, beta2, eps, l1_coeff, step, total_steps, N, flags, &k)) != CAST_OK) return rc;
    if (!w || !m || !v || !g || !w_fwd_bf16 || !meta) return CAST_ERR_NULL;
    if ((rc = check_shape(rows, cols, M, scale != nullptr, scale_groups)) != CAST_OK) return rc;
    const uint64_t fwd_total = fwd_elems_of(rows, cols, N, M, flags);
    if ((rc = check_pointers(w, m, v, g, w_fwd_bf16, meta, scale, scale_groups, rows, cols, fwd_total)) != CAST_OK) return rc;
    if (cols > c->max_block) return CAST_ERR_PLAN;
    int dev = -1;
    CAST_CUDA_TRY(cudaGetDevice(&dev));
    if (dev != c->device) return CAST_ERR_PLAN;
    const void* ptrs[7] = {w, m, v, g, w_fwd_bf16, meta, scale};
    if ((rc = check_host_memory(ptrs, 7)) != CAST_OK) return rc;

    unsigned long long* d_flip = nullptr;
    if (flags & CAST_F_COUNT_FLIPS) {
        if (c->n_flip_pending == kFlipCounters && (rc = sync_ctx(c)) != CAST_OK) return rc;
        d_flip = c->d_flips + c->n_flip_pending;
        c->flip_dst[c->n_flip_pending++] = flip_count;
    }
    const bool need_prev = !(flags & CAST_F_RESELECT) || (flags & CAST_F_COUNT_FLIPS);
    const int64_t rows_per_block = c->max_block / cols;
    auto queue_all = [&]() -> int {
        for (int64_t r0 = 0; r0 < rows; r0 += rows_per_block) {
            const int64_t nr = (rows - r0 < rows_per_block) ? rows - r0 : rows_per_block;
            const size_t P = (size_t)nr * (size_t)cols, off = (size_t)r0 * (size_t)cols;
            Slot& s = c->slot[c->next_slot];
            c->next_slot = (c->next_slot + 1) % c->n_slots;
            CAST_CUDA_TRY(cudaMemcpyAsync(s.w, w + off, 4 * P, cudaMemcpyHostToDevice, s.stream));
            CAST_CUDA_TRY(cudaMemcpyAsync(s.m, m + off, 4 * P, cudaMemcpyHostToDevice, s.stream));
            CAST_CUDA_TRY(cudaMemcpyAsync(s.v, v + off, 4 * P, cudaMemcpyHostToDevice, s.stream));
            CAST_CUDA_TRY(cudaMemcpyAsync(s.g, g + off, 2 * P, cudaMemcpyHostToDevice, s.stream));
            if (need_prev)
                CAST_CUDA_TRY(cudaMemcpyAsync(s.meta, meta + off / 32, P / 8, cudaMemcpyHostToDevice, s.stream));
            if (scale)
                CAST_CUDA_TRY(cudaMemcpyAsync(s.scale, scale + (size_t)r0 * (size_t)scale_groups,
                                              4 * (size_t)nr * (size_t)scale_groups, cudaMemcpyHostToDevice, s.stream));
            const TensorDesc d = make_desc(s.w, s.m, s.v, s.g, s.fwd, s.meta, scale ? s.scale : nullptr, scale_groups, nr, cols);
            const int launch_rc = launch_single(d, M, k, d_flip, s.stream);
            if (launch_rc != CAST_OK) return launch_rc;
            CAST_CUDA_TRY(cudaMemcpyAsync(w + off, s.w, 4 * P, cudaMemcpyDeviceToHost, s.stream));
            CAST_CUDA_TRY(cudaMemcpyAsync(m + off, s.m, 4 * P, cudaMemcpyDeviceToHost, s.stream));
            CAST_CUDA_TRY(cudaMemcpyAsync(v + off, s.v, 4 * P, cudaMemcpyDeviceToHost, s.stream));
            const size_t fwd_scale_n = (flags & CAST_F_EMIT_COMPRESSED) ? (size_t)N : 1, fwd_scale_m = (flags & CAST_F_EMIT_COMPRESSED) ? (size_t)M : 1;
            CAST_CUDA_TRY(cudaMemcpyAsync(w_fwd_bf16 + off / fwd_scale_m * fwd_scale_n, s.fwd, 2 * (P / fwd_scale_m * fwd_scale_n),
                                          cudaMemcpyDeviceToHost, s.stream));
            CAST_CUDA_TRY(cudaMemcpyAsync(meta + off / 32, s.meta, P / 8, cudaMemcpyDeviceToHost, s.stream));
        }
        return CAST_OK;
    };
    rc = queue_all();
    if (rc != CAST_OK) {
        // a call failed part-way: wait for the copies already queued, so that nothing is still reading or writing the
        // caller's host buffers when the error comes back (the state in them may be partly updated)
        for (int i = 0; i < c->n_slots; ++i) (void)cudaStreamSynchronize(c->slot[i].stream);
        (void)cudaGetLastError();
    }
    return rc;
}

extern "C" int cast_host_ctx_sync(void* ctx)
{
    HostCtx* c = (HostCtx*)ctx;
    if (!c || c->magic != kCtxMagic) return CAST_ERR_PLAN;
    return sync_ctx(c);
}

extern "C" int cast_host_ctx_destroy(void* ctx)
{
    HostCtx* c = (HostCtx*)ctx;
    if (!c || c->magic != kCtxMagic) return CAST_ERR_PLAN;
    const int rc = sync_ctx(c);
    free_ctx(c);
    return rc;
}
