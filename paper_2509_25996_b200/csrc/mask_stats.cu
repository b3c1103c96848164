// Mask statistics of CAST, App. C: ||M - M_ref||_0 (numerator of the flip rate r_t against the previous
// mask, of the initial flip rate i_t against the initial mask) and the two sums of the sparse weight ratio
// S_t = ||W (.) M||_1 / ||W||_1.  A read-only streaming reduction: 4 B of weight and 1/8 B (2/8 B with a
// reference mask) of metadata per parameter, HBM-bound.
//
// One thread owns units of 8 consecutive columns (two 128-bit weight loads, one metadata byte per mask).
// A CTA of 256 threads covers a tile of 32768 parameters in 4 batches of 4 units per thread, the loads of a
// batch issued before any use; magnitudes are summed in fp64 (|w| converts exactly), reduced by warp
// shuffles and shared memory, and each CTA adds its three partial results to the caller's counters with one
// atomic each (so few CTAs per byte that the same-address atomics stay off the critical path).  All
// matrices of a plan go in one grid, found through the same parameter-space tables as the step's.
#include <cstring>

#include "cast_internal.h"

namespace cast {

bool plan_tensor(const void* plan, int i, int* M, const float** w, const uint32_t** meta, uint32_t* n_units);

namespace {

constexpr int kStatsThreads = 256;
constexpr int kStatsUnitsPerThread = 4;    // units loaded together by a thread
constexpr int kStatsIters = 4;             // such batches per CTA
constexpr int kStatsBatchUnits = kStatsThreads * kStatsUnitsPerThread;
constexpr int kStatsTileUnits = kStatsBatchUnits * kStatsIters;        // 4096 units = 32768 parameters per CTA

// One matrix of a statistics launch, and the tables of the launch (kernel parameter space, like the step's).
struct StatsDesc {
    const float* w;
    const uint8_t* meta;
    const uint8_t* meta_ref;      // nullptr: no reference mask
    uint32_t n_units;
    uint32_t pad_;
};
struct StatsParams {
    uint32_t n_tensors;
    uint32_t hint_shift;
    uint16_t hint[kHintEntries];
    uint32_t tile_start[kMaxLaunchTensors + 1];
    StatsDesc desc[kMaxLaunchTensors];
};

__device__ __forceinline__ double warp_sum(double x)
{
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) x += __shfl_down_sync(0xFFFFFFFFu, x, d);
    return x;
}

__global__ void __launch_bounds__(kStatsThreads)
mask_stats_kernel(const __grid_constant__ StatsParams p, bool bitmask, cast_mask_stats_t* __restrict__ out)
{
    const uint32_t tile = blockIdx.x;
    uint32_t k = p.hint[tile >> p.hint_shift];
    while (tile >= p.tile_start[k + 1]) ++k;
    const StatsDesc& t = p.desc[k];
    const bool has_ref = t.meta_ref != nullptr;
    const uint32_t tile_first = (tile - p.tile_start[k]) * kStatsTileUnits;

    uint32_t flips = 0;
    double kept = 0.0, total = 0.0;
#pragma unroll 1
    for (int it = 0; it < kStatsIters; ++it) {
        const uint32_t first = tile_first + it * kStatsBatchUnits + threadIdx.x;
        if (first - threadIdx.x >= t.n_units) break;
        float4 a[kStatsUnitsPerThread], b[kStatsUnitsPerThread];
        uint32_t mb[kStatsUnitsPerThread], rb[kStatsUnitsPerThread];
#pragma unroll
        for (int j = 0; j < kStatsUnitsPerThread; ++j) {
            const uint32_t unit = first + j * kStatsThreads;
            a[j] = b[j] = make_float4(0.f, 0.f, 0.f, 0.f);
            mb[j] = rb[j] = 0;
            if (unit < t.n_units) {
                const float* q = t.w + (size_t)unit * kUnitElems;
                a[j] = ld_f4(q);
                b[j] = ld_f4(q + 4);
                mb[j] = t.meta[unit];
                if (has_ref) rb[j] = t.meta_ref[unit];
            }
        }
#pragma unroll
        for (int j = 0; j < kStatsUnitsPerThread; ++j) {
            const uint32_t unit = first + j * kStatsThreads;
            if (unit >= t.n_units) continue;               // an index-form byte 0 is not "nothing kept"
            const uint32_t keep = keep_from_meta_byte(mb[j], bitmask);
            if (has_ref) flips += (uint32_t)__popc(keep ^ keep_from_meta_byte(rb[j], bitmask));
            const float x[8] = {a[j].x, a[j].y, a[j].z, a[j].w, b[j].x, b[j].y, b[j].z, b[j].w};
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const double m = (double)fabsf(x[i]);
                total += m;
                if ((keep >> i) & 1u) kept += m;
            }
        }
    }
    flips = __reduce_add_sync(0xFFFFFFFFu, flips);
    kept = warp_sum(kept);
    total = warp_sum(total);
    __shared__ uint32_t s_flips[kStatsThreads / 32];
    __shared__ double s_kept[kStatsThreads / 32], s_total[kStatsThreads / 32];
    const int warp = threadIdx.x >> 5;
    if ((threadIdx.x & 31) == 0) { s_flips[warp] = flips; s_kept[warp] = kept; s_total[warp] = total; }
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned long long f = 0;
        double ks = 0.0, ts = 0.0;
#pragma unroll
        for (int i = 0; i < kStatsThreads / 32; ++i) { f += s_flips[i]; ks += s_kept[i]; ts += s_total[i]; }
        if (f) atomicAdd(&out->mask_diff, f);
        atomicAdd(&out->kept_abs_sum, ks);
        atomicAdd(&out->total_abs_sum, ts);
    }
}

int launch_stats(StatsParams* p, bool bitmask, cast_mask_stats_t* stats, cudaStream_t s)
{
    fill_hint_table(p->n_tensors, p->tile_start, p->hint, &p->hint_shift);
    const uint32_t tiles = p->tile_start[p->n_tensors];
    if (tiles == 0) return CAST_OK;
    mask_stats_kernel<<<tiles, kStatsThreads, 0, s>>>(*p, bitmask, stats);
    CAST_CUDA_TRY(cudaGetLastError());
    count_launch();
    return CAST_OK;
}

int check_stats_args(int M, uint32_t flags, const cast_mask_stats_t* stats)
{
    if (!stats) return CAST_ERR_NULL;
    if (flags & ~(uint32_t)CAST_F_META_BITMASK) return CAST_ERR_HYPER;
    if (!(M == 2 || M == 4 || M == 8 || M == 16 || M == 32)) return CAST_ERR_NM;
    if (!(flags & CAST_F_META_BITMASK) && M != 4) return CAST_ERR_NM;
    if ((uintptr_t)stats & 7u) return CAST_ERR_ALIGN;
    return CAST_OK;
}

}  // namespace
}  // namespace cast

using namespace cast;

extern "C" int cast_mask_stats(const float* w, const uint32_t* meta, const uint32_t* meta_ref,
                               int64_t rows, int64_t cols, int M, uint32_t flags,
                               cast_mask_stats_t* stats, cast_stream_t stream)
{
    if (!w || !meta) return CAST_ERR_NULL;
    int rc;
    if ((rc = check_stats_args(M, flags, stats)) != CAST_OK) return rc;
    if ((rc = check_shape(rows, cols, M, false, 1)) != CAST_OK) return rc;
    if (((uintptr_t)w & 15u) || ((uintptr_t)meta & 15u) || ((uintptr_t)meta_ref & 15u)) return CAST_ERR_ALIGN;
    const void* ptrs[4] = {w, meta, meta_ref, stats};
    if ((rc = check_device_memory(ptrs, 4)) != CAST_OK) return rc;
    StatsParams p;
    std::memset(&p, 0, sizeof p);
    p.n_tensors = 1;
    p.desc[0].w = w;
    p.desc[0].meta = (const uint8_t*)meta;
    p.desc[0].meta_ref = (const uint8_t*)meta_ref;
    p.desc[0].n_units = (uint32_t)((uint64_t)rows * (uint64_t)cols / kUnitElems);
    p.tile_start[1] = (p.desc[0].n_units + kStatsTileUnits - 1) / kStatsTileUnits;
    return launch_stats(&p, (flags & CAST_F_META_BITMASK) != 0, stats, (cudaStream_t)stream);
}

extern "C" int cast_plan_mask_stats(void* plan, const uint32_t* const* meta_ref, uint32_t flags,
                                    cast_mask_stats_t* stats, cast_stream_t stream)
{
    const int n = plan_tensor_count(plan);
    if (n < 0) return CAST_ERR_PLAN;
    int M = 0;
    const float* w;
    const uint32_t* meta;
    uint32_t n_units;
    plan_tensor(plan, 0, &M, &w, &meta, &n_units);
    int rc;
    if ((rc = check_stats_args(M, flags, stats)) != CAST_OK) return rc;
    const void* sp[1] = {stats};
    if ((rc = check_device_memory(sp, 1)) != CAST_OK) return rc;
    if (meta_ref)
        for (int i = 0; i < n; ++i) {
            if (!meta_ref[i]) return CAST_ERR_NULL;
            if ((uintptr_t)meta_ref[i] & 15u) return CAST_ERR_ALIGN;
            const void* rp[1] = {meta_ref[i]};
            if ((rc = check_device_memory(rp, 1)) != CAST_OK) return rc;
        }
    int i = 0;
    while (i < n) {
        StatsParams p;
        std::memset(&p, 0, sizeof p);
        uint64_t tiles = 0;
        while (i < n && p.n_tensors < (uint32_t)kMaxLaunchTensors) {
            plan_tensor(plan, i, &M, &w, &meta, &n_units);
            StatsDesc& d = p.desc[p.n_tensors];
            d.w = w;
            d.meta = (const uint8_t*)meta;
            d.meta_ref = meta_ref ? (const uint8_t*)meta_ref[i] : nullptr;
            d.n_units = n_units;
            p.tile_start[p.n_tensors] = (uint32_t)tiles;
            tiles += (n_units + kStatsTileUnits - 1) / kStatsTileUnits;
            ++p.n_tensors;
            ++i;
        }
        p.tile_start[p.n_tensors] = (uint32_t)tiles;
        if ((rc = launch_stats(&p, (flags & CAST_F_META_BITMASK) != 0, stats, (cudaStream_t)stream)) != CAST_OK) return rc;
    }
    return CAST_OK;
}
