// The AdamS step with its tiles staged through shared memory by bulk asynchronous copies instead of per-thread
// 128-bit loads and stores (CAST_F_BULK_STAGING; what plan steps of model size take by default).  Same arithmetic
// (compute_unit of the plain kernels), same results bit for bit.  Built for the configurations listed at the end of
// this file; measured on B200 it is as fast as the plain form in short runs and 0-3 % faster in sustained ones (the
// tile traffic bypasses the L1/texture path: less power, higher clock under the board's power cap).
//
// Per CTA (128 threads, one tile of 1024 parameters): one elected thread arms an mbarrier with the tile's byte count
// and issues four bulk copies global -> shared (w, m, v: 4 KB each, g: 2 KB; this GPU's own memory, no multicast).
// Meanwhile every thread loads what does not come through the tile (its previous metadata byte, its scale), so that
// these travel with the tile.  All threads then wait on the barrier's phase, compute from shared memory, write w, m, v
// and the forward weight back into the same shared memory, make those writes visible to the asynchronous proxy, and the
// elected thread issues four bulk copies shared -> global and waits until they have read the shared memory.  The
// metadata byte goes out by an ordinary store.  14.4 KB of shared memory; the register budget (8 or 9 CTAs per SM) is
// chosen per variant from measurements (staged_ctas_per_sm below).
//
// The wait on the barrier is bounded: a phase that has not completed after 2^16 polls with back-off (about 2 ms) is
// counted in a device-side counter (cast_bulk_timeout_count) and, for plans, in a word of host memory that the plan's
// next step checks; the CTA waits once more with the same limit and then gives up without storing.  Every copy starts
// on a 16-byte boundary (tiles start at multiples of 1024 elements of 16-byte aligned buffers) and has a size that is
// a multiple of 16 bytes (a matrix has a multiple of 4 units).
#include "cast_internal.h"

namespace cast {
namespace {

constexpr uint32_t kPollLimit = 1u << 16;      // ~2 ms with the back-off below; a tile's copies take microseconds

__device__ unsigned long long g_bulk_timeouts;      // phases given up on, over the life of the process

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void barrier_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void barrier_expect(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool barrier_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t done;
    asm volatile("{ .reg .pred p;\n\t"
                 "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p; }" : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    return done != 0;
}
// Polls the phase with a limit; false if it gave up.
__device__ __forceinline__ bool barrier_wait_bounded(uint32_t bar, uint32_t parity)
{
    for (uint32_t i = 0; i < kPollLimit; ++i) {
        if (barrier_try_wait(bar, parity)) return true;
        if (i > 64) __nanosleep(32);
    }
    return false;
}
__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst_smem), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_store(void* dst, uint32_t src_smem, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src_smem), "r"(bytes) : "memory");
}

struct __align__(128) BulkTile {
    float w[kTileUnits * kUnitElems];
    float m[kTileUnits * kUnitElems];
    float v[kTileUnits * kUnitElems];
    uint16_t g[kTileUnits * kUnitElems];       // gradient in, forward weight out
    unsigned long long barrier;
};

template <int M, uint32_t F, bool TF>
__device__ __forceinline__ void bulk_tile(const TensorDesc& t, const StepConsts& c, uint32_t first_unit,
                                          unsigned long long* flip_count, MaskStats* stats, unsigned long long* fail_word)
{
    using Cfg = StepCfg<M, F, TF>;
    static_assert(M <= 8 && !Cfg::of_scaled, "staged form: groups inside a thread, no scale gradient");
    static_assert(!Cfg::compressed || (TF && !Cfg::bitmask), "staged compressed emission: 2:4 with index-form metadata");
    __shared__ BulkTile tile;
    const uint32_t units = min((uint32_t)kTileUnits, t.n_units - first_unit);       // a matrix's last tile may be short
    const size_t e0 = (size_t)first_unit * kUnitElems;
    const uint32_t bar = smem_addr(&tile.barrier);
    if (threadIdx.x == 0) {
        barrier_init(bar, 1);
        const uint32_t b4 = units * kUnitElems * 4u, b2 = units * kUnitElems * 2u;
        barrier_expect(bar, 3u * b4 + b2);
        bulk_load(smem_addr(tile.w), t.w + e0, b4, bar);
        bulk_load(smem_addr(tile.m), t.m + e0, b4, bar);
        bulk_load(smem_addr(tile.v), t.v + e0, b4, bar);
        bulk_load(smem_addr(tile.g), t.g + e0, b2, bar);
    }
    // what does not come through the tile is asked for now, so that it travels while the tile does
    const uint32_t u_idx = threadIdx.x;
    const bool active = u_idx < units;
    uint32_t prev_byte = 0, ref_byte = 0;
    float a = 1.0f;
    const bool has_ref = Cfg::stats && t.meta_ref != nullptr;      // uniform over the CTA
    if (active) {
        if constexpr (Cfg::need_prev) prev_byte = reinterpret_cast<const uint8_t*>(t.meta)[first_unit + u_idx];
        if (has_ref) ref_byte = t.meta_ref[first_unit + u_idx];
        if (t.scale != nullptr) a = __ldg(t.scale + (uint32_t)(((uint64_t)(first_unit + u_idx) * t.seg_magic) >> t.seg_shift));
    }
    __syncthreads();                            // the barrier is initialised before anyone polls it
    bool arrived = barrier_wait_bounded(bar, 0);
    if (!arrived) {
        if (threadIdx.x == 0) {
            atomicAdd(&g_bulk_timeouts, 1ull);
            if (fail_word != nullptr) atomicAdd_system(fail_word, 1ull);      // host memory: the next call on the host sees it
        }
        arrived = barrier_wait_bounded(bar, 0); // the copies may still land: give them the same time again
    }
    if (!__syncthreads_and(arrived)) return;    // nothing is stored for a tile whose data did not arrive (uniform over the CTA)

    UnitRegs u;
    UnitSums sums;
    float gw_sum = 0.0f;
    uint2 kept_out = make_uint2(0u, 0u);
    if (active) {
        const float4 w0 = *reinterpret_cast<const float4*>(tile.w + u_idx * 8), w1 = *reinterpret_cast<const float4*>(tile.w + u_idx * 8 + 4);
        const float4 m0 = *reinterpret_cast<const float4*>(tile.m + u_idx * 8), m1 = *reinterpret_cast<const float4*>(tile.m + u_idx * 8 + 4);
        const float4 v0 = *reinterpret_cast<const float4*>(tile.v + u_idx * 8), v1 = *reinterpret_cast<const float4*>(tile.v + u_idx * 8 + 4);
        u.g = *reinterpret_cast<const uint4*>(tile.g + u_idx * 8);
        u.w[0] = w0.x; u.w[1] = w0.y; u.w[2] = w0.z; u.w[3] = w0.w; u.w[4] = w1.x; u.w[5] = w1.y; u.w[6] = w1.z; u.w[7] = w1.w;
        u.m[0] = m0.x; u.m[1] = m0.y; u.m[2] = m0.z; u.m[3] = m0.w; u.m[4] = m1.x; u.m[5] = m1.y; u.m[6] = m1.z; u.m[7] = m1.w;
        u.v[0] = v0.x; u.v[1] = v0.y; u.v[2] = v0.z; u.v[3] = v0.w; u.v[4] = v1.x; u.v[5] = v1.y; u.v[6] = v1.z; u.v[7] = v1.w;
    } else {
        u.g = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int i = 0; i < 8; ++i) { u.w[i] = 0.f; u.m[i] = 0.f; u.v[i] = 0.f; }
    }
    u.prev_byte = prev_byte;
    u.ref_byte = ref_byte;
    UnitSums mine;
    compute_unit<M, F, TF>(u, c, a, has_ref, gw_sum, mine);
    if (active) {
        sums = mine;
        *reinterpret_cast<float4*>(tile.w + u_idx * 8) = make_float4(u.w[0], u.w[1], u.w[2], u.w[3]);
        *reinterpret_cast<float4*>(tile.w + u_idx * 8 + 4) = make_float4(u.w[4], u.w[5], u.w[6], u.w[7]);
        *reinterpret_cast<float4*>(tile.m + u_idx * 8) = make_float4(u.m[0], u.m[1], u.m[2], u.m[3]);
        *reinterpret_cast<float4*>(tile.m + u_idx * 8 + 4) = make_float4(u.m[4], u.m[5], u.m[6], u.m[7]);
        *reinterpret_cast<float4*>(tile.v + u_idx * 8) = make_float4(u.v[0], u.v[1], u.v[2], u.v[3]);
        *reinterpret_cast<float4*>(tile.v + u_idx * 8 + 4) = make_float4(u.v[4], u.v[5], u.v[6], u.v[7]);
        if constexpr (Cfg::compressed) {
            // the kept pair of each group, picked by the index nibbles: 4 values per unit
            const uint32_t mb = u.meta_byte;
            kept_out = make_uint2(kept_pair_by_index(u.g.x, u.g.y, mb & 3u, (mb >> 2) & 3u),
                                  kept_pair_by_index(u.g.z, u.g.w, (mb >> 4) & 3u, mb >> 6));
        } else {
            *reinterpret_cast<uint4*>(tile.g + u_idx * 8) = u.g;
        }
        if constexpr (Cfg::reselect) reinterpret_cast<uint8_t*>(t.meta)[first_unit + u_idx] = (uint8_t)u.meta_byte;
    }
    if constexpr (Cfg::compressed) {
        // packed densely, a unit's 8 bytes land in the gradient slot of another unit: every thread has read its
        // gradient before anyone writes
        __syncthreads();
        if (active) *reinterpret_cast<uint2*>(tile.g + u_idx * 4) = kept_out;
    }
    // The flip count rides on the barrier the stores need anyway: a reduction after the stores made every warp wait
    // for the elected thread's wait on them (4:8 with flips over the 7B set: 27.45 against 26.35 ms).
    __shared__ uint32_t warp_flips[kThreads / 32], warp_diff[kThreads / 32];
    __shared__ double warp_kept[kThreads / 32], warp_total[kThreads / 32];
    if constexpr (Cfg::count_flips) {
        const uint32_t f = __reduce_add_sync(0xFFFFFFFFu, sums.flips);
        if ((threadIdx.x & 31) == 0) warp_flips[threadIdx.x >> 5] = f;
    }
    if constexpr (Cfg::stats) {      // the App. C sums of the step's epilogue take the same ride
        const uint32_t d = __reduce_add_sync(0xFFFFFFFFu, sums.mask_diff);
        double k = sums.kept_abs, tt = sums.total_abs;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            k += __shfl_down_sync(0xFFFFFFFFu, k, o);
            tt += __shfl_down_sync(0xFFFFFFFFu, tt, o);
        }
        if ((threadIdx.x & 31) == 0) { warp_diff[threadIdx.x >> 5] = d; warp_kept[threadIdx.x >> 5] = k; warp_total[threadIdx.x >> 5] = tt; }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // this thread's shared-memory writes, for the bulk stores
    __syncthreads();
    if (threadIdx.x == 0) {
        const uint32_t b4 = units * kUnitElems * 4u, b2 = units * kUnitElems * 2u;
        bulk_store(t.w + e0, smem_addr(tile.w), b4);
        bulk_store(t.m + e0, smem_addr(tile.m), b4);
        bulk_store(t.v + e0, smem_addr(tile.v), b4);
        if constexpr (Cfg::compressed) bulk_store(t.w_fwd + e0 / 2, smem_addr(tile.g), b2 / 2);      // units are a multiple of 4: 16-byte sizes
        else bulk_store(t.w_fwd + e0, smem_addr(tile.g), b2);
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        if constexpr (Cfg::count_flips) {
            unsigned long long total = 0;
#pragma unroll
            for (int i = 0; i < kThreads / 32; ++i) total += warp_flips[i];
            if (total) atomicAdd(flip_count, total);
        }
        if constexpr (Cfg::stats) {
            unsigned long long d = 0;
            double k = 0.0, tt = 0.0;
#pragma unroll
            for (int i = 0; i < kThreads / 32; ++i) { d += warp_diff[i]; k += warp_kept[i]; tt += warp_total[i]; }
            MaskStats* slot = stats + (blockIdx.x & (kStatSlots - 1u));
            if (d) atomicAdd(&slot->mask_diff, d);
            atomicAdd(&slot->kept_abs_sum, k);
            atomicAdd(&slot->total_abs_sum, tt);
        }
        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");      // the shared memory has been read: the CTA may end
    }
}

// Resident CTAs per SM a variant is compiled for (64 or 56 registers per thread; 48 was measured too).  Sustained runs
// are limited by the board's power cap as much as by HBM, and which budget wins depends on the code ptxas makes of each
// variant: measured on the LLaMA2-7B set (ms per step at 8 / 9 / 10 CTAs): select 26.70 / 26.94 / 27.1, select + flips
// 27.2 / 27.5 / 29.8, bitmask 26.76 / 26.82 / 27.06, bitmask + flips 27.2 / 27.4 / 28.7, select + dense 26.65 / 26.77 /
// 26.70, refresh (select + flips + dense) 27.05 / 26.8 / 28.8, stored mask 26.23 / 26.15 / 26.36, 4:8 select 27.0 /
// 26.3 / 29.1, 4:8 select + flips 27.4 / 26.95 / 29.4, 1:4 select + flips 26.6 / 26.4 / 27.2.
template <int M, uint32_t F, bool TF>
constexpr int staged_ctas_per_sm()
{
    constexpr uint32_t refresh = kReselect | kCountFlips | kEmitDense;
    return (TF && (F & kReselect) && F != refresh) ? 8 : 9;
}

template <int M, uint32_t F, bool TF>
__global__ void __launch_bounds__(kThreads, staged_ctas_per_sm<M, F, TF>())
adams_nm_bulk_kernel(const __grid_constant__ TensorDesc t, const __grid_constant__ StepConsts c, unsigned long long* __restrict__ flip_count,
                     unsigned long long* fail_word)
{
    bulk_tile<M, F, TF>(t, c, blockIdx.x * kTileUnits, flip_count, nullptr, fail_word);
}

template <int M, uint32_t F, bool TF>
__global__ void __launch_bounds__(kThreads, staged_ctas_per_sm<M, F, TF>())
adams_nm_multi_bulk_kernel(const __grid_constant__ MultiParams p, const __grid_constant__ StepConsts c,
                           unsigned long long* __restrict__ flip_count, MaskStats* __restrict__ stats, unsigned long long* fail_word)
{
    const uint32_t tile = blockIdx.x;
    uint32_t k = p.hint[tile >> p.hint_shift];
    while (tile >= p.tile_start[k + 1]) ++k;
    bulk_tile<M, F, TF>(p.desc[k], c, (tile - p.tile_start[k]) * kTileUnits, flip_count, stats, fail_word);
}

template <int M, uint32_t F, bool TF>
int launch_bulk_t(const StepLaunch& a)
{
    if (a.single) {
        if constexpr ((F & kMaskStats) != 0) return CAST_ERR_NM;      // the statistics epilogue exists for plans only
        else adams_nm_bulk_kernel<M, F, TF><<<tiles_of(*a.single), kThreads, 0, a.stream>>>(*a.single, *a.c, a.flip_count, a.fail_word);
    } else {
        adams_nm_multi_bulk_kernel<M, F, TF><<<a.multi->tile_start[a.multi->n_tensors], kThreads, 0, a.stream>>>(
            *a.multi, *a.c, a.flip_count, a.stats, a.fail_word);
    }
    CAST_CUDA_TRY(cudaGetLastError());
    return CAST_OK;
}

// The configurations the staged form is built for: the steps of training and of the listed workloads.
//   2:4:      select (index or bitmask form), with flips, with dense emission; stored mask with pruned / dense emission
//   general N:M in groups of 4 or 8 (4:8, 1:4, ...): select, with flips (bitmask form)
//   2:4 also: compressed emission with index-form metadata
//   2:4 also: the stored-mask step with the statistics epilogue (26.6 against 27.65 ms plain)
// (measured in this form too and faster plain: the refresh step with the statistics epilogue, 27.6 against 26.8 ms per 7B
//  step, and the steps with the scale gradient, refresh 28.2 against 26.85 ms)
constexpr uint32_t RS = kReselect, FL = kCountFlips, BM = kMetaBitmask, DN = kEmitDense, CP = kEmitCompressed, ST = kMaskStats;
#define CAST_BULK_CASES_2OF4(X) X(4, RS, true) X(4, RS | FL, true) X(4, RS | BM, true) X(4, RS | BM | FL, true) X(4, RS | DN, true) \
    X(4, RS | FL | DN, true) X(4, 0u, true) X(4, DN, true) X(4, RS | CP, true) X(4, DN | ST, true)
// (groups of 16 and 32 columns were measured in this form too: 31.0 / 33.1 against 26.8 / 27.8 ms on the plain path --
// the sorted keys of the cross-lane merge end up in local memory next to the tile code -- so they stay plain)
#define CAST_BULK_CASES_NM(X) X(4, RS | BM, false) X(4, RS | BM | FL, false) X(8, RS | BM, false) X(8, RS | BM | FL, false)

}  // namespace

bool bulk_variant_exists(int M, int n_keep, uint32_t flag_word)
{
    const bool two_four = M == 4 && n_keep == 2;
#define CAST_X(MM, FF, TT) if (M == MM && two_four == TT && flag_word == (FF)) return true;
    CAST_BULK_CASES_2OF4(CAST_X) CAST_BULK_CASES_NM(CAST_X)
#undef CAST_X
    return false;
}

int launch_bulk(const StepLaunch& a, int M, uint32_t flag_word)
{
    const bool two_four = M == 4 && a.c->n_keep == 2;
#define CAST_X(MM, FF, TT) if (M == MM && two_four == TT && flag_word == (FF)) return launch_bulk_t<MM, FF, TT>(a);
    CAST_BULK_CASES_2OF4(CAST_X) CAST_BULK_CASES_NM(CAST_X)
#undef CAST_X
    return CAST_ERR_NM;
}

}  // namespace cast

extern "C" int cast_bulk_timeout_count(unsigned long long* count_out)
{
    if (!count_out) return CAST_ERR_NULL;
    CAST_CUDA_TRY(cudaMemcpyFromSymbol(count_out, cast::g_bulk_timeouts, sizeof(unsigned long long)));
    return CAST_OK;
}
