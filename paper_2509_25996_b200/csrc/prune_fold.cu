// Final pruning of CAST (Alg. 2, final loop; Alg. 1, last lines): W^ = W (.) M with the scale of Eq. 12 folded
// in, as bf16, in the dense layout (pruned slots +0) or compressed to the kept entries, plus the mask
// metadata.  The mask is chosen now by magnitude (Eq. 6, exactly N per group) or read from stored metadata.
// No optimizer state is touched.  Streaming, HBM-bound: 4 B read, 2 (or 2 N / M) + 1/8 B written per parameter.
//
// Same unit layout (8 columns per thread and access) and the same selection code as the AdamS step; a CTA of
// 128 threads takes 4 units per thread (4096 parameters); all matrices of a plan go in one grid.
#include <cstring>

#include "cast_internal.h"

namespace cast {

namespace {

// One matrix of a pruning launch, and the tables of the launch (kernel parameter space, like the step's).
struct PruneDesc {
    const float* w;
    const float* scale;
    uint8_t* meta;
    uint16_t* out;
    uint32_t n_units, seg_magic, seg_shift, pad_;
};
struct PruneParams {
    uint32_t n_tensors;
    uint32_t hint_shift;
    uint16_t hint[kHintEntries];
    uint32_t tile_start[kMaxLaunchTensors + 1];
    PruneDesc desc[kMaxLaunchTensors];
};

constexpr int kPruneUnitsPerThread = 4;                               // units a thread handles, loads issued together
constexpr int kPruneTileUnits = kThreads * kPruneUnitsPerThread;      // 512 units = 4096 parameters per CTA

// A CTA of the step moves 28 KB; this pass moves 6 bytes per parameter, so a CTA takes four times the
// parameters (with one unit per thread the grid launched CTAs faster than they could be scheduled).
// The flag word (reselect, metadata form, compressed output) and "N:M is 2:4" are template arguments, as in the
// step: the integer work per parameter (compares, keep bits, index nibbles) is what this kernel is bound by
// besides HBM, so nothing is decided at run time and only what a configuration needs is computed.
template <int M, uint32_t F, bool TF>
__global__ void __launch_bounds__(kThreads)
prune_fold_kernel(const __grid_constant__ PruneParams p, int n_keep)
{
    constexpr bool reselect = (F & kReselect) != 0, bitmask = (F & kMetaBitmask) != 0, compressed = (F & kEmitCompressed) != 0;
    static_assert(TF || bitmask, "index-form metadata is 2:4 only");
    static_assert(!compressed || M <= 8, "the compressed form needs the group in one thread");
    const uint32_t tile = blockIdx.x;
    uint32_t k = p.hint[tile >> p.hint_shift];
    while (tile >= p.tile_start[k + 1]) ++k;
    const PruneDesc& t = p.desc[k];
    const uint32_t first = (tile - p.tile_start[k]) * kPruneTileUnits + threadIdx.x;
    float x[kPruneUnitsPerThread][8];
    float a[kPruneUnitsPerThread];
    uint32_t stored[kPruneUnitsPerThread];
#pragma unroll
    for (int j = 0; j < kPruneUnitsPerThread; ++j) {
        const uint32_t unit = first + j * kThreads;
        a[j] = 1.0f;
        stored[j] = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) x[j][i] = 0.0f;
        if (unit < t.n_units) {
            const float4 lo = ld_f4(t.w + (size_t)unit * kUnitElems), hi = ld_f4(t.w + (size_t)unit * kUnitElems + 4);
            x[j][0] = lo.x; x[j][1] = lo.y; x[j][2] = lo.z; x[j][3] = lo.w; x[j][4] = hi.x; x[j][5] = hi.y; x[j][6] = hi.z; x[j][7] = hi.w;
            if constexpr (!reselect) stored[j] = t.meta[unit];
            if (t.scale != nullptr) a[j] = __ldg(t.scale + (uint32_t)(((uint64_t)unit * t.seg_magic) >> t.seg_shift));
        }
    }
#pragma unroll
    for (int j = 0; j < kPruneUnitsPerThread; ++j) {
        const uint32_t unit = first + j * kThreads;
        const bool active = unit < t.n_units;
        bool kept[8];
        uint32_t keep = 0, meta_byte;
        if constexpr (reselect && TF) {                                           // the predicate network of the step
            uint32_t ab[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) ab[i] = abs_bits(x[j][i]);
            select_2of4(ab, kept);
            select_2of4(ab + 4, kept + 4);
            if constexpr (bitmask) {
#pragma unroll
                for (int i = 0; i < 8; ++i) keep |= (kept[i] ? 1u : 0u) << i;
                meta_byte = keep;
            } else {
                meta_byte = idx2_from_kept(kept) | (idx2_from_kept(kept + 4) << 4);   // kept positions, lo | hi << 2 per group
            }
        } else {
            if constexpr (reselect) {
                uint32_t ab[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) ab[i] = abs_bits(x[j][i]);
                keep = select_top_n<M>(ab, n_keep);                               // all lanes shuffle for M > 8
                meta_byte = keep;
            } else {
                keep = keep_from_meta_byte(stored[j], bitmask);
                meta_byte = stored[j];
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) kept[i] = (keep >> i) & 1u;
        }
        if (!active) continue;
        float f[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) f[i] = (kept[i] || compressed) ? a[j] * x[j][i] : 0.0f;      // compressed: the kept ones are picked out below
        const uint4 packed = make_uint4(pack_bf16x2(f[0], f[1]), pack_bf16x2(f[2], f[3]), pack_bf16x2(f[4], f[5]), pack_bf16x2(f[6], f[7]));
        if constexpr (!compressed) {
            *reinterpret_cast<uint4*>(t.out + (size_t)unit * kUnitElems) = packed;
        } else if constexpr (TF && !bitmask) {
            *reinterpret_cast<uint2*>(t.out + (size_t)unit * 4) =
                make_uint2(kept_pair_by_index(packed.x, packed.y, meta_byte & 3u, (meta_byte >> 2) & 3u),
                           kept_pair_by_index(packed.z, packed.w, (meta_byte >> 4) & 3u, meta_byte >> 6));
        } else if constexpr (TF) {
            *reinterpret_cast<uint2*>(t.out + (size_t)unit * 4) =
                make_uint2(kept_pair_2of4(packed.x, packed.y, meta_byte & 0xFu), kept_pair_2of4(packed.z, packed.w, meta_byte >> 4));
        } else {
            store_kept_values<M>(t.out, unit, keep, packed, n_keep);
        }
        t.meta[unit] = (uint8_t)meta_byte;
    }
}

inline uint32_t prune_tiles(uint32_t n_units) { return (n_units + kPruneTileUnits - 1) / kPruneTileUnits; }

template <int M, uint32_t F, bool TF>
int launch_f(const PruneParams& p, int N, cudaStream_t s)
{
    prune_fold_kernel<M, F, TF><<<p.tile_start[p.n_tensors], kThreads, 0, s>>>(p, N);
    CAST_CUDA_TRY(cudaGetLastError());
    count_launch();
    return CAST_OK;
}

// Picks the instantiation of (flags, 2:4 or not) for one group size.
template <int M>
int launch_t(const PruneParams& p, int N, uint32_t flags, cudaStream_t s)
{
    constexpr uint32_t RS = kReselect, BM = kMetaBitmask, CP = kEmitCompressed;
    const bool two_four = M == 4 && N == 2;
    if constexpr (M == 4) {
        if (two_four) {
            switch (flags) {
                case 0u:           return launch_f<4, 0u, true>(p, N, s);
                case RS:           return launch_f<4, RS, true>(p, N, s);
                case BM:           return launch_f<4, BM, true>(p, N, s);
                case RS | BM:      return launch_f<4, RS | BM, true>(p, N, s);
                case CP:           return launch_f<4, CP, true>(p, N, s);
                case RS | CP:      return launch_f<4, RS | CP, true>(p, N, s);
                case BM | CP:      return launch_f<4, BM | CP, true>(p, N, s);
                case RS | BM | CP: return launch_f<4, RS | BM | CP, true>(p, N, s);
            }
            return CAST_ERR_HYPER;
        }
    }
    switch (flags) {
        case BM:           return launch_f<M, BM, false>(p, N, s);
        case RS | BM:      return launch_f<M, RS | BM, false>(p, N, s);
    }
    if constexpr (M <= 8) {
        switch (flags) {
            case BM | CP:      return launch_f<M, BM | CP, false>(p, N, s);
            case RS | BM | CP: return launch_f<M, RS | BM | CP, false>(p, N, s);
        }
    }
    return CAST_ERR_NM;
}

int launch(PruneParams* p, int N, int M, uint32_t flags, cudaStream_t s)
{
    fill_hint_table(p->n_tensors, p->tile_start, p->hint, &p->hint_shift);
    if (p->tile_start[p->n_tensors] == 0) return CAST_OK;
    switch (M) {
        case 2:  return launch_t<2>(*p, N, flags, s);
        case 4:  return launch_t<4>(*p, N, flags, s);
        case 8:  return launch_t<8>(*p, N, flags, s);
        case 16: return launch_t<16>(*p, N, flags, s);
        case 32: return launch_t<32>(*p, N, flags, s);
    }
    return CAST_ERR_NM;
}

int check_prune_flags(int N, int M, uint32_t flags)
{
    if (flags & ~(uint32_t)(CAST_F_RESELECT | CAST_F_META_BITMASK | CAST_F_EMIT_COMPRESSED)) return CAST_ERR_HYPER;
    return check_nm_flags(N, M, flags, nullptr);
}

}  // namespace
}  // namespace cast

using namespace cast;

extern "C" int cast_prune_fold(const float* w, const float* scale, int scale_groups, uint32_t* meta, cast_bf16* out,
                               int64_t rows, int64_t cols, int N, int M, uint32_t flags, cast_stream_t stream)
{
    if (!w || !meta || !out) return CAST_ERR_NULL;
    int rc;
    if ((rc = check_prune_flags(N, M, flags)) != CAST_OK) return rc;
    if ((rc = check_shape(rows, cols, M, scale != nullptr, scale_groups)) != CAST_OK) return rc;
    const uint64_t P = (uint64_t)rows * (uint64_t)cols;
    const uint64_t out_bytes = 2 * fwd_elems_of(rows, cols, N, M, flags);
    const void* ptrs[4] = {w, meta, out, scale};
    const uint64_t bytes[4] = {4 * P, P / 8, out_bytes, scale ? 4ull * (uint64_t)rows * (uint64_t)scale_groups : 0};
    for (int i = 0; i < 4; ++i) {
        if (ptrs[i] && ((uintptr_t)ptrs[i] & 15u)) return CAST_ERR_ALIGN;
        for (int j = i + 1; j < 4; ++j)
            if (ptrs[i] && ptrs[j] && (uintptr_t)ptrs[i] < (uintptr_t)ptrs[j] + bytes[j] && (uintptr_t)ptrs[j] < (uintptr_t)ptrs[i] + bytes[i])
                return CAST_ERR_ALIAS;
    }
    if ((rc = check_device_memory(ptrs, 4)) != CAST_OK) return rc;
    const TensorDesc d = make_desc(nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, scale, scale_groups, rows, cols);
    PruneParams p;
    std::memset(&p, 0, sizeof p);
    p.n_tensors = 1;
    p.desc[0] = PruneDesc{w, scale, (uint8_t*)meta, out, d.n_units, d.seg_magic, d.seg_shift, 0};
    p.tile_start[1] = prune_tiles(d.n_units);
    return launch(&p, N, M, flags, (cudaStream_t)stream);
}

extern "C" int cast_plan_prune_fold(void* plan, cast_bf16* const* out, uint32_t flags, cast_stream_t stream)
{
    const int n = plan_tensor_count(plan);
    if (n < 0) return CAST_ERR_PLAN;
    if (!out) return CAST_ERR_NULL;
    int N = 0, M = 0, rc;
    TensorDesc d;
    plan_tensor_desc(plan, 0, &N, &M, &d);
    if ((rc = check_prune_flags(N, M, flags)) != CAST_OK) return rc;
    for (int i = 0; i < n; ++i) {
        if (!out[i]) return CAST_ERR_NULL;
        if ((uintptr_t)out[i] & 15u) return CAST_ERR_ALIGN;
        plan_tensor_desc(plan, i, &N, &M, &d);
        const uint64_t P = (uint64_t)d.n_units * kUnitElems;
        const uint64_t ob = 2 * ((flags & CAST_F_EMIT_COMPRESSED) ? P / (uint64_t)M * (uint64_t)N : P);
        const uintptr_t o = (uintptr_t)out[i];
        if ((o < (uintptr_t)d.w + 4 * P && (uintptr_t)d.w < o + ob) || (o < (uintptr_t)d.meta + P / 8 && (uintptr_t)d.meta < o + ob))
            return CAST_ERR_ALIAS;
        const void* op[1] = {out[i]};
        if ((rc = check_device_memory(op, 1)) != CAST_OK) return rc;
    }
    int i = 0;
    while (i < n) {
        PruneParams p;
        std::memset(&p, 0, sizeof p);
        uint64_t tiles = 0;
        while (i < n && p.n_tensors < (uint32_t)kMaxLaunchTensors) {
            plan_tensor_desc(plan, i, &N, &M, &d);
            p.desc[p.n_tensors] = PruneDesc{d.w, d.scale, (uint8_t*)d.meta, out[i], d.n_units, d.seg_magic, d.seg_shift, 0};
            p.tile_start[p.n_tensors] = (uint32_t)tiles;
            tiles += prune_tiles(d.n_units);
            ++p.n_tensors;
            ++i;
        }
        p.tile_start[p.n_tensors] = (uint32_t)tiles;
        if ((rc = launch(&p, N, M, flags, (cudaStream_t)stream)) != CAST_OK) return rc;
    }
    return CAST_OK;
}
