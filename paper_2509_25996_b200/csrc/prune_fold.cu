// Final pruning of CAST (Alg. 2, final loop; Alg. 1, last lines): W^ = W (.) M with the scale of Eq. 12 folded
// in, as bf16, in the dense layout (pruned slots +0) or compressed to the kept entries, plus the mask
// metadata.  The mask is chosen now by magnitude (Eq. 6, exactly N per group) or read from stored metadata.
// No optimizer state is touched.  Streaming, HBM-bound: 4 B read, 2 (or 2 N / M) + 1/8 B written per parameter.
//
// Same thread layout as the AdamS step (one unit of 8 columns per thread, one CTA of 128 threads per tile of
// 1024 parameters) and the same selection code.
#include "cast_internal.h"

namespace cast {
namespace {

template <int M>
__global__ void __launch_bounds__(kThreads)
prune_fold_kernel(const float* __restrict__ w, const float* __restrict__ scale, uint32_t seg_magic, uint32_t seg_shift,
                  uint8_t* __restrict__ meta, uint16_t* __restrict__ out, uint32_t n_units, int n_keep, uint32_t flags)
{
    const uint32_t unit = blockIdx.x * kTileUnits + threadIdx.x;
    const bool active = unit < n_units;
    const bool bitmask = (flags & kMetaBitmask) != 0;
    float x[8];
    uint32_t ab[8];
    float a = 1.0f;
    uint32_t stored = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) x[i] = 0.0f;
    if (active) {
        const float4 lo = ld_f4(w + (size_t)unit * kUnitElems), hi = ld_f4(w + (size_t)unit * kUnitElems + 4);
        x[0] = lo.x; x[1] = lo.y; x[2] = lo.z; x[3] = lo.w; x[4] = hi.x; x[5] = hi.y; x[6] = hi.z; x[7] = hi.w;
        if (!(flags & kReselect)) stored = meta[unit];
        if (scale != nullptr) a = __ldg(scale + (uint32_t)(((uint64_t)unit * seg_magic) >> seg_shift));
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) ab[i] = abs_bits(x[i]);
    uint32_t keep;
    if (flags & kReselect) keep = select_by_rank<M>(ab, n_keep);      // uniform branch: all lanes shuffle
    else keep = keep_from_meta_byte(stored, bitmask);
    if (!active) return;
    bool kept[8];
    float f[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        kept[i] = (keep >> i) & 1u;
        f[i] = kept[i] ? a * x[i] : 0.0f;
    }
    const uint4 packed = make_uint4(pack_bf16x2(f[0], f[1]), pack_bf16x2(f[2], f[3]), pack_bf16x2(f[4], f[5]), pack_bf16x2(f[6], f[7]));
    bool compressed = false;
    if constexpr (M <= 8) compressed = (flags & kEmitCompressed) != 0;
    if (compressed) store_kept_values<M>(out, unit, keep, packed, n_keep);
    else *reinterpret_cast<uint4*>(out + (size_t)unit * kUnitElems) = packed;
    meta[unit] = (uint8_t)(bitmask ? keep : (idx2_from_kept(kept) | (idx2_from_kept(kept + 4) << 4)));
}

template <int M>
int launch(const float* w, const float* scale, uint32_t magic, uint32_t shift, uint32_t* meta, uint16_t* out,
           uint32_t n_units, int N, uint32_t flags, cudaStream_t s)
{
    const uint32_t tiles = (n_units + kTileUnits - 1) / kTileUnits;
    prune_fold_kernel<M><<<tiles, kThreads, 0, s>>>(w, scale, magic, shift, (uint8_t*)meta, out, n_units, N, flags);
    CAST_CUDA_TRY(cudaGetLastError());
    count_launch();
    return CAST_OK;
}

}  // namespace
}  // namespace cast

using namespace cast;

extern "C" int cast_prune_fold(const float* w, const float* scale, int scale_groups, uint32_t* meta, cast_bf16* out,
                               int64_t rows, int64_t cols, int N, int M, uint32_t flags, cast_stream_t stream)
{
    if (!w || !meta || !out) return CAST_ERR_NULL;
    if (flags & ~(uint32_t)(CAST_F_RESELECT | CAST_F_META_BITMASK | CAST_F_EMIT_COMPRESSED)) return CAST_ERR_HYPER;
    int rc;
    if ((rc = check_nm_flags(N, M, flags, nullptr)) != CAST_OK) return rc;
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
    cudaStream_t s = (cudaStream_t)stream;
    switch (M) {
        case 2:  return launch<2>(w, scale, d.seg_magic, d.seg_shift, meta, out, d.n_units, N, flags, s);
        case 4:  return launch<4>(w, scale, d.seg_magic, d.seg_shift, meta, out, d.n_units, N, flags, s);
        case 8:  return launch<8>(w, scale, d.seg_magic, d.seg_shift, meta, out, d.n_units, N, flags, s);
        case 16: return launch<16>(w, scale, d.seg_magic, d.seg_shift, meta, out, d.n_units, N, flags, s);
        case 32: return launch<32>(w, scale, d.seg_magic, d.seg_shift, meta, out, d.n_units, N, flags, s);
    }
    return CAST_ERR_NM;
}
