// Measurement aids (no arithmetic of the method): kernels with the launch shape and the memory access pattern of
// the AdamS step and nothing else, so that a benchmark can put two floors beside a measured step:
//   cast_probe_launch   an empty grid of n_ctas CTAs of 128 threads: what launching and draining that many CTAs costs;
//   cast_probe_stream   the step's loads and stores (two 128-bit accesses per fp32 array and one per bf16 array per
//                       thread, one metadata byte, one CTA of 128 threads per 1024 parameters) with one bit flip per
//                       word between them: the rate at which this device streams 28.125 bytes per parameter in
//                       exactly that pattern.
#include "cast_internal.h"

namespace cast {
namespace {

__global__ void __launch_bounds__(kThreads, kMinCtasPerSm) probe_empty_kernel() {}

// w, m, v are rewritten in place with their sign bits flipped (so that the stores cannot be dropped), the gradient
// goes out as the forward weight, and a metadata byte is written per unit.
__global__ void __launch_bounds__(kThreads, kMinCtasPerSm)
probe_stream_kernel(float* __restrict__ w, float* __restrict__ m, float* __restrict__ v, const uint16_t* __restrict__ g,
                    uint16_t* __restrict__ w_fwd, uint8_t* __restrict__ meta, uint32_t n_units)
{
    const uint32_t unit = blockIdx.x * kTileUnits + threadIdx.x;
    if (unit >= n_units) return;
    const size_t e = (size_t)unit * kUnitElems;
    float4 a[6] = {ld_f4(w + e), ld_f4(w + e + 4), ld_f4(m + e), ld_f4(m + e + 4), ld_f4(v + e), ld_f4(v + e + 4)};
    const uint4 gg = *reinterpret_cast<const uint4*>(g + e);
#pragma unroll
    for (int i = 0; i < 6; ++i) {
        a[i].x = -a[i].x; a[i].y = -a[i].y; a[i].z = -a[i].z; a[i].w = -a[i].w;
    }
    st_f4(w + e, a[0]); st_f4(w + e + 4, a[1]);
    st_f4(m + e, a[2]); st_f4(m + e + 4, a[3]);
    st_f4(v + e, a[4]); st_f4(v + e + 4, a[5]);
    *reinterpret_cast<uint4*>(w_fwd + e) = gg;
    meta[unit] = (uint8_t)(gg.x ^ gg.w);
}

}  // namespace
}  // namespace cast

using namespace cast;

extern "C" int cast_probe_launch(int64_t n_ctas, cast_stream_t stream)
{
    if (n_ctas < 1 || (uint64_t)n_ctas > kMaxTiles) return CAST_ERR_SHAPE;
    probe_empty_kernel<<<(unsigned)n_ctas, kThreads, 0, (cudaStream_t)stream>>>();
    CAST_CUDA_TRY(cudaGetLastError());
    count_launch();
    return CAST_OK;
}

extern "C" int cast_probe_stream(float* w, float* m, float* v, const cast_bf16* g, cast_bf16* w_fwd, uint32_t* meta,
                                 int64_t n_params, cast_stream_t stream)
{
    if (!w || !m || !v || !g || !w_fwd || !meta) return CAST_ERR_NULL;
    if (n_params < 32 || n_params % 32 != 0 || n_params > 0x7FFFFFFF) return CAST_ERR_SHAPE;
    int rc;
    if ((rc = check_pointers(w, m, v, g, w_fwd, meta, nullptr, 1, 1, n_params, (uint64_t)n_params)) != CAST_OK) return rc;
    const void* ptrs[6] = {w, m, v, g, w_fwd, meta};
    if ((rc = check_device_memory(ptrs, 6)) != CAST_OK) return rc;
    const uint32_t n_units = (uint32_t)(n_params / kUnitElems);
    probe_stream_kernel<<<(n_units + kTileUnits - 1) / kTileUnits, kThreads, 0, (cudaStream_t)stream>>>(
        w, m, v, g, w_fwd, reinterpret_cast<uint8_t*>(meta), n_units);
    CAST_CUDA_TRY(cudaGetLastError());
    count_launch();
    return CAST_OK;
}
