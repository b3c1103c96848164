// Host-side helpers shared by the entry points of the library (not part of the public ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/cast_adams.h"
#include "adams_kernel.cuh"

namespace cast {

// Remember a failed CUDA call for cast_last_cuda_error() and return CAST_ERR_CUDA.
int cuda_failed(cudaError_t e);

#define CAST_CUDA_TRY(expr)                                  \
    do {                                                     \
        cudaError_t cast_e_ = (expr);                        \
        if (cast_e_ != cudaSuccess) return ::cast::cuda_failed(cast_e_); \
    } while (0)

// One more kernel launched (for cast_kernel_launch_count).
void count_launch();

// N:M, flags and the flip counter pointer.
int check_nm_flags(int N, int M, uint32_t flags, const void* flip_count);

// Hyper-parameter ranges; on success fills the folded per-iteration scalars.
int make_step_consts(float lr, float beta1, float beta2, float eps, float l1_coeff,
                     int64_t step, int64_t total_steps, int N, uint32_t flags, StepConsts* out);

// Shape rules of one matrix (does not look at pointers).
int check_shape(int64_t rows, int64_t cols, int M, bool has_scale, int scale_groups);

// Null / alignment / overlap rules of one matrix's pointers (addresses only, never dereferenced).
// `fwd_elems` is the number of bf16 elements of w_fwd (rows*cols, or rows*cols*N/M in compressed form).
int check_pointers(const void* w, const void* m, const void* v, const void* g, const void* w_fwd,
                   const void* meta, const void* scale, int scale_groups, int64_t rows, int64_t cols,
                   uint64_t fwd_elems);

// Elements of the forward-weight buffer of one matrix under `flags`.
inline uint64_t fwd_elems_of(int64_t rows, int64_t cols, int N, int M, uint32_t flags)
{
    const uint64_t P = (uint64_t)rows * (uint64_t)cols;
    return (flags & CAST_F_EMIT_COMPRESSED) ? P / (uint64_t)M * (uint64_t)N : P;
}

// Every given pointer must be device-accessible memory on the current device.
int check_device_memory(const void* const* ptrs, int n);

// Kernel-side description of one (already validated) matrix.
TensorDesc make_desc(float* w, float* m, float* v, const uint16_t* g, uint16_t* w_fwd, uint32_t* meta,
                     const float* scale, int scale_groups, int64_t rows, int64_t cols, float* scale_grad = nullptr,
                     const uint32_t* meta_ref = nullptr, const float* scale_chain = nullptr);

// The optional scale-gradient buffer of one matrix: needs a scale, 16-byte alignment, device memory, no overlap
// with the matrix's other buffers (checked by address only).
int check_scale_grad(const float* scale_grad, const float* scale, int scale_groups, int64_t rows,
                     const void* const* others, const uint64_t* other_bytes, int n_others);

inline uint32_t tiles_of(const TensorDesc& d) { return (d.n_units + kTileUnits - 1) / kTileUnits; }

// One launch of the step: over one matrix (`single`) or over a table of matrices (`multi`), both passed by value
// as kernel parameters.  The kernel is picked by M, N and the compile-time part of c->flags.
struct StepLaunch {
    const TensorDesc* single;
    const MultiParams* multi;
    const StepConsts* c;
    unsigned long long* flip_count;
    MaskStats* stats;                 // the plan's kStatSlots accumulators, or nullptr
    cudaStream_t stream;
    unsigned long long* fail_word;    // host memory the staged kernels report a copy they gave up on to, or nullptr
    bool prefer_staged;               // no access path was asked for: take the staged one where it is built
};
int launch_single(const TensorDesc& d, int M, const StepConsts& c, unsigned long long* flip_count, cudaStream_t stream);
int launch_multi(const MultiParams& p, int M, const StepConsts& c, unsigned long long* flip_count, cudaStream_t stream,
                 MaskStats* stat_slots = nullptr, unsigned long long* fail_word = nullptr);

// Fill the tile-to-matrix hint table (kHintEntries entries) of a launch whose tile_start[0..n_tensors] is set:
// hint[b] = the matrix that holds tile b << *hint_shift.
void fill_hint_table(uint32_t n_tensors, const uint32_t* tile_start, uint16_t* hint, uint32_t* hint_shift);
inline void fill_hints(MultiParams* p) { fill_hint_table(p->n_tensors, p->tile_start, p->hint, &p->hint_shift); }

// Host-side view of a plan (for the entry points that work on a plan's matrices).
int plan_tensor_count(const void* plan);
bool plan_tensor_desc(const void* plan, int i, int* N, int* M, TensorDesc* desc);

// A grid holds at most this many tiles (one CTA per tile, gridDim.x < 2^31).
constexpr uint64_t kMaxTiles = 0x7FFFFFFFull;

}  // namespace cast
