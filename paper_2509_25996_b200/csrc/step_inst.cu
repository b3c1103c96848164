// Instantiations of the AdamS step kernels.  This file is compiled once per slice (group size M, 2:4 or not,
// with or without the statistics epilogue, literal or alternate reading of Eq. 8; see build_ext.py), each time with
// every valid compile-time flag word of the slice, so that no combination of flags is decided inside a kernel and
// the compilation runs in parallel.  Every object exports one function,
// launch_step_m<M>_tf<0|1>_s<0|1>_v<0|1>(flag_word, launch).
#include <utility>

#include "cast_internal.h"

#ifndef CAST_INST_M          // defaults, so that the file also compiles on its own
#define CAST_INST_M 4
#define CAST_INST_TF 1
#define CAST_INST_STATS 0
#define CAST_INST_V 0
#endif

#define CAST_CAT_(a, b, c, d, e, f, g, h) a##b##c##d##e##f##g##h
#define CAST_CAT(a, b, c, d, e, f, g, h) CAST_CAT_(a, b, c, d, e, f, g, h)
#define CAST_INST_FN CAST_CAT(launch_step_m, CAST_INST_M, _tf, CAST_INST_TF, _s, CAST_INST_STATS, _v, CAST_INST_V)

namespace cast {
namespace {

constexpr int kM = CAST_INST_M;
constexpr bool kTwoFour = CAST_INST_TF != 0;
constexpr bool kStats = CAST_INST_STATS != 0;
constexpr bool kAltV = CAST_INST_V != 0;

template <uint32_t F>
int launch_word(const StepLaunch& a)
{
    if (a.single) {
        // one CTA per tile: the hardware scheduler hands tiles out in address order
        if constexpr (kStats) return CAST_ERR_NM;      // the statistics epilogue exists for plans only
        else adams_nm_kernel<kM, F, kTwoFour><<<tiles_of(*a.single), kThreads, 0, a.stream>>>(*a.single, *a.c, a.flip_count, a.stats);
    } else {
        adams_nm_multi_kernel<kM, F, kTwoFour><<<a.multi->tile_start[a.multi->n_tensors], kThreads, 0, a.stream>>>(
            *a.multi, *a.c, a.flip_count, a.stats);
    }
    CAST_CUDA_TRY(cudaGetLastError());
    return CAST_OK;
}

// Tries one flag word: launches its kernel if it is the one asked for.
template <uint32_t F>
bool try_word(uint32_t flag_word, const StepLaunch& a, int& rc)
{
    if constexpr (((F & kMaskStats) != 0) == kStats && ((F & kVKeptFromG) != 0) == kAltV && step_kernel_exists(kM, kTwoFour, F)) {
        if (flag_word == F) {
            rc = launch_word<F>(a);
            return true;
        }
    }
    return false;
}

// Walks all flag words at compile time.
template <uint32_t... Fs>
int walk(uint32_t flag_word, const StepLaunch& a, std::integer_sequence<uint32_t, Fs...>)
{
    int rc = CAST_ERR_NM;
    (void)(try_word<Fs>(flag_word, a, rc) || ...);
    return rc;
}

}  // namespace

int CAST_INST_FN(uint32_t flag_word, const StepLaunch& a)
{
    return walk(flag_word, a, std::make_integer_sequence<uint32_t, kFlagWords>{});
}

}  // namespace cast
