// Device code of the fused AdamS N:M step (CAST, arxiv 2509.25996: Alg. 1, Eq. 6-8, Eq. 12).
//
// Streaming kernel, HBM-bound: 14 B read and 14.125 B written per parameter.  One thread owns
// a "unit" of 8 consecutive columns (32 B of each fp32 array, 16 B of each bf16 array, one
// metadata byte), so every group of M <= 8 columns lives in one thread's registers and the
// top-N selection is a register-only comparison network; groups of 16 or 32 columns are shared
// by 2 or 4 neighbouring lanes through warp shuffles.  A warp covers 256 consecutive parameters:
// 1 KB of each fp32 array, 512 B of each bf16 array and one 32-byte sector of metadata.
//
// Launch shape: one CTA of 128 threads per tile of 1024 parameters, one unit per thread, no loop.
// Measured on B200, small short-lived CTAs (7 resident per SM, the hardware scheduler handing out
// tiles in address order) stream faster than a persistent grid-stride loop of the same body, and as
// fast with 128-bit as with 256-bit accesses.  This file holds the arithmetic (compute_unit) and the
// kernels of the plain access path (per-thread loads and stores); bulk_step.cu wraps the same
// compute_unit in the staged path (the tile moved by bulk asynchronous copies through shared memory),
// which is as fast in short runs and 2-7 % faster in sustained ones.
//
// Instruction budget: at ~6.8 TB/s an SM retires ~0.85 parameters per clock, so the body has to stay
// well under ~100 thread instructions per parameter or instruction issue (and, under the board's
// power cap, the SM clock) becomes the limit.  Hence: the flag word is a compile-time constant of the
// kernel (one instantiation per valid combination of selection, metadata form, emission, flip counting,
// scale gradient and statistics), the 2:4 selection is six comparisons and four 3-input predicate
// functions per group, and the update uses the approximate reciprocal and square root units (error
// analysis below).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace cast {

constexpr int kThreads = 128;          // threads per CTA
constexpr int kUnitElems = 8;          // parameters per thread
constexpr int kTileUnits = kThreads;   // units per tile (1024 parameters)
constexpr int kMinCtasPerSm = 7;       // register budget most kernels are compiled for (plain_ctas_per_sm below)

// flag bits (values of the public header)
constexpr uint32_t kReselect = 1u << 0;
constexpr uint32_t kCountFlips = 1u << 1;
constexpr uint32_t kMetaBitmask = 1u << 2;
constexpr uint32_t kVKeptFromG = 1u << 3;
constexpr uint32_t kEmitDense = 1u << 4;
constexpr uint32_t kEmitCompressed = 1u << 5;
constexpr uint32_t kGradOfScaled = 1u << 6;
constexpr uint32_t kMaskStats = 1u << 7;

// Every flag is a template argument of the kernels (even the alternate reading of Eq. 8, one select per parameter,
// cost 1.4 % of the headline step when it was read at run time).
constexpr uint32_t kCompileTimeFlags = kReselect | kCountFlips | kMetaBitmask | kVKeptFromG | kEmitDense | kEmitCompressed |
                                       kGradOfScaled | kMaskStats;
constexpr uint32_t kFlagWords = 256;   // compile-time flag words live in [0, kFlagWords)

// Which (M, two_four, flag word) combinations are instantiated.  `two_four` says N == 2 and M == 4: the kept set
// comes from the comparison network, the metadata may be in index form and the compressed form is two byte
// permutes.  The host normalises a flag word before it looks for its kernel: kCountFlips is dropped without
// kReselect (a reused mask has no flips).
__host__ __device__ constexpr bool step_kernel_exists(int M, bool two_four, uint32_t f)
{
    if (f & ~kCompileTimeFlags) return false;
    if ((f & kCountFlips) && !(f & kReselect)) return false;
    if ((f & kEmitDense) && (f & kEmitCompressed)) return false;
    if ((f & kEmitCompressed) && M > kUnitElems) return false;
    if (two_four && M != 4) return false;
    if (!two_four && !(f & kMetaBitmask)) return false;      // index-form metadata is 2:4 only
    return true;
}

// One matrix as the kernel sees it.
struct TensorDesc {
    float* w;
    float* m;
    float* v;
    const uint16_t* g;
    uint16_t* w_fwd;
    uint32_t* meta;
    const float* scale;        // A[rows][n] or nullptr
    float* scale_grad;         // dL/dA[rows][n], added to, or nullptr
    const uint8_t* meta_ref;   // reference mask of the statistics (same form as meta), or nullptr
    const float* scale_chain;  // A the forward pass that produced g was scaled with (`scale` itself where the caller gave none)
    uint32_t n_units;          // rows * cols / 8
    uint32_t seg_magic;        // unit / seg_units == (uint64(unit) * seg_magic) >> seg_shift
    uint32_t seg_shift;
    uint32_t pad_;
};

// Scalars of one iteration, folded on the host in double precision.
struct StepConsts {
    double beta1;       // beta1
    double omb1;        // 1 - beta1
    double c_mu;        // 1 - alpha_t                  (Eq. 7)
    double c_sign;      // alpha_t * lambda             (Eq. 7)
    float beta2;        // beta2
    float omb2;         // 1 - beta2
    float inv_bc2_s;    // 2^64 / (1 - beta2^t)        the update runs on sqrt(v^) and eps scaled by 2^32 (see
    float lr_bc1_s;     // 2^32 lr / (1 - beta1^t)      update_term), so that the flushing sqrt/rcp units never
    float eps_s;        // 2^32 eps                     see a subnormal
    int32_t n_keep;     // N
    uint32_t flags;
};

__device__ __forceinline__ float4 ld_f4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ void st_f4(float* p, float4 x) { *reinterpret_cast<float4*>(p) = x; }

// Approximate units: sqrt.approx.ftz.f32 has a maximum relative error of 2^-23 over the positive normal range,
// rcp.approx.ftz.f32 of 1 ulp (PTX ISA); both are single instructions and flush subnormals to zero.
__device__ __forceinline__ float sqrt_approx_ftz(float x) { float r; asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x)); return r; }
__device__ __forceinline__ float rcp_approx_ftz(float x) { float r; asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x)); return r; }

// lr mu^ / (sqrt(v^) + eps) with numerator and denominator both scaled by 2^32 (exact, powers of two):
//   sqrt(2^64 v^) = 2^32 sqrt(v^)  -- a subnormal v (down to 2^-149) becomes normal before the flushing sqrt;
//   2^32 eps is normal for every positive float eps, so the denominator and its reciprocal are normal too
//   (the reciprocal would only be flushed for v^ > 2^188, where the true update is below 1e-28 anyway).
__device__ __forceinline__ float update_term(float mu_t, float v_new, const StepConsts& c)
{
    return (c.lr_bc1_s * mu_t) * rcp_approx_ftz(sqrt_approx_ftz(v_new * c.inv_bc2_s) + c.eps_s);
}

// |w| as an integer: for non-NaN floats the bit pattern without the sign orders exactly like the
// absolute value, and -0 equals +0.
__device__ __forceinline__ uint32_t abs_bits(float x) { return __float_as_uint(x) & 0x7FFFFFFFu; }

// Order inside a group (Eq. 6 with exactly N kept, Eq. 4): larger |w| first, lower column first
// among equal magnitudes.  Column j (< k) comes before column k iff a[j] >= a[k].

// 2:4: a column is kept iff at least two of the other three do not come before it.
__device__ __forceinline__ bool at_least_two(bool x, bool y, bool z) { return (x && y) || (x && z) || (y && z); }
__device__ __forceinline__ void select_2of4(const uint32_t* a, bool* kept)
{
    const bool c01 = a[0] >= a[1], c02 = a[0] >= a[2], c03 = a[0] >= a[3];
    const bool c12 = a[1] >= a[2], c13 = a[1] >= a[3], c23 = a[2] >= a[3];
    kept[0] = at_least_two(c01, c02, c03);
    kept[1] = at_least_two(!c01, c12, c13);
    kept[2] = at_least_two(!c02, !c12, c23);
    kept[3] = at_least_two(!c03, !c13, !c23);
}

// General N:M, M <= 8 (the group lives in this thread): rank of a column = how many columns of its group come
// before it; kept iff rank < N.  Returns the keep mask of the unit (bit j = column j of the unit is kept).
template <int M>
__device__ __forceinline__ uint32_t select_by_rank(const uint32_t (&a)[8], int n_keep)
{
    static_assert(M <= 8, "wider groups are shared by lanes: select_wide");
    int rank[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) rank[i] = 0;
#pragma unroll
    for (int base = 0; base < 8; base += M) {
#pragma unroll
        for (int j = 0; j < M; ++j) {
#pragma unroll
            for (int k = j + 1; k < M; ++k) {
                const bool j_first = a[base + j] >= a[base + k];
                rank[base + k] += j_first ? 1 : 0;
                rank[base + j] += j_first ? 0 : 1;
            }
        }
    }
    uint32_t keep = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) keep |= (rank[i] < n_keep ? 1u : 0u) << i;
    return keep;
}

// Groups of 16 or 32 columns are shared by L = 2 or 4 neighbouring lanes (8 columns each, lower lane = lower
// columns).  The kept set is {|w| > tau} plus, among the columns with |w| == tau in column order, as many as
// are still missing to N, where tau is the N-th largest magnitude of the group -- the same set as "rank < N"
// under the order of Eq. 6 used everywhere else.  tau comes from a bitonic sort of the group's 31-bit keys
// (minimum / maximum instructions only, no indices carried): each lane sorts its 8 keys with a 19-exchange
// network, pairs of lanes merge (exchange against the partner's reversed run, then a local 12-exchange bitonic
// merge), and for L = 4 the two sorted 16-runs merge the same way across lanes.  All lanes of the warp call this.
__device__ __forceinline__ void exchange_desc(uint32_t& first, uint32_t& second)
{
    const uint32_t hi = max(first, second), lo = min(first, second);
    first = hi;
    second = lo;
}
__device__ __forceinline__ void sort8_desc(uint32_t (&s)[8])
{
    exchange_desc(s[0], s[1]); exchange_desc(s[2], s[3]); exchange_desc(s[4], s[5]); exchange_desc(s[6], s[7]);
    exchange_desc(s[0], s[2]); exchange_desc(s[1], s[3]); exchange_desc(s[4], s[6]); exchange_desc(s[5], s[7]);
    exchange_desc(s[1], s[2]); exchange_desc(s[5], s[6]); exchange_desc(s[0], s[4]); exchange_desc(s[3], s[7]);
    exchange_desc(s[1], s[5]); exchange_desc(s[2], s[6]);
    exchange_desc(s[1], s[4]); exchange_desc(s[3], s[6]);
    exchange_desc(s[2], s[4]); exchange_desc(s[3], s[5]);
    exchange_desc(s[3], s[4]);
}
__device__ __forceinline__ void bitonic_merge8_desc(uint32_t (&s)[8])
{
#pragma unroll
    for (int d = 4; d > 0; d >>= 1)
#pragma unroll
        for (int i = 0; i < 8; ++i)
            if (!(i & d)) exchange_desc(s[i], s[i + d]);
}
// One cross-lane step of a bitonic merge: every key meets the key `REVERSED ? 7 - i : i` of lane ^ d; the lane
// on the `upper` side keeps the smaller one, the other the larger one.
template <bool REVERSED>
__device__ __forceinline__ void exchange_lanes_desc(uint32_t (&s)[8], int d, bool upper)
{
    uint32_t r[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) r[i] = __shfl_xor_sync(0xFFFFFFFFu, s[REVERSED ? 7 - i : i], d);
#pragma unroll
    for (int i = 0; i < 8; ++i) s[i] = upper ? min(s[i], r[i]) : max(s[i], r[i]);
}

template <int M>
__device__ __forceinline__ uint32_t select_wide(const uint32_t (&a)[8], int n_keep)
{
    static_assert(M == 16 || M == 32, "groups of 16 or 32 columns");
    constexpr unsigned L = M / 8;
    const unsigned lane = threadIdx.x & 31u;
    const unsigned pos = lane & (L - 1u);                  // this lane's place in its group
    uint32_t s[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) s[i] = a[i];
    sort8_desc(s);
    exchange_lanes_desc<true>(s, 1, (pos & 1u) != 0);      // two sorted 8-runs -> upper / lower half of 16
    bitonic_merge8_desc(s);
    if constexpr (L == 4) {
        exchange_lanes_desc<true>(s, 3, (pos & 2u) != 0);  // two sorted 16-runs -> upper / lower half of 32
        exchange_lanes_desc<false>(s, 1, (pos & 1u) != 0);
        bitonic_merge8_desc(s);
    }
    // the group's keys now stand in descending order across its lanes: place q is s[q & 7] of lane q >> 3
    const int q = n_keep - 1;                              // uniform
    uint32_t cand = s[0];
#pragma unroll
    for (int i = 1; i < 8; ++i) cand = ((q & 7) == i) ? s[i] : cand;
    const uint32_t tau = __shfl_sync(0xFFFFFFFFu, cand, (int)(lane & ~(L - 1u)) + (q >> 3));
    uint32_t gt = 0, eq = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        gt |= (a[i] > tau ? 1u : 0u) << i;
        eq |= (a[i] == tau ? 1u : 0u) << i;
    }
    // columns above tau in the whole group, columns equal to tau in the lower lanes of the group
    int above = __popc(gt);
    const int equal_here = __popc(eq);
    int equal_incl = equal_here;
#pragma unroll
    for (unsigned d = 1; d < L; d <<= 1) {
        above += __shfl_xor_sync(0xFFFFFFFFu, above, (int)d);
        const int up = __shfl_up_sync(0xFFFFFFFFu, equal_incl, d);
        if (pos >= d) equal_incl += up;
    }
    int missing = n_keep - above - (equal_incl - equal_here);      // ties this lane may still keep, in column order
    uint32_t keep = gt;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const bool e = (eq >> i) & 1u;
        keep |= ((e && missing > 0) ? 1u : 0u) << i;
        missing -= e ? 1 : 0;
    }
    return keep;
}

template <int M>
__device__ __forceinline__ uint32_t select_top_n(const uint32_t (&a)[8], int n_keep)
{
    if constexpr (M <= 8) return select_by_rank<M>(a, n_keep);
    else return select_wide<M>(a, n_keep);
}

// 2:4 index form: one nibble per group, lo | hi << 2 with lo < hi the positions of the kept pair.
__device__ __forceinline__ uint32_t idx2_from_kept(const bool* k)
{
    const uint32_t lo = k[0] ? 0u : (k[1] ? 1u : 2u);
    const uint32_t hi = k[3] ? 3u : (k[2] ? 2u : 1u);
    return lo | (hi << 2);
}
__device__ __forceinline__ uint32_t keep_nibble_from_idx2(uint32_t f)
{
    return (1u << (f & 3u)) | (1u << ((f >> 2) & 3u));
}
__device__ __forceinline__ uint32_t keep_from_meta_byte(uint32_t b, bool bitmask)
{
    if (bitmask) return b;
    return keep_nibble_from_idx2(b & 0xFu) | (keep_nibble_from_idx2(b >> 4) << 4);
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));   // round to nearest even
    return r;
}

// Compressed form of the forward weight: only the kept entries, in column order, 8 N / M per unit (M <= 8).
// `packed` holds the unit's 8 bf16 values.  Every group keeps exactly N, so the slot of a kept column is the
// number of kept columns before it in the unit.  The values are scattered into a private 16-byte row of
// shared memory and read back as a vector (16, 8 or 4 bytes; other counts go out as 2-byte stores).
// 2:4: the kept pair of a group (columns lo < hi: two of the four bf16 halves of registers r01, r23) picked by
// one byte permute.  Half h of the register pair is bytes 2h, 2h + 1: selector = (2lo, 2lo + 1, 2hi, 2hi + 1).
__device__ __forceinline__ uint32_t kept_pair_by_index(uint32_t r01, uint32_t r23, uint32_t lo, uint32_t hi)
{
    return __byte_perm(r01, r23, 0x1010u + 0x22u * lo + 0x2200u * hi);
}
__device__ __forceinline__ uint32_t kept_pair_2of4(uint32_t r01, uint32_t r23, uint32_t nibble)   // nibble = keep bits
{
    const uint32_t lo = (nibble & 1u) ? 0u : ((nibble & 2u) ? 1u : 2u);
    const uint32_t hi = (nibble & 8u) ? 3u : ((nibble & 4u) ? 2u : 1u);
    return kept_pair_by_index(r01, r23, lo, hi);
}

template <int M>
__device__ __forceinline__ void store_kept_values(uint16_t* base, uint32_t unit, uint32_t keep, uint4 packed, int n_keep)
{
    __shared__ __align__(16) uint16_t s_comp[kThreads * 8];
    uint16_t* mine = s_comp + threadIdx.x * 8;
    const uint32_t hw[4] = {packed.x, packed.y, packed.z, packed.w};
#pragma unroll
    for (int i = 0; i < 8; ++i)
        if ((keep >> i) & 1u)
            mine[__popc(keep & ((1u << i) - 1u))] = (uint16_t)(hw[i >> 1] >> (16 * (i & 1)));
    const uint32_t cnt = (uint32_t)(8 * n_keep) / (uint32_t)M;
    uint16_t* dst = base + (size_t)unit * cnt;
    if (cnt == 8) *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(mine);
    else if (cnt == 4) *reinterpret_cast<uint2*>(dst) = *reinterpret_cast<const uint2*>(mine);
    else if (cnt == 2) *reinterpret_cast<uint32_t*>(dst) = *reinterpret_cast<const uint32_t*>(mine);
    else
        for (uint32_t k = 0; k < cnt; ++k) dst[k] = mine[k];
}

// Registers of one unit: state and gradient in, updated state, forward weight and metadata out.
struct UnitRegs {
    float w[8], m[8], v[8];
    uint4 g;               // 8 bf16 gradients in; 8 bf16 forward weights out
    uint32_t prev_byte;    // metadata byte of the unit before the step (when it is read)
    uint32_t ref_byte;     // byte of the statistics' reference mask (when there is one)
    uint32_t meta_byte;    // metadata byte after the step
    uint32_t keep;         // keep mask of the unit (bit j = column j kept), where the configuration needs it as bits
};

// What one CTA adds to the caller's counters: flips (App. C, numerator of r_t) and the mask statistics
// (App. C: ||M_t - M_ref||_0, ||W_t (.) M_t||_1, ||W_t||_1 on the updated weights).
struct UnitSums {
    uint32_t flips = 0;
    uint32_t mask_diff = 0;
    double kept_abs = 0.0, total_abs = 0.0;
};

// Device view of the statistics accumulator (layout of cast_mask_stats_t in the public header).  The step kernels
// add to one of kStatSlots such accumulators, picked by the CTA's index: three atomics per CTA from millions of
// CTAs onto ONE 32-byte sector serialise in its L2 slice (about a nanosecond each: 50 instead of 27 ms per step on
// a 6.5 G-parameter model); spread over 1024 sectors they cost nothing measurable.  A one-CTA kernel then folds the
// slots into the caller's accumulator and clears them.
constexpr uint32_t kStatSlots = 1024;
struct MaskStats {
    unsigned long long mask_diff;
    unsigned long long reserved_;
    double kept_abs_sum;
    double total_abs_sum;
};

// Compile-time view of a flag word.
template <int M, uint32_t F, bool TF>
struct StepCfg {
    static_assert(step_kernel_exists(M, TF, F), "no such kernel");
    static constexpr bool reselect = (F & kReselect) != 0;
    static constexpr bool count_flips = (F & kCountFlips) != 0;
    static constexpr bool bitmask = (F & kMetaBitmask) != 0;
    static constexpr bool dense = (F & kEmitDense) != 0;
    static constexpr bool compressed = (F & kEmitCompressed) != 0;
    static constexpr bool of_scaled = (F & kGradOfScaled) != 0;
    static constexpr bool stats = (F & kMaskStats) != 0;
    static constexpr bool v_from_g = (F & kVKeptFromG) != 0;
    static constexpr bool network = TF && reselect;               // kept set from the 2:4 comparison network
    static constexpr bool need_prev = !reselect || count_flips;   // the stored metadata is read
};

// Arithmetic of one unit, registers only (and warp shuffles for M > 8: every lane of the warp must
// call this, lanes without data pass zeros).  `a` is the unit's scale A[r, segment].
//
// Precision.  The first moment and the decayed first moment are sums of terms of opposite sign and
// like size (beta1 m against (1 - beta1) g, (1 - alpha) mu against alpha lambda), so they are formed
// in fp64 from the exact inputs: in fp32 a cancellation leaves mu with a large relative error, which
// the quotient mu / sqrt(v) carries into w wherever v is small as well.  Everything after is a
// product or a sum of like signs and stays in fp32.  The update lr mu^ / (sqrt(v^) + eps) uses the
// approximate square root and reciprocal: its relative error is below ~5e-7 (2^-23 each, plus five
// roundings of 2^-24), i.e. below 2.5e-10 absolute for updates up to 5e-4, which is under both the
// fp32 spacing of typical weights (1.9e-9 at 0.02) and the 1e-9 floor of the accepted error.
template <int M, uint32_t F, bool TF>
__device__ __forceinline__ void compute_unit(UnitRegs& u, const StepConsts& c, float a, bool has_ref, float& gw_sum, UnitSums& sums,
                                             float a_chain = 1.0f)
{
    using Cfg = StepCfg<M, F, TF>;
    uint32_t ab[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) ab[i] = abs_bits(u.w[i]);

    bool kept[8];
    uint32_t keep = 0;                  // as bits, where some consumer below wants bits
    if constexpr (Cfg::network) {
        select_2of4(ab, kept);
        select_2of4(ab + 4, kept + 4);
        constexpr bool want_bits = Cfg::bitmask || Cfg::stats;
        if constexpr (want_bits) {
#pragma unroll
            for (int i = 0; i < 8; ++i) keep |= (kept[i] ? 1u : 0u) << i;
        }
        if constexpr (Cfg::bitmask) u.meta_byte = keep;
        else u.meta_byte = idx2_from_kept(kept) | (idx2_from_kept(kept + 4) << 4);
        if constexpr (Cfg::count_flips) {
            if constexpr (Cfg::bitmask) sums.flips = (uint32_t)__popc(keep ^ u.prev_byte);
            // equal index bytes are equal masks (most units, most steps): the decode is skipped there -- except in the
            // kernels that also carry the scale gradient, where the branch costs registers (spills; measured slower)
            else if (Cfg::of_scaled || u.meta_byte != u.prev_byte)
                sums.flips = (uint32_t)__popc(keep_from_meta_byte(u.meta_byte, false) ^ keep_from_meta_byte(u.prev_byte, false));
        }
    } else {
        if constexpr (Cfg::reselect) {
            keep = select_top_n<M>(ab, c.n_keep);              // all lanes shuffle for M > 8
            u.meta_byte = keep;                                 // only 2:4 has an index form
            if constexpr (Cfg::count_flips) sums.flips = (uint32_t)__popc(keep ^ u.prev_byte);
        } else {
            keep = keep_from_meta_byte(u.prev_byte, Cfg::bitmask);   // the stored mask, as it is
            u.meta_byte = u.prev_byte;
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) kept[i] = (keep >> i) & 1u;
    }
    u.keep = keep;
    if constexpr (Cfg::stats) {
        if (has_ref) sums.mask_diff = (uint32_t)__popc(keep ^ keep_from_meta_byte(u.ref_byte, Cfg::bitmask));
    }

    const uint32_t gw[4] = {u.g.x, u.g.y, u.g.z, u.g.w};
    const int sign_hi = __double2hiint(c.c_sign), sign_lo = __double2loint(c.c_sign);
    // With kGradOfScaled the gradient is taken with respect to W_scale = Diag(A) W (Eq. 12): the chain rule
    // gives dL/dW = A g (formed exactly in fp64) and dL/dA = sum of g W over the row segment, whose part
    // for this unit is returned in gw_sum (fp32 chain of 8 fused multiply-adds on the weights before the update).
    // The chain-rule factor is a_chain: the scale of the forward pass that produced g (the unit's `a` unless the
    // caller keeps the previous emission's scale apart from the one being trained).
    const double omb1_g = Cfg::of_scaled ? c.omb1 * (double)a_chain : c.omb1;
    gw_sum = 0.0f;
    float fwd[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        float g32 = __uint_as_float((i & 1) ? (gw[i >> 1] & 0xFFFF0000u) : (gw[i >> 1] << 16));
        if constexpr (Cfg::of_scaled) gw_sum = fmaf(g32, u.w[i], gw_sum);
        // first moment, stored undecayed (Alg. 1)
        const double mu = fma(c.beta1, (double)u.m[i], omb1_g * (double)g32);
        if constexpr (Cfg::of_scaled && Cfg::v_from_g) g32 *= a_chain;      // the alternate reading of v below uses dL/dW itself
        const float mu_f = (float)mu;
        u.m[i] = mu_f;
        // proportional L1 decay outside the kept set (Eq. 7): alpha lambda Sign(w), Sign(+-0) = 0
        const bool w_zero = ab[i] == 0u;
        const double sgn_term = __hiloint2double(w_zero ? 0 : (sign_hi ^ (int)(__float_as_uint(u.w[i]) & 0x80000000u)),
                                                 w_zero ? 0 : sign_lo);
        const float mu_t = kept[i] ? mu_f : (float)fma(c.c_mu, mu, sgn_term);
        // second moment from the decayed first moment (Eq. 8)
        const float src = (Cfg::v_from_g && kept[i]) ? g32 : mu_t;
        const float vn = fmaf(c.beta2, u.v[i], (c.omb2 * src) * src);
        u.v[i] = vn;
        // bias-corrected update (Alg. 1): w - (lr / bc1) mu~ / (sqrt(v / bc2) + eps)
        const float wn = u.w[i] - update_term(mu_t, vn, c);
        u.w[i] = wn;
        if constexpr (Cfg::stats) {                  // |w_t| converts exactly; fp64 sums
            const double mag = (double)fabsf(wn);
            sums.total_abs += mag;
            if (kept[i]) sums.kept_abs += mag;
        }
        // forward weight: scaled (Eq. 12), pruned by the mask unless the dense form is asked for (the compressed
        // form picks the kept values out afterwards, so it needs no zeros either)
        fwd[i] = (kept[i] || Cfg::dense || Cfg::compressed) ? a * wn : 0.0f;
    }
    u.g.x = pack_bf16x2(fwd[0], fwd[1]);
    u.g.y = pack_bf16x2(fwd[2], fwd[3]);
    u.g.z = pack_bf16x2(fwd[4], fwd[5]);
    u.g.w = pack_bf16x2(fwd[6], fwd[7]);
}

// dL/dA of Eq. 12: sums gw_sum over the lanes of the warp that share a row segment (segments are runs of consecutive
// lanes), then one atomic per run.  Lanes without data carry a segment of their own and add nothing.  All lanes of
// the warp call this (the pointer is uniform over the CTA).
__device__ __forceinline__ void add_scale_grad(float* scale_grad, uint32_t seg, bool active, float gw_sum)
{
    if (scale_grad == nullptr) return;
    const unsigned lane = threadIdx.x & 31u;
    const uint32_t my_seg = active ? seg : 0xFFFFFFFFu;
    float p = active ? gw_sum : 0.0f;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const float q = __shfl_up_sync(0xFFFFFFFFu, p, d);
        const uint32_t s = __shfl_up_sync(0xFFFFFFFFu, my_seg, d);
        if (lane >= (unsigned)d && s == my_seg) p += q;
    }
    const uint32_t next_seg = __shfl_down_sync(0xFFFFFFFFu, my_seg, 1);
    if (active && (lane == 31u || next_seg != my_seg)) atomicAdd(scale_grad + seg, p);
}

// The whole per-unit body: loads, arithmetic, stores.
// `active` is false for threads past the end of the matrix; they take part in the shuffles only.
template <int M, uint32_t F, bool TF>
__device__ __forceinline__ void process_unit(const TensorDesc& t, const StepConsts& c, uint32_t unit, bool active, UnitSums& sums)
{
    using Cfg = StepCfg<M, F, TF>;
    UnitRegs u;
    u.g = make_uint4(0, 0, 0, 0);
    u.prev_byte = 0;
    u.ref_byte = 0;
    const size_t e = (size_t)unit * kUnitElems;
    float a = 1.0f, a_chain = 1.0f;
    uint32_t seg = 0;
    const bool has_ref = Cfg::stats && t.meta_ref != nullptr;      // uniform over the CTA

    if (active) {
        const float4 w0 = ld_f4(t.w + e), w1 = ld_f4(t.w + e + 4);
        const float4 m0 = ld_f4(t.m + e), m1 = ld_f4(t.m + e + 4);
        const float4 v0 = ld_f4(t.v + e), v1 = ld_f4(t.v + e + 4);
        u.g = *reinterpret_cast<const uint4*>(t.g + e);
        if constexpr (Cfg::need_prev) u.prev_byte = reinterpret_cast<const uint8_t*>(t.meta)[unit];
        if (has_ref) u.ref_byte = t.meta_ref[unit];
        if (t.scale != nullptr) {
            seg = (uint32_t)(((uint64_t)unit * t.seg_magic) >> t.seg_shift);   // row * n + segment of the row
            a = __ldg(t.scale + seg);
            if constexpr (Cfg::of_scaled) a_chain = __ldg(t.scale_chain + seg);      // the host points it at `scale` where there is no other
        }
        u.w[0] = w0.x; u.w[1] = w0.y; u.w[2] = w0.z; u.w[3] = w0.w; u.w[4] = w1.x; u.w[5] = w1.y; u.w[6] = w1.z; u.w[7] = w1.w;
        u.m[0] = m0.x; u.m[1] = m0.y; u.m[2] = m0.z; u.m[3] = m0.w; u.m[4] = m1.x; u.m[5] = m1.y; u.m[6] = m1.z; u.m[7] = m1.w;
        u.v[0] = v0.x; u.v[1] = v0.y; u.v[2] = v0.z; u.v[3] = v0.w; u.v[4] = v1.x; u.v[5] = v1.y; u.v[6] = v1.z; u.v[7] = v1.w;
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) { u.w[i] = 0.f; u.m[i] = 0.f; u.v[i] = 0.f; }
    }

    float gw_sum;
    UnitSums mine;
    compute_unit<M, F, TF>(u, c, a, has_ref, gw_sum, mine, a_chain);
    if constexpr (Cfg::of_scaled) add_scale_grad(t.scale_grad, seg, active, gw_sum);

    if (active) {
        st_f4(t.w + e, make_float4(u.w[0], u.w[1], u.w[2], u.w[3]));
        st_f4(t.w + e + 4, make_float4(u.w[4], u.w[5], u.w[6], u.w[7]));
        st_f4(t.m + e, make_float4(u.m[0], u.m[1], u.m[2], u.m[3]));
        st_f4(t.m + e + 4, make_float4(u.m[4], u.m[5], u.m[6], u.m[7]));
        st_f4(t.v + e, make_float4(u.v[0], u.v[1], u.v[2], u.v[3]));
        st_f4(t.v + e + 4, make_float4(u.v[4], u.v[5], u.v[6], u.v[7]));
        if constexpr (!Cfg::compressed) {
            *reinterpret_cast<uint4*>(t.w_fwd + e) = u.g;
        } else if constexpr (TF && !Cfg::bitmask) {
            // the index-form metadata byte holds the kept positions of both groups: lo | hi << 2 per nibble
            const uint32_t mb = u.meta_byte;
            *reinterpret_cast<uint2*>(t.w_fwd + (size_t)unit * 4) =
                make_uint2(kept_pair_by_index(u.g.x, u.g.y, mb & 3u, (mb >> 2) & 3u),
                           kept_pair_by_index(u.g.z, u.g.w, (mb >> 4) & 3u, mb >> 6));
        } else if constexpr (TF) {
            *reinterpret_cast<uint2*>(t.w_fwd + (size_t)unit * 4) =
                make_uint2(kept_pair_2of4(u.g.x, u.g.y, u.meta_byte & 0xFu), kept_pair_2of4(u.g.z, u.g.w, u.meta_byte >> 4));
        } else {
            store_kept_values<M>(t.w_fwd, unit, u.keep, u.g, c.n_keep);
        }
        if constexpr (Cfg::reselect) reinterpret_cast<uint8_t*>(t.meta)[unit] = (uint8_t)u.meta_byte;   // else unchanged
        sums = mine;
    }
}

// Tables of one multi-tensor launch, passed by value in kernel parameter space (constant bank): a CTA
// lives only a few microseconds, so finding its matrix must not cost a chain of global-memory
// round trips, and the constant cache is not swept by the streaming data the way L1 is.
// The tile index space is the concatenation of all matrices' tiles (each matrix padded to whole
// tiles): tile_start[k] is the first tile of matrix k, tile_start[n] the total.
// hint[b >> hint_shift] is the matrix that holds tile (b >> hint_shift) << hint_shift, from which the
// CTA walks forward (usually zero or one step).
constexpr int kMaxLaunchTensors = 320;
constexpr int kHintEntries = 256;
struct MultiParams {
    uint32_t n_tensors;
    uint32_t hint_shift;
    uint16_t hint[kHintEntries];
    uint32_t tile_start[kMaxLaunchTensors + 1];
    TensorDesc desc[kMaxLaunchTensors];
};
static_assert(sizeof(MultiParams) + sizeof(StepConsts) + 32 <= 32764, "kernel parameters are limited to 32764 bytes");
static_assert(sizeof(TensorDesc) == 96, "one matrix of a launch table");

// What the CTA counted, added to the caller's counters: one atomic per counter per CTA.
template <bool FLIPS, bool STATS>
__device__ __forceinline__ void add_sums(UnitSums x, unsigned long long* flip_count, MaskStats* stats)
{
    if constexpr (FLIPS || STATS) {
        __shared__ uint32_t s_flips[kThreads / 32], s_diff[kThreads / 32];
        __shared__ double s_kept[kThreads / 32], s_total[kThreads / 32];
        const int warp = threadIdx.x >> 5;
        const bool lead = (threadIdx.x & 31) == 0;
        if constexpr (FLIPS) {
            const uint32_t f = __reduce_add_sync(0xFFFFFFFFu, x.flips);
            if (lead) s_flips[warp] = f;
        }
        if constexpr (STATS) {
            const uint32_t d = __reduce_add_sync(0xFFFFFFFFu, x.mask_diff);
            double k = x.kept_abs, t = x.total_abs;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                k += __shfl_down_sync(0xFFFFFFFFu, k, o);
                t += __shfl_down_sync(0xFFFFFFFFu, t, o);
            }
            if (lead) { s_diff[warp] = d; s_kept[warp] = k; s_total[warp] = t; }
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            if constexpr (FLIPS) {
                unsigned long long total = 0;
#pragma unroll
                for (int i = 0; i < kThreads / 32; ++i) total += s_flips[i];
                if (total) atomicAdd(flip_count, total);
            }
            if constexpr (STATS) {
                unsigned long long d = 0;
                double k = 0.0, t = 0.0;
#pragma unroll
                for (int i = 0; i < kThreads / 32; ++i) { d += s_diff[i]; k += s_kept[i]; t += s_total[i]; }
                MaskStats* slot = stats + (blockIdx.x & (kStatSlots - 1u));
                if (d) atomicAdd(&slot->mask_diff, d);
                atomicAdd(&slot->kept_abs_sum, k);
                atomicAdd(&slot->total_abs_sum, t);
            }
        }
    }
}

// One matrix: CTA b handles tile b.
// Resident CTAs per SM a variant of the plain kernels is compiled for (85, 73, 64 registers per thread at 6, 7, 8).  In
// sustained runs under the board's power cap the variants that do more work per parameter react to the budget by 1-4 %,
// in either direction; the exceptions to 7 are the measured winners on the LLaMA2-7B set (ms per step at 6 / 7 / 8):
// 2:4 refresh 27.45 / 28.7 / 27.97, 2:4 refresh with the statistics 28.9 / 28.7 / 27.7, 4:8 select 28.2 / 27.8 / 27.2, 4:8
// refresh with the scale gradient 31.3 / 28.6 / 27.97, 8:16 select 28.4 / 27.3 / 26.8, 8:16 select + flips 28.4 / 29.3 /
// 29.2, 8:32 select 29.1 / 28.4 / 28.0, 8:32 select + flips 28.97 / 30.3 / 29.45.
template <int M, uint32_t F, bool TF>
constexpr int plain_ctas_per_sm()
{
    constexpr uint32_t refresh = kReselect | kCountFlips | kEmitDense;
    if (TF) return F == refresh ? 6 : F == (refresh | kMaskStats) ? 8 : kMinCtasPerSm;
    if (M == 8) return 8;
    if (M >= 16) return (F & kGradOfScaled) ? kMinCtasPerSm : (F & kCountFlips) ? 6 : 8;
    return kMinCtasPerSm;
}

template <int M, uint32_t F, bool TF>
__global__ void __launch_bounds__(kThreads, plain_ctas_per_sm<M, F, TF>())
adams_nm_kernel(const __grid_constant__ TensorDesc t, const __grid_constant__ StepConsts c,
                unsigned long long* __restrict__ flip_count, MaskStats* __restrict__ stats)
{
    const uint32_t unit = blockIdx.x * kTileUnits + threadIdx.x;
    UnitSums sums;
    process_unit<M, F, TF>(t, c, unit, unit < t.n_units, sums);
    add_sums<StepCfg<M, F, TF>::count_flips, StepCfg<M, F, TF>::stats>(sums, flip_count, stats);
}

// Up to kMaxLaunchTensors matrices in one grid: CTA b handles tile b of the concatenated index space.
template <int M, uint32_t F, bool TF>
__global__ void __launch_bounds__(kThreads, plain_ctas_per_sm<M, F, TF>())
adams_nm_multi_kernel(const __grid_constant__ MultiParams p, const __grid_constant__ StepConsts c,
                      unsigned long long* __restrict__ flip_count, MaskStats* __restrict__ stats)
{
    const uint32_t tile = blockIdx.x;
    uint32_t k = p.hint[tile >> p.hint_shift];
    while (tile >= p.tile_start[k + 1]) ++k;
    const TensorDesc& t = p.desc[k];
    const uint32_t unit = (tile - p.tile_start[k]) * kTileUnits + threadIdx.x;
    UnitSums sums;
    process_unit<M, F, TF>(t, c, unit, unit < t.n_units, sums);
    add_sums<StepCfg<M, F, TF>::count_flips, StepCfg<M, F, TF>::stats>(sums, flip_count, stats);
}

}  // namespace cast
