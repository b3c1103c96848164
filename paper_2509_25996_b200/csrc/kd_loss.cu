// Training loss of CAST (Sec. 4.3, Eq. 13) per token, L = eta D_KL(P_t || P_s) + (1 - eta) L_ce, and its gradient
// with respect to the student logits, grad_scale (P_s - eta P_t - (1 - eta) onehot), in one kernel.
//
// Streaming and reduction-bound: a row of `vocab` logits per token, 2 + 2 B read and 2 B written per logit.
// One CTA per token.  With
//     D_KL(P_t || P_s) = E_{P_t}[t - s] + lse(s) - lse(t),        L_ce = lse(s) - s_label,
// a single sweep over the row yields everything the loss needs: the running maxima and sums of exp of both rows
// (online softmax: a sum is rescaled when its maximum moves) and sum exp(t - max t) (t - s).  The gradient needs
// the finished normalisers, i.e. a second sweep over the same values: the row is simply read again -- the rows in
// flight (a few CTAs per SM x 2 x vocab x 2 B, tens of MB) sit well inside the 126 MB L2, so the second sweep does
// not go to HBM.  (Keeping rows of up to 32768 logits in registers between the sweeps, 8 vectors per thread and
// row, was measured slower: 118 registers allow one CTA per SM, whose phases then do not overlap.)
// The kernel is co-limited by the special-function unit: four exponentials per logit (two per sweep) at 16 per
// clock and SM is the same ~1.1e12 logits/s as 6 B per logit at the HBM rate.
// Arithmetic in fp32 in the base-2 domain (ex2.approx: 2 ulp; argument error ~1e-7 |x log2 e|); reductions by warp
// shuffles and shared memory.  No device-side waits.
#include <cmath>

#include "cast_internal.h"

namespace cast {
namespace {

constexpr float kLog2e = 1.4426950408889634f;      // exponentials are taken as 2^(x log2 e): one fused multiply-add and
constexpr float kLn2 = 0.6931471805599453f;        // one ex2 instruction each
__device__ __forceinline__ float ex2(float x) { float r; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x)); return r; }

// Online softmax state of both rows, in the base-2 domain: ms2 = fl(max s * log2 e) is the shift every student term
// of this partial sum was formed with, zs = sum 2^(s log2 e - ms2); likewise mt2, zt for the teacher row, and
// a = sum 2^(t log2 e - mt2) (t - s).  lse(s) = (ms2 + log2 zs) ln 2 whatever rounding ms2 carries.
struct RowSums { float ms2, zs, mt2, zt, a; };

__device__ __forceinline__ void merge(RowSums& x, const RowSums& y)
{
    const float ms2 = fmaxf(x.ms2, y.ms2), mt2 = fmaxf(x.mt2, y.mt2);
    // a partial state that has seen nothing has shift -inf and sums 0: its factor is 2^-inf = 0, or 1 when both are empty
    const float fxs = (x.ms2 == ms2) ? 1.0f : ex2(x.ms2 - ms2), fys = (y.ms2 == ms2) ? 1.0f : ex2(y.ms2 - ms2);
    const float fxt = (x.mt2 == mt2) ? 1.0f : ex2(x.mt2 - mt2), fyt = (y.mt2 == mt2) ? 1.0f : ex2(y.mt2 - mt2);
    x.zs = x.zs * fxs + y.zs * fys;
    x.zt = x.zt * fxt + y.zt * fyt;
    x.a = x.a * fxt + y.a * fyt;
    x.ms2 = ms2;
    x.mt2 = mt2;
}

__device__ __forceinline__ void unpack8(uint4 p, float (&f)[8])
{
    const uint32_t w[4] = {p.x, p.y, p.z, p.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
}

__device__ __forceinline__ void absorb8(RowSums& r, const float (&s)[8], const float (&t)[8])
{
    float cs = s[0], ct = t[0];
#pragma unroll
    for (int i = 1; i < 8; ++i) { cs = fmaxf(cs, s[i]); ct = fmaxf(ct, t[i]); }
    cs *= kLog2e;
    ct *= kLog2e;
    if (cs > r.ms2) { r.zs *= ex2(r.ms2 - cs); r.ms2 = cs; }
    if (ct > r.mt2) { const float f = ex2(r.mt2 - ct); r.zt *= f; r.a *= f; r.mt2 = ct; }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        r.zs += ex2(fmaf(s[i], kLog2e, -r.ms2));
        const float e = ex2(fmaf(t[i], kLog2e, -r.mt2));
        r.zt += e;
        r.a = fmaf(e, t[i] - s[i], r.a);
    }
}

template <int THREADS>
__device__ __forceinline__ RowSums block_merge(RowSums r)
{
    __shared__ RowSums part[THREADS / 32];
    __shared__ RowSums total;
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        RowSums o;
        o.ms2 = __shfl_xor_sync(0xFFFFFFFFu, r.ms2, d); o.zs = __shfl_xor_sync(0xFFFFFFFFu, r.zs, d);
        o.mt2 = __shfl_xor_sync(0xFFFFFFFFu, r.mt2, d); o.zt = __shfl_xor_sync(0xFFFFFFFFu, r.zt, d);
        o.a = __shfl_xor_sync(0xFFFFFFFFu, r.a, d);
        merge(r, o);
    }
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = r;
    __syncthreads();
    if (threadIdx.x == 0) {
        RowSums t = part[0];
        for (int i = 1; i < THREADS / 32; ++i) merge(t, part[i]);
        total = t;
    }
    __syncthreads();
    return total;
}

__device__ __forceinline__ uint32_t pack2(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

struct Finished { float lse_s2, lse_t2; };      // log-sum-exp of both rows in the base-2 domain

// loss of the token from the finished sums; written by one thread
__device__ __forceinline__ Finished finish(const RowSums& r, const uint16_t* s_row, int label, float eta, float* loss_out)
{
    Finished f;
    f.lse_s2 = r.ms2 + log2f(r.zs);
    f.lse_t2 = r.mt2 + log2f(r.zt);
    if (threadIdx.x == 0) {
        const float lse_s = f.lse_s2 * kLn2;
        const float kl = r.a / r.zt + (f.lse_s2 - f.lse_t2) * kLn2;                       // E_t[t - s] + lse(s) - lse(t)
        float ce = 0.0f;
        if (label >= 0) ce = lse_s - __uint_as_float((uint32_t)s_row[label] << 16);       // -log P_s(label)
        *loss_out = eta * kl + (1.0f - eta) * ce;
    }
    return f;
}

// gradient of 8 logits starting at column `col`
__device__ __forceinline__ uint4 grad8(const float (&s)[8], const float (&t)[8], const Finished& f, int col, int label,
                                       float eta, float ps_weight, float onehot_weight, float grad_scale)
{
    float g[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const float ps = ex2(fmaf(s[i], kLog2e, -f.lse_s2)), pt = ex2(fmaf(t[i], kLog2e, -f.lse_t2));
        float x = fmaf(ps_weight, ps, -eta * pt);
        if (col + i == label) x -= onehot_weight;
        g[i] = grad_scale * x;
    }
    return make_uint4(pack2(g[0], g[1]), pack2(g[2], g[3]), pack2(g[4], g[5]), pack2(g[6], g[7]));
}

// vocab % 8 == 0.  CH > 0 (not used by the entry point): the row (at most CH * THREADS vectors) is kept in registers
// between the two sweeps.
template <int THREADS, int CH>
__global__ void __launch_bounds__(THREADS)
kd_loss_kernel(const uint16_t* __restrict__ student, const uint16_t* __restrict__ teacher, const int32_t* __restrict__ labels,
               float* __restrict__ loss, uint16_t* __restrict__ grad, int vocab, float eta, float grad_scale)
{
    const size_t row = (size_t)blockIdx.x * (size_t)vocab;
    const uint4* s_vec = reinterpret_cast<const uint4*>(student + row);
    const uint4* t_vec = reinterpret_cast<const uint4*>(teacher + row);
    const int n_vec = vocab / 8;
    int label = labels[blockIdx.x];
    if (label >= vocab) label = -1;          // out of range: no target (never read past the row)
    RowSums r = {-INFINITY, 0.0f, -INFINITY, 0.0f, 0.0f};
    constexpr int HELD = CH > 0 ? CH : 1;
    uint4 sv[HELD], tv[HELD];
    if constexpr (CH > 0) {
#pragma unroll
        for (int k = 0; k < CH; ++k) {
            const int c = threadIdx.x + k * THREADS;
            if (c < n_vec) { sv[k] = s_vec[c]; tv[k] = t_vec[c]; }
        }
#pragma unroll
        for (int k = 0; k < CH; ++k) {
            if (threadIdx.x + k * THREADS < n_vec) {
                float s[8], t[8];
                unpack8(sv[k], s); unpack8(tv[k], t);
                absorb8(r, s, t);
            }
        }
    } else {
        for (int c = threadIdx.x; c < n_vec; c += THREADS) {
            float s[8], t[8];
            unpack8(s_vec[c], s); unpack8(t_vec[c], t);
            absorb8(r, s, t);
        }
    }
    r = block_merge<THREADS>(r);
    const Finished f = finish(r, student + row, label, eta, loss + blockIdx.x);
    if (grad == nullptr) return;
    // with a target: P_s - eta P_t - (1 - eta) onehot; without: the cross-entropy share of P_s drops out too
    const float ps_weight = label >= 0 ? 1.0f : eta, onehot_weight = label >= 0 ? 1.0f - eta : 0.0f;
    uint4* g_vec = reinterpret_cast<uint4*>(grad + row);
    if constexpr (CH > 0) {
#pragma unroll
        for (int k = 0; k < CH; ++k) {
            const int c = threadIdx.x + k * THREADS;
            if (c < n_vec) {
                float s[8], t[8];
                unpack8(sv[k], s); unpack8(tv[k], t);
                g_vec[c] = grad8(s, t, f, c * 8, label, eta, ps_weight, onehot_weight, grad_scale);
            }
        }
    } else {
        for (int c = threadIdx.x; c < n_vec; c += THREADS) {
            float s[8], t[8];
            unpack8(s_vec[c], s); unpack8(t_vec[c], t);
            g_vec[c] = grad8(s, t, f, c * 8, label, eta, ps_weight, onehot_weight, grad_scale);
        }
    }
}

// any vocab: scalar accesses (rows need not be 16-byte aligned)
template <int THREADS>
__global__ void __launch_bounds__(THREADS)
kd_loss_scalar_kernel(const uint16_t* __restrict__ student, const uint16_t* __restrict__ teacher, const int32_t* __restrict__ labels,
                      float* __restrict__ loss, uint16_t* __restrict__ grad, int vocab, float eta, float grad_scale)
{
    const size_t row = (size_t)blockIdx.x * (size_t)vocab;
    int label = labels[blockIdx.x];
    if (label >= vocab) label = -1;          // out of range: no target (never read past the row)
    RowSums r = {-INFINITY, 0.0f, -INFINITY, 0.0f, 0.0f};
    for (int x = threadIdx.x; x < vocab; x += THREADS) {
        const float s = __uint_as_float((uint32_t)student[row + x] << 16), t = __uint_as_float((uint32_t)teacher[row + x] << 16);
        const float s2 = s * kLog2e, t2 = t * kLog2e;
        if (s2 > r.ms2) { r.zs *= ex2(r.ms2 - s2); r.ms2 = s2; }
        if (t2 > r.mt2) { const float fct = ex2(r.mt2 - t2); r.zt *= fct; r.a *= fct; r.mt2 = t2; }
        r.zs += ex2(fmaf(s, kLog2e, -r.ms2));
        const float e = ex2(fmaf(t, kLog2e, -r.mt2));
        r.zt += e;
        r.a = fmaf(e, t - s, r.a);
    }
    r = block_merge<THREADS>(r);
    const Finished f = finish(r, student + row, label, eta, loss + blockIdx.x);
    if (grad == nullptr) return;
    const float ps_weight = label >= 0 ? 1.0f : eta, onehot_weight = label >= 0 ? 1.0f - eta : 0.0f;
    for (int x = threadIdx.x; x < vocab; x += THREADS) {
        const float s = __uint_as_float((uint32_t)student[row + x] << 16), t = __uint_as_float((uint32_t)teacher[row + x] << 16);
        float g = fmaf(ps_weight, ex2(fmaf(s, kLog2e, -f.lse_s2)), -eta * ex2(fmaf(t, kLog2e, -f.lse_t2)));
        if (x == label) g -= onehot_weight;
        grad[row + x] = (uint16_t)(pack2(grad_scale * g, 0.0f) & 0xFFFFu);
    }
}

}  // namespace
}  // namespace cast

using namespace cast;

extern "C" int cast_kd_loss(const cast_bf16* student_logits, const cast_bf16* teacher_logits, const int32_t* labels,
                            float* loss, cast_bf16* grad_logits, int64_t tokens, int64_t vocab,
                            float eta, float grad_scale, cast_stream_t stream)
{
    if (!student_logits || !teacher_logits || !labels || !loss) return CAST_ERR_NULL;
    if (tokens < 1 || vocab < 1 || tokens > 0x7FFFFFFF || vocab > 0x7FFFFFF8) return CAST_ERR_SHAPE;
    if (!(eta >= 0.0f && eta <= 1.0f) || !std::isfinite(grad_scale)) return CAST_ERR_HYPER;
    if (((uintptr_t)student_logits & 1u) || ((uintptr_t)teacher_logits & 1u) || ((uintptr_t)grad_logits & 1u) ||
        ((uintptr_t)labels & 3u) || ((uintptr_t)loss & 3u)) return CAST_ERR_ALIGN;
    const uint64_t bytes = 2ull * (uint64_t)tokens * (uint64_t)vocab;
    if (grad_logits) {
        const uintptr_t g = (uintptr_t)grad_logits, s = (uintptr_t)student_logits, t = (uintptr_t)teacher_logits;
        if ((g < s + bytes && s < g + bytes) || (g < t + bytes && t < g + bytes)) return CAST_ERR_ALIAS;
    }
    const void* ptrs[5] = {student_logits, teacher_logits, labels, loss, grad_logits};
    int rc;
    if ((rc = check_device_memory(ptrs, 5)) != CAST_OK) return rc;
    cudaStream_t s = (cudaStream_t)stream;
    const unsigned grid = (unsigned)tokens;
    const bool vec = vocab % 8 == 0 && !((uintptr_t)student_logits & 15u) && !((uintptr_t)teacher_logits & 15u) &&
                     !((uintptr_t)grad_logits & 15u);
    // measured on B200: 512 threads per row up to ~64 K logits, 128 beyond (more rows in flight per SM)
    if (vec && vocab <= 65536)
        kd_loss_kernel<512, 0><<<grid, 512, 0, s>>>(student_logits, teacher_logits, labels, loss, grad_logits, (int)vocab, eta, grad_scale);
    else if (vec)
        kd_loss_kernel<128, 0><<<grid, 128, 0, s>>>(student_logits, teacher_logits, labels, loss, grad_logits, (int)vocab, eta, grad_scale);
    else
        kd_loss_scalar_kernel<256><<<grid, 256, 0, s>>>(student_logits, teacher_logits, labels, loss, grad_logits, (int)vocab, eta, grad_scale);
    CAST_CUDA_TRY(cudaGetLastError());
    count_launch();
    return CAST_OK;
}
