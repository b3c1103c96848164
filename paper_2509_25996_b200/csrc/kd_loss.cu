// Training loss of CAST (Sec. 4.3, Eq. 13) per token, L = eta D_KL(P_t || P_s) + (1 - eta) L_ce, and its gradient
// with respect to the student logits, grad_scale (P_s - eta P_t - (1 - eta) onehot), in one kernel.
//
// Streaming and reduction-bound: a row of `vocab` logits per token, 2 + 2 B read and 2 B written per logit.  With
//     D_KL(P_t || P_s) = E_{P_t}[t - s] + lse(s) - lse(t),        L_ce = lse(s) - s_label,
// a single sweep over the row yields everything the loss needs: the running maxima and sums of exp of both rows
// (online softmax: a sum is rescaled when its maximum moves) and sum exp(t - max t) (t - s).  The gradient needs
// the finished normalisers, i.e. a second sweep over the same values: the row is read again, and that second read
// has to come from the L2, not from HBM (6 instead of 10 B per logit).  Two things keep it there:
//   * the rows in flight are bounded: a row is handled by a cluster of CTAs (1 CTA for short rows, 8 for rows
//     beyond 64 K logits), each CTA sweeping its own segment of the row; the clusters' CTAs exchange their five
//     partial sums through distributed shared memory (plain loads of a peer CTA's shared memory between two cluster
//     barriers).  With 8 CTAs per row a 128 K-logit vocabulary has ~140 rows (~110 MB with their gradients) in flight
//     instead of the ~2400 rows (1.2 GB) of one small CTA per row, whose second sweep went to HBM entirely;
//   * the second sweep runs back to front, so it starts on the lines the first sweep touched last.
// The kernel is co-limited by the special-function unit: four exponentials per logit (two per sweep) at 16 per
// clock and SM is the same ~1.1e12 logits/s as 6 B per logit at the HBM rate; everything else per logit is kept
// small: the weights of the gradient's two terms are folded into the exponents (one subtraction gives the
// gradient), the label is looked for once per vector.
// Arithmetic in fp32 in the base-2 domain (ex2.approx: 2 ulp; argument error ~1e-7 |x log2 e|); reductions by warp
// shuffles and shared memory.  No device-side waits other than the cluster's hardware barrier, at which every CTA of
// a cluster arrives unconditionally.
#include <cmath>

#include <cooperative_groups.h>

#include "cast_internal.h"

namespace cg = cooperative_groups;

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

// Largest of the 8 bf16 values of a vector, taken on the packed pairs (three 2-wide maxima, then the two halves).
__device__ __forceinline__ float max8_bf16(uint4 p)
{
    uint32_t m;
    asm("{ .reg .b32 a, b;\n\t"
        "max.bf16x2 a, %1, %2;\n\t"
        "max.bf16x2 b, %3, %4;\n\t"
        "max.bf16x2 %0, a, b; }" : "=r"(m) : "r"(p.x), "r"(p.y), "r"(p.z), "r"(p.w));
    return fmaxf(__uint_as_float(m << 16), __uint_as_float(m & 0xFFFF0000u));
}

// One vector of both rows into the running sums.  Called by all lanes of a warp (there is a vote inside); a lane
// with `have` false has no vector in this trip and leaves its sums alone.
__device__ __forceinline__ void absorb8(RowSums& r, uint4 sp, uint4 tp, bool have)
{
    const float cs = max8_bf16(sp) * kLog2e, ct = max8_bf16(tp) * kLog2e;
    // A running maximum moves in the first few vectors of a row and almost never after: the whole warp skips the
    // rescaling with one vote instead of issuing its predicated-off instructions for every vector.
    if (__any_sync(0xFFFFFFFFu, have && (cs > r.ms2 || ct > r.mt2))) {
        if (have && cs > r.ms2) { r.zs *= ex2(r.ms2 - cs); r.ms2 = cs; }
        if (have && ct > r.mt2) { const float f = ex2(r.mt2 - ct); r.zt *= f; r.a *= f; r.mt2 = ct; }
    }
    if (have) {
        float s[8], t[8];
        unpack8(sp, s);
        unpack8(tp, t);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            r.zs += ex2(fmaf(s[i], kLog2e, -r.ms2));
            const float e = ex2(fmaf(t[i], kLog2e, -r.mt2));
            r.zt += e;
            r.a = fmaf(e, t[i] - s[i], r.a);
        }
    }
}

// The same for one lane on its own (no vote): the form the one-CTA-per-row kernel uses.  Measured on B200 the voted
// form is ~7 % faster for rows split over a cluster (few trips per CTA) and ~2 % slower for a whole row per CTA.
__device__ __forceinline__ void absorb8_lane(RowSums& r, uint4 sp, uint4 tp)
{
    float s[8], t[8];
    unpack8(sp, s);
    unpack8(tp, t);
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
__device__ __forceinline__ Finished finish(const RowSums& r, const uint16_t* s_row, int label, float eta, float* loss_out,
                                           bool writer = true)
{
    Finished f;
    f.lse_s2 = r.ms2 + log2f(r.zs);
    f.lse_t2 = r.mt2 + log2f(r.zt);
    if (writer && threadIdx.x == 0) {
        const float lse_s = f.lse_s2 * kLn2;
        const float kl = r.a / r.zt + (f.lse_s2 - f.lse_t2) * kLn2;                       // E_t[t - s] + lse(s) - lse(t)
        float ce = 0.0f;
        if (label >= 0) ce = lse_s - __uint_as_float((uint32_t)s_row[label] << 16);       // -log P_s(label)
        *loss_out = eta * kl + (1.0f - eta) * ce;
    }
    return f;
}

// What the second sweep needs: exponent offsets with the weights of the gradient's two terms folded in,
//   |grad_scale| w_s P_s = 2^(s log2 e + off_s),  off_s = log2(|grad_scale| w_s) - lse_s2     (w_s = 1, or eta without a target)
//   |grad_scale| eta P_t = 2^(t log2 e + off_t),  off_t = log2(|grad_scale| eta) - lse_t2
// (a zero weight gives off = -inf and a term that is exactly 0), the sign of grad_scale, and the one-hot term.
struct GradConsts { float off_s, off_t, onehot; uint32_t sign_bits; };   // sign_bits: 0x80008000 flips a packed pair

__device__ __forceinline__ GradConsts grad_consts(const Finished& f, int label, float eta, float grad_scale)
{
    const float mag = fabsf(grad_scale);
    GradConsts g;
    g.off_s = log2f(mag * (label >= 0 ? 1.0f : eta)) - f.lse_s2;
    g.off_t = log2f(mag * eta) - f.lse_t2;
    g.sign_bits = grad_scale < 0.0f ? 0x80008000u : 0u;      // the sign of grad_scale is applied to the packed result
    g.onehot = label >= 0 ? mag * (1.0f - eta) : 0.0f;
    return g;
}

// gradient of 8 logits, without the one-hot term (the label's owner adds it after its sweep)
__device__ __forceinline__ uint4 grad8(uint4 sp, uint4 tp, const GradConsts& k)
{
    float s[8], t[8], g[8];
    unpack8(sp, s);
    unpack8(tp, t);
#pragma unroll
    for (int i = 0; i < 8; ++i)
        g[i] = ex2(fmaf(s[i], kLog2e, k.off_s)) - ex2(fmaf(t[i], kLog2e, k.off_t));
    return make_uint4(pack2(g[0], g[1]) ^ k.sign_bits, pack2(g[2], g[3]) ^ k.sign_bits, pack2(g[4], g[5]) ^ k.sign_bits,
                      pack2(g[6], g[7]) ^ k.sign_bits);
}

// vocab % 8 == 0.  A cluster of CLUSTER CTAs handles one row (token); CTA `rank` of the cluster sweeps the vectors
// [rank * per, min(n_vec, (rank + 1) * per)) of it.
template <int THREADS, int CLUSTER>
__global__ void __launch_bounds__(THREADS)
kd_loss_kernel(const uint16_t* __restrict__ student, const uint16_t* __restrict__ teacher, const int32_t* __restrict__ labels,
               float* __restrict__ loss, uint16_t* __restrict__ grad, int vocab, float eta, float grad_scale)
{
    const unsigned token = blockIdx.x / CLUSTER;
    unsigned rank = 0;
    if constexpr (CLUSTER > 1) rank = cg::this_cluster().block_rank();
    const size_t row = (size_t)token * (size_t)vocab;
    const uint4* s_vec = reinterpret_cast<const uint4*>(student + row);
    const uint4* t_vec = reinterpret_cast<const uint4*>(teacher + row);
    const int n_vec = vocab / 8;
    const int per = (n_vec + CLUSTER - 1) / CLUSTER;
    const int v0 = (int)rank * per, v1 = min(n_vec, v0 + per);
    int label = labels[token];
    if (label >= vocab) label = -1;          // out of range: no target (never read past the row)

    RowSums r = {-INFINITY, 0.0f, -INFINITY, 0.0f, 0.0f};
    // cluster form: all lanes of a warp make the same number of trips (the vote inside absorb8 needs the whole warp);
    // in the last trip some lanes may have no vector
    if constexpr (CLUSTER > 1) {
        const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
        const int warp_first = v0 + (int)(threadIdx.x & ~31u);
#pragma unroll 2
        for (int base = warp_first; base < v1; base += THREADS) {
            const int c = base + (int)(threadIdx.x & 31u);
            const bool have = c < v1;
            absorb8(r, have ? s_vec[c] : zero, have ? t_vec[c] : zero, have);
        }
    } else {
#pragma unroll 2
        for (int c = v0 + (int)threadIdx.x; c < v1; c += THREADS) absorb8_lane(r, s_vec[c], t_vec[c]);
    }
    r = block_merge<THREADS>(r);
    if constexpr (CLUSTER > 1) {
        // every CTA of the cluster publishes the sums of its segment and merges all of them (in rank order, so that
        // all CTAs of the row get the same bits)
        __shared__ RowSums mine;
        cg::cluster_group cluster = cg::this_cluster();
        if (threadIdx.x == 0) mine = r;
        cluster.sync();
        RowSums total = *cluster.map_shared_rank(&mine, 0);
#pragma unroll
        for (int k = 1; k < CLUSTER; ++k) merge(total, *cluster.map_shared_rank(&mine, k));
        cluster.sync();                      // no CTA leaves (or overwrites `mine`) while a peer may still read it
        r = total;
    }
    const Finished f = finish(r, student + row, label, eta, loss + token, rank == 0);
    if (grad == nullptr) return;
    const GradConsts k = grad_consts(f, label, eta, grad_scale);
    uint4* g_vec = reinterpret_cast<uint4*>(grad + row);
    // back to front: the second sweep starts on the part of the segment the first sweep read last
#pragma unroll 2
    for (int c = v1 - 1 - (int)threadIdx.x; c >= v0; c -= THREADS) g_vec[c] = grad8(s_vec[c], t_vec[c], k);
    // The one-hot term of the label's column: recomputed and stored by the thread that stored the label's vector
    // (program order puts this store after that one), instead of a test in every trip of the sweep.
    const int cv = label >> 3;                 // label < 0 gives a negative vector index: no owner
    if (cv >= v0 && cv < v1 && (unsigned)((v1 - 1 - cv) % THREADS) == threadIdx.x) {
        const float s = __uint_as_float((uint32_t)student[row + label] << 16), t = __uint_as_float((uint32_t)teacher[row + label] << 16);
        const float g = ex2(fmaf(s, kLog2e, k.off_s)) - ex2(fmaf(t, kLog2e, k.off_t)) - k.onehot;
        grad[row + label] = (uint16_t)((pack2(g, 0.0f) ^ k.sign_bits) & 0xFFFFu);
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
    if (vec && vocab <= 65536) {
        // one CTA of 512 threads per row: ~450 rows of <= 256 KB in flight, inside the L2
        kd_loss_kernel<512, 1><<<grid, 512, 0, s>>>(student_logits, teacher_logits, labels, loss, grad_logits, (int)vocab, eta, grad_scale);
        CAST_CUDA_TRY(cudaGetLastError());
    } else if (vec) {
        // a cluster of 8 CTAs of 256 threads per row: the rows in flight stay inside the L2 for long rows too
        constexpr int kCluster = 8;
        if ((uint64_t)tokens * kCluster > 0x7FFFFFFFull) return CAST_ERR_SHAPE;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(grid * kCluster);
        cfg.blockDim = dim3(256);
        // Residency is left to the registers (8 CTAs per SM, ~140 rows in flight): capping it at 5 CTAs per SM by a
        // dummy shared-memory request brings the DRAM traffic from 7.6 down to 5.9 B per logit but costs 11 % of time
        // (0.95 against 0.85 ms for 4096 x 128256), and so does any such request, even one that leaves the residency
        // alone (28 KB: 0.955 ms): the shared-memory carve-out shrinks the L1 the sweeps run through.
        cfg.stream = s;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = kCluster;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        CAST_CUDA_TRY(cudaLaunchKernelEx(&cfg, kd_loss_kernel<256, kCluster>, (const uint16_t*)student_logits, (const uint16_t*)teacher_logits,
                                         labels, loss, (uint16_t*)grad_logits, (int)vocab, eta, grad_scale));
    } else {
        kd_loss_scalar_kernel<256><<<grid, 256, 0, s>>>(student_logits, teacher_logits, labels, loss, grad_logits, (int)vocab, eta, grad_scale);
        CAST_CUDA_TRY(cudaGetLastError());
    }
    count_launch();
    return CAST_OK;
}
