// Device helpers, the kernel for one-element blocks and the two-pass kernels
// (partial sums -> finalize -> update) that handle any block length and any
// alignment.  Update rule: Algorithm 1 of the paper.
#ifndef ADAMMINI_KERNELS_BASIC_CUH_
#define ADAMMINI_KERNELS_BASIC_CUH_

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "adammini_internal.h"

namespace am {

constexpr int kThreads = 256;            // CTA size of the kernels in this file
constexpr int kSmallMaxL = 64;           // blocks up to this length go to the short-block kernels
constexpr int kSmallVecMaxL = 3;         // ... and up to this length, when aligned, straight through registers (small_kernel)
constexpr int64_t kPieceMax = 32768;     // elements per partial sum, two-pass path
constexpr int64_t kMaxPiecesPerBlock = 16384;
constexpr int64_t kWideBlockPieces = 256;   // blocks with at least this many partial sums are finalized by a whole CTA

// ---------------------------------------------------------------------------
// small helpers
// ---------------------------------------------------------------------------
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// Four consecutive gradients, widened exactly to float.
// (every gradient is multiplied by `gscale` as it is loaded: 1.0f leaves it bit-exact)
template <int GD>
__device__ __forceinline__ float4 load_g4(const void *g, int64_t i, float gscale) {
    float4 r;
    if (GD == AM_BF16) {
        const uint2 u = *reinterpret_cast<const uint2 *>(static_cast<const uint16_t *>(g) + i);
        r = make_float4(bf16_lo(u.x), bf16_hi(u.x), bf16_lo(u.y), bf16_hi(u.y));
    } else {
        r = *reinterpret_cast<const float4 *>(static_cast<const float *>(g) + i);
    }
    r.x *= gscale; r.y *= gscale; r.z *= gscale; r.w *= gscale;
    return r;
}

template <int GD>
__device__ __forceinline__ float load_g1(const void *g, int64_t i, float gscale) {
    if (GD == AM_BF16)
        return __uint_as_float(static_cast<uint32_t>(static_cast<const uint16_t *>(g)[i]) << 16) * gscale;
    return static_cast<const float *>(g)[i] * gscale;
}

__device__ __forceinline__ float effective_gscale(float gscale, const float *gscale_dev) {
    return gscale_dev ? gscale * *gscale_dev : gscale;
}
__device__ __forceinline__ bool step_skipped(const float *skip_flag) {
    return skip_flag != nullptr && *skip_flag != 0.f;
}

// bf16 copy of updated parameters, round to nearest even
__device__ __forceinline__ void store_bf16x4(uint16_t *dst, const float4 &p) {
    const __nv_bfloat162 lo = __floats2bfloat162_rn(p.x, p.y), hi = __floats2bfloat162_rn(p.z, p.w);
    uint2 u;
    u.x = *reinterpret_cast<const uint32_t *>(&lo);
    u.y = *reinterpret_cast<const uint32_t *>(&hi);
    *reinterpret_cast<uint2 *>(dst) = u;
}
__device__ __forceinline__ void store_bf16(uint16_t *dst, float p) {
    const __nv_bfloat16 b = __float2bfloat16_rn(p);
    *dst = *reinterpret_cast<const uint16_t *>(&b);
}

// Elementwise part of Algorithm 1: first moment, decoupled decay on the old
// parameter, then the Adam term with the block's step size
//   step = eta_t / ((1-beta1^t) (sqrt(v_hat) + eps)).
// lr_wd is eta_t*lambda, or 0 for tensors exempt from decay (then p stays p exactly).
__device__ __forceinline__ void update_one(float g, float &m, float &p, float beta1, float omb1,
                                           float lr_wd, float step) {
    m = fmaf(omb1, g, beta1 * m);
    const float decayed = fmaf(-lr_wd, p, p);
    p = fmaf(-step, m, decayed);
}

__device__ __forceinline__ void update_four(const float4 &g, float4 &m, float4 &p, float beta1, float omb1,
                                            float lr_wd, float step) {
    update_one(g.x, m.x, p.x, beta1, omb1, lr_wd, step);
    update_one(g.y, m.y, p.y, beta1, omb1, lr_wd, step);
    update_one(g.z, m.z, p.z, beta1, omb1, lr_wd, step);
    update_one(g.w, m.w, p.w, beta1, omb1, lr_wd, step);
}

// Per-block scalars in double: new v_b from the block statistic (mean of g*g in
// Algorithm 1) and the step size (see update_one).
__device__ __forceinline__ float block_step_from_statistic(double statistic, float v_old,
                                                           const StepScalars &s, float *v_new) {
    const double vn = s.omb2 * statistic + s.beta2 * static_cast<double>(v_old);
    *v_new = static_cast<float>(vn);
    const double denom = sqrt(vn * s.inv_bc2) + s.eps;
    return static_cast<float>(s.lr_over_bc1 / denom);
}
__device__ __forceinline__ float block_step(double sum_sq, double L, float v_old,
                                            const StepScalars &s, float *v_new) {
    return block_step_from_statistic(sum_sq / L, v_old, s, v_new);
}

// The ablation statistics of the paper's appendix combine like this: sums for
// the mean, the 1-norm and the 2-norm (of g*g, resp. of (g*g)^2), max, min.
__device__ __forceinline__ double stat_combine(double a, double b, int statistic) {
    if (statistic == 1) return a > b ? a : b;
    if (statistic == 2) return a < b ? a : b;
    return a + b;
}
__device__ __forceinline__ double stat_identity(int statistic) {
    if (statistic == 1) return 0.0;                    // g*g >= 0
    if (statistic == 2) return __longlong_as_double(0x7ff0000000000000LL);   // +inf
    return 0.0;
}
__device__ __forceinline__ double stat_term(float g, int statistic) {
    const float sq = g * g;
    return statistic == 4 ? static_cast<double>(sq) * static_cast<double>(sq) : static_cast<double>(sq);
}
__device__ __forceinline__ double stat_finish(double acc, double L, int statistic) {
    if (statistic == 0) return acc / L;
    if (statistic == 4) return sqrt(acc);
    return acc;
}
__device__ __forceinline__ double warp_stat(double x, int statistic) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x = stat_combine(x, __shfl_xor_sync(0xffffffffu, x, o), statistic);
    return x;
}

// Segment lookup: the last segment whose unit_begin is <= unit, by a whole (converged) warp:
// 32 probes per round, so a table of up to 1024 segments takes two dependent loads where a
// binary search by one thread takes ten.  Every lane returns the result.  A CTA of these
// kernels lives for a few microseconds, and nothing can be requested from memory before its
// segment is known: on a table of 94 matrices the tile kernel went from 0.96 to 1.00 of the
// measured copy bandwidth with this.
__device__ __forceinline__ int find_seg_warp(const Seg *segs, int n_segs, int64_t unit) {
    const int lane = threadIdx.x & 31;
    int lo = 0, hi = n_segs;                    // the answer lies in [lo, hi)
    while (hi - lo > 1) {
        const int step = (hi - lo + 31) >> 5;
        const int idx = lo + lane * step;
        const bool le = idx < hi && segs[idx].unit_begin <= unit;
        const unsigned ball = __ballot_sync(0xffffffffu, le);      // a prefix of the lanes (lane 0 always)
        const int k = 31 - __clz(static_cast<int>(ball | 1u));
        lo += k * step;
        hi = hi < lo + step ? hi : lo + step;
    }
    return lo;
}

__device__ __forceinline__ double warp_sum(double x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

// ---------------------------------------------------------------------------
// Short blocks (L <= 64): float32 scalars throughout.  L == 1 (this is AdamW), 2 and 3
// with everything 16-byte aligned run here, straight from registers; every
// other case runs on the tile kernel (kernels_tile.cuh).
// ---------------------------------------------------------------------------
struct SmallScalars {
    float beta1, omb1, beta2, omb2, inv_bc2, lr_over_bc1, eps, lr_wd, gscale;
    const float *gscale_dev;
    const float *skip_flag;
    int statistic;
    int stall;                          // test hook of the tile kernel: the bulk copies are announced but not issued
    unsigned long long wait_limit_ns;   // polling time after which the tile kernel's wait gives up
};

__device__ __forceinline__ float small_block_step(float mean_sq, float v_old, const SmallScalars &s,
                                                  float *v_new) {
    const float vn = fmaf(s.omb2, mean_sq, s.beta2 * v_old);
    *v_new = vn;
    const float denom = __fsqrt_rn(vn * s.inv_bc2) + s.eps;
    return __fdiv_rn(s.lr_over_bc1, denom);
}

// Blocks of one, two or three elements, everything 16-byte aligned: a thread takes
// E = lcm(L, 4) consecutive elements per round (E / 4 16-byte accesses to each of g, m, p
// and E / L whole blocks with their v), so nothing passes through shared memory and no
// lane idles.  L == 1 is AdamW.
template <int L> struct SmallVec {
    static constexpr int E = L == 3 ? 12 : 4;                     // elements per thread per round
    static constexpr int NB = E / L;                              // blocks per thread per round
    static constexpr int kRounds = L == 3 ? 1 : 4;                // rounds per CTA unit
    static constexpr int kUnit = kThreads * E * kRounds;          // elements per CTA unit
};

// Statistic of one block of L gradients (already scaled): mean of g*g, or an ablation variant.
template <int L>
__device__ __forceinline__ float small_block_statistic(const float *g, int statistic) {
    if (L == 1) return g[0] * g[0];                               // every statistic of a one-element block
    if (statistic == 0 || statistic == 3) {
        float sum = g[0] * g[0];
#pragma unroll
        for (int k = 1; k < L; ++k) sum = fmaf(g[k], g[k], sum);
        return statistic == 0 ? __fdiv_rn(sum, static_cast<float>(L)) : sum;
    }
    double acc = stat_identity(statistic);
#pragma unroll
    for (int k = 0; k < L; ++k) acc = stat_combine(acc, stat_term(g[k], statistic), statistic);
    return static_cast<float>(stat_finish(acc, static_cast<double>(L), statistic));
}

template <int GD, int L>
__device__ __forceinline__ void small_body(const DevTensor &t, int64_t local, float *__restrict__ v,
                                           const SmallScalars &sc) {
    typedef SmallVec<L> V;
    const float lr_wd = t.wd ? sc.lr_wd : 0.f;
    const float gscale = effective_gscale(sc.gscale, sc.gscale_dev);
    float *vt = v + t.v_offset;
    const int64_t base = local * V::kUnit;
#pragma unroll
    for (int r = 0; r < V::kRounds; ++r) {
        const int64_t i = base + (static_cast<int64_t>(r) * kThreads + threadIdx.x) * V::E;
        if (i >= t.numel) break;
        float g[V::E], m[V::E], p[V::E], vv[V::NB];
#pragma unroll
        for (int q = 0; q < V::E / 4; ++q) {
            const float4 g4 = load_g4<GD>(t.g, i + 4 * q, gscale);
            const float4 m4 = *reinterpret_cast<const float4 *>(t.m + i + 4 * q);
            const float4 p4 = *reinterpret_cast<const float4 *>(t.p + i + 4 * q);
            g[4 * q] = g4.x; g[4 * q + 1] = g4.y; g[4 * q + 2] = g4.z; g[4 * q + 3] = g4.w;
            m[4 * q] = m4.x; m[4 * q + 1] = m4.y; m[4 * q + 2] = m4.z; m[4 * q + 3] = m4.w;
            p[4 * q] = p4.x; p[4 * q + 1] = p4.y; p[4 * q + 2] = p4.z; p[4 * q + 3] = p4.w;
        }
        const int64_t b0 = i / L;                                 // exact: i is a multiple of E
        if (V::NB == 4) {
            const float4 v4 = *reinterpret_cast<const float4 *>(vt + b0);
            vv[0] = v4.x; vv[1] = v4.y; vv[2] = v4.z; vv[3] = v4.w;
        } else {
            const float2 v2 = *reinterpret_cast<const float2 *>(vt + b0);
            vv[0] = v2.x; vv[1] = v2.y;
        }
#pragma unroll
        for (int b = 0; b < V::NB; ++b) {
            const float st = small_block_step(small_block_statistic<L>(g + b * L, sc.statistic), vv[b], sc, &vv[b]);
#pragma unroll
            for (int k = 0; k < L; ++k) update_one(g[b * L + k], m[b * L + k], p[b * L + k], sc.beta1, sc.omb1, lr_wd, st);
        }
#pragma unroll
        for (int q = 0; q < V::E / 4; ++q) {
            const float4 m4 = make_float4(m[4 * q], m[4 * q + 1], m[4 * q + 2], m[4 * q + 3]);
            const float4 p4 = make_float4(p[4 * q], p[4 * q + 1], p[4 * q + 2], p[4 * q + 3]);
            *reinterpret_cast<float4 *>(t.m + i + 4 * q) = m4;
            *reinterpret_cast<float4 *>(t.p + i + 4 * q) = p4;
            if (t.p_bf16) store_bf16x4(t.p_bf16 + i + 4 * q, p4);
        }
        if (V::NB == 4) *reinterpret_cast<float4 *>(vt + b0) = make_float4(vv[0], vv[1], vv[2], vv[3]);
        else *reinterpret_cast<float2 *>(vt + b0) = make_float2(vv[0], vv[1]);
    }
}

// Whether a tensor of blocks of L elements can take small_kernel: every access above is aligned.
__host__ __device__ inline bool small_vec_ok(int64_t L, int64_t numel, int64_t v_offset) {
    if (L == 1) return numel % 4 == 0 && v_offset % 4 == 0;
    if (L == 2) return numel % 4 == 0 && v_offset % 2 == 0;
    if (L == 3) return numel % 12 == 0 && v_offset % 4 == 0;
    return false;
}
__host__ __device__ inline int64_t small_vec_unit(int64_t L) {
    return L == 3 ? SmallVec<3>::kUnit : SmallVec<1>::kUnit;
}

// One launch per block length present (the units of the segments of one length are
// consecutive, starting at first_unit), so that the AdamW case keeps the registers it needs
// and no more.
template <int L>
__global__ void __launch_bounds__(kThreads, L == 3 ? 3 : 4)
small_kernel(const DevTensor *__restrict__ tensors, const Seg *__restrict__ segs, int n_segs,
             float *__restrict__ v, SmallScalars sc, int64_t first_unit) {
    if (step_skipped(sc.skip_flag)) return;
    const int64_t unit = first_unit + blockIdx.x;
    const Seg seg = segs[find_seg_warp(segs, n_segs, unit)];
    const DevTensor &t = tensors[seg.tensor];
    const int64_t local = unit - seg.unit_begin;
    if (t.gdtype == AM_BF16) small_body<AM_BF16, L>(t, local, v, sc);
    else small_body<AM_F32, L>(t, local, v, sc);
}

// ---------------------------------------------------------------------------
// two-pass path.  Units of the partial and update kernels are pieces:
// piece (b, j) of a tensor covers elements [b*L + j*piece_len, ...) of block b.
// ---------------------------------------------------------------------------
struct PieceRef {
    const DevTensor *t;
    int64_t block, start, n, local;
    bool vec;               // the tensor's arrays start 16-byte aligned: 16-byte accesses where the element index allows
};

// Elements of a piece before the first one on a 16-byte boundary.
__device__ __forceinline__ int64_t piece_lead(const PieceRef &r) {
    const int64_t lead = (4 - (r.start & 3)) & 3;
    return lead < r.n ? lead : r.n;
}

__device__ __forceinline__ PieceRef decode_piece(const DevTensor *tensors, const Seg *segs, int n_segs,
                                                 int64_t unit) {
    const Seg seg = segs[find_seg_warp(segs, n_segs, unit)];
    PieceRef r;
    r.t = &tensors[seg.tensor];
    r.local = unit - seg.unit_begin;
    r.block = r.local / r.t->pieces_per_block;
    const int64_t j = r.local - r.block * r.t->pieces_per_block;
    const int64_t off = j * r.t->piece_len;
    r.start = r.block * r.t->L + off;
    const int64_t left = r.t->L - off;
    r.n = left < r.t->piece_len ? left : r.t->piece_len;
    r.vec = seg.aux != 0;
    return r;
}

// Sum of squares of one piece.  Per-thread float chains stay short (<= 64 terms
// per accumulator); everything above a thread is double and combined in a
// fixed order, so results do not depend on scheduling.
template <int GD>
__device__ __forceinline__ double piece_sum_sq(const PieceRef &r, float gscale) {
    double tot = 0.0;
    if (r.vec) {
        // 16-byte accesses from the first element on a 16-byte boundary; up to three single
        // elements before it and after the last full group (none when the block length is a
        // multiple of four)
        const int64_t lead = piece_lead(r), nvec = (r.n - lead) & ~int64_t(3);
        float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
        int chain = 0;
        if (threadIdx.x < lead) {
            const float g = load_g1<GD>(r.t->g, r.start + threadIdx.x, gscale);
            a0 = fmaf(g, g, a0);
        }
        for (int64_t i = lead + nvec + threadIdx.x; i < r.n; i += kThreads) {
            const float g = load_g1<GD>(r.t->g, r.start + i, gscale);
            a1 = fmaf(g, g, a1);
        }
        for (int64_t i = lead + static_cast<int64_t>(threadIdx.x) * 4; i < lead + nvec; i += kThreads * 4) {
            const float4 g = load_g4<GD>(r.t->g, r.start + i, gscale);
            a0 = fmaf(g.x, g.x, a0); a1 = fmaf(g.y, g.y, a1);
            a2 = fmaf(g.z, g.z, a2); a3 = fmaf(g.w, g.w, a3);
            if (++chain == 64) {
                tot += (static_cast<double>(a0) + static_cast<double>(a1)) +
                       (static_cast<double>(a2) + static_cast<double>(a3));
                a0 = a1 = a2 = a3 = 0.f;
                chain = 0;
            }
        }
        tot += (static_cast<double>(a0) + static_cast<double>(a1)) +
               (static_cast<double>(a2) + static_cast<double>(a3));
    } else {
        float a = 0.f;
        int chain = 0;
        for (int64_t i = threadIdx.x; i < r.n; i += kThreads) {
            const float g = load_g1<GD>(r.t->g, r.start + i, gscale);
            a = fmaf(g, g, a);
            if (++chain == 64) { tot += static_cast<double>(a); a = 0.f; chain = 0; }
        }
        tot += static_cast<double>(a);
    }
    return tot;
}

// Max, min or sum of (g*g)^2 over one piece (the ablation statistics): plain
// double accumulation per thread; these variants are not performance paths.
template <int GD>
__device__ __forceinline__ double piece_statistic(const PieceRef &r, float gscale, int statistic) {
    double acc = stat_identity(statistic);
    for (int64_t i = threadIdx.x; i < r.n; i += kThreads)
        acc = stat_combine(acc, stat_term(load_g1<GD>(r.t->g, r.start + i, gscale), statistic), statistic);
    return acc;
}

__global__ void __launch_bounds__(kThreads)
twopass_partial_kernel(const DevTensor *__restrict__ tensors, const Seg *__restrict__ segs, int n_segs,
                       double *__restrict__ partials, float gscale_host, const float *gscale_dev,
                       const float *skip_flag, int statistic) {
    __shared__ double warp_part[kThreads / 32];
    if (step_skipped(skip_flag)) return;
    const float gscale = effective_gscale(gscale_host, gscale_dev);
    const PieceRef r = decode_piece(tensors, segs, n_segs, blockIdx.x);
    const bool plain_sum = statistic == 0 || statistic == 3;       // both need the sum of g*g
    double w;
    if (plain_sum)
        w = warp_sum(r.t->gdtype == AM_BF16 ? piece_sum_sq<AM_BF16>(r, gscale) : piece_sum_sq<AM_F32>(r, gscale));
    else
        w = warp_stat(r.t->gdtype == AM_BF16 ? piece_statistic<AM_BF16>(r, gscale, statistic)
                                             : piece_statistic<AM_F32>(r, gscale, statistic), statistic);
    if ((threadIdx.x & 31) == 0) warp_part[threadIdx.x >> 5] = w;
    __syncthreads();
    if (threadIdx.x == 0) {
        double s = warp_part[0];
#pragma unroll
        for (int k = 1; k < kThreads / 32; ++k) s = plain_sum ? s + warp_part[k] : stat_combine(s, warp_part[k], statistic);
        partials[r.t->piece_base + r.local] = s;
    }
}

// One warp per block: fixed-order sum of the block's partials, then v_b and
// the block's step size.
__global__ void __launch_bounds__(kThreads)
twopass_finalize_kernel(const DevTensor *__restrict__ tensors, const Seg *__restrict__ segs, int n_segs,
                        int64_t n_units, const double *__restrict__ partials,
                        float *__restrict__ block_steps, float *__restrict__ v, StepScalars sc) {
    const int64_t unit = static_cast<int64_t>(blockIdx.x) * (kThreads / 32) + (threadIdx.x >> 5);
    if (unit >= n_units || step_skipped(sc.skip_flag)) return;
    const int lane = threadIdx.x & 31;
    const Seg seg = segs[find_seg_warp(segs, n_segs, unit)];
    const DevTensor &t = tensors[seg.tensor];
    if (t.pieces_per_block >= kWideBlockPieces) return;      // twopass_finalize_wide_kernel's
    const int64_t b = unit - seg.unit_begin;
    const double *src = partials + t.piece_base + b * t.pieces_per_block;
    const int statistic = sc.statistic;
    double s = stat_identity(statistic);
    for (int64_t j = lane; j < t.pieces_per_block; j += 32) s = stat_combine(s, src[j], statistic);
    s = warp_stat(s, statistic);
    if (lane == 0) {
        if (t.part_index >= 0) {
            // a part of a block: the whole block's sum of g*g comes from outside (unscaled gradients)
            const double gs = static_cast<double>(effective_gscale(sc.gscale, sc.gscale_dev));
            s = sc.part_sums[t.part_index] * gs * gs;
        }
        float vn;
        const float st = block_step_from_statistic(stat_finish(s, static_cast<double>(t.mean_len), statistic),
                                                   v[t.v_offset + b], sc, &vn);
        v[t.v_offset + b] = vn;
        block_steps[t.block_base + b] = st;
    }
}

// Local sums of g*g of the tensors that are parts of blocks: one warp per such
// tensor adds the tensor's partial sums (written by twopass_partial_kernel with
// a gradient scale of 1) in a fixed order.
__global__ void __launch_bounds__(kThreads)
part_sums_kernel(const DevTensor *__restrict__ tensors, const int32_t *__restrict__ part_tensors, int n_parts,
                 const double *__restrict__ partials, double *__restrict__ out) {
    const int unit = blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5);
    if (unit >= n_parts) return;
    const int lane = threadIdx.x & 31;
    const DevTensor &t = tensors[part_tensors[unit]];
    const double *src = partials + t.piece_base;
    double s = 0.0;
    for (int64_t j = lane; j < t.pieces_per_block; j += 32) s += src[j];
    s = warp_sum(s);
    if (lane == 0) out[unit] = s;
}

// One CTA per block, for blocks with many partial sums (a whole large tensor as
// one block): every thread adds a strided share, then a fixed-order tree.
__global__ void __launch_bounds__(kThreads)
twopass_finalize_wide_kernel(const DevTensor *__restrict__ tensors, const Seg *__restrict__ segs, int n_segs,
                             const double *__restrict__ partials, float *__restrict__ block_steps,
                             float *__restrict__ v, StepScalars sc) {
    __shared__ double warp_part[kThreads / 32];
    if (step_skipped(sc.skip_flag)) return;
    const int64_t unit = blockIdx.x;
    const Seg seg = segs[find_seg_warp(segs, n_segs, unit)];
    const DevTensor &t = tensors[seg.tensor];
    const int64_t b = unit - seg.unit_begin;
    const double *src = partials + t.piece_base + b * t.pieces_per_block;
    const int statistic = sc.statistic;
    double s = stat_identity(statistic);
    for (int64_t j = threadIdx.x; j < t.pieces_per_block; j += kThreads) s = stat_combine(s, src[j], statistic);
    s = warp_stat(s, statistic);
    if ((threadIdx.x & 31) == 0) warp_part[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        s = warp_part[0];
#pragma unroll
        for (int k = 1; k < kThreads / 32; ++k) s = stat_combine(s, warp_part[k], statistic);
        if (t.part_index >= 0) {
            const double gs = static_cast<double>(effective_gscale(sc.gscale, sc.gscale_dev));
            s = sc.part_sums[t.part_index] * gs * gs;
        }
        float vn;
        const float st = block_step_from_statistic(stat_finish(s, static_cast<double>(t.mean_len), statistic),
                                                   v[t.v_offset + b], sc, &vn);
        v[t.v_offset + b] = vn;
        block_steps[t.block_base + b] = st;
    }
}

template <int GD>
__device__ __forceinline__ void twopass_update_body(const PieceRef &r, const float *__restrict__ block_steps,
                                                    const StepScalars &sc) {
    const DevTensor &t = *r.t;
    const float st = block_steps[t.block_base + r.block];
    const float lr_wd = t.wd ? sc.lr_wd : 0.f;
    const float gscale = effective_gscale(sc.gscale, sc.gscale_dev);
    if (r.vec) {
        const int64_t lead = piece_lead(r), nvec = (r.n - lead) & ~int64_t(3);
        for (int64_t i = lead + static_cast<int64_t>(threadIdx.x) * 4; i < lead + nvec; i += kThreads * 4) {
            const int64_t e = r.start + i;
            const float4 g = load_g4<GD>(t.g, e, gscale);
            float4 m = *reinterpret_cast<const float4 *>(t.m + e);
            float4 p = *reinterpret_cast<const float4 *>(t.p + e);
            update_four(g, m, p, sc.beta1, sc.omb1, lr_wd, st);
            *reinterpret_cast<float4 *>(t.m + e) = m;
            *reinterpret_cast<float4 *>(t.p + e) = p;
            if (t.p_bf16) store_bf16x4(t.p_bf16 + e, p);
        }
        // the up to three single elements either side
        for (int64_t i = threadIdx.x; i < r.n - nvec; i += kThreads) {
            const int64_t e = r.start + (i < lead ? i : i + nvec);
            const float g = load_g1<GD>(t.g, e, gscale);
            float m = t.m[e], p = t.p[e];
            update_one(g, m, p, sc.beta1, sc.omb1, lr_wd, st);
            t.m[e] = m;
            t.p[e] = p;
            if (t.p_bf16) store_bf16(t.p_bf16 + e, p);
        }
    } else {
        for (int64_t i = threadIdx.x; i < r.n; i += kThreads) {
            const int64_t e = r.start + i;
            const float g = load_g1<GD>(t.g, e, gscale);
            float m = t.m[e], p = t.p[e];
            update_one(g, m, p, sc.beta1, sc.omb1, lr_wd, st);
            t.m[e] = m;
            t.p[e] = p;
            if (t.p_bf16) store_bf16(t.p_bf16 + e, p);
        }
    }
}

__global__ void __launch_bounds__(kThreads, 5)
twopass_update_kernel(const DevTensor *__restrict__ tensors, const Seg *__restrict__ segs, int n_segs,
                      const float *__restrict__ block_steps, StepScalars sc) {
    if (step_skipped(sc.skip_flag)) return;
    const PieceRef r = decode_piece(tensors, segs, n_segs, blockIdx.x);
    if (r.t->gdtype == AM_BF16) twopass_update_body<AM_BF16>(r, block_steps, sc);
    else twopass_update_body<AM_F32>(r, block_steps, sc);
}

}  // namespace am

#endif  // ADAMMINI_KERNELS_BASIC_CUH_
