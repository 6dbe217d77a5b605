// Short blocks (block length <= 64, any alignment), float32 scalars throughout.
//
// A CTA handles one tile of whole blocks (up to 4096 elements).  One thread
// starts three bulk asynchronous copies (g, m and p of the tile, completion
// counted on an mbarrier), so that about 50 KB per CTA are in flight without
// holding a register.  When they have landed, the gradients are widened and
// re-laid into rows padded to an odd stride, one thread per block adds up its
// row (Algorithm 1: v = (1-beta2) mean(g*g) + beta2 v; no bank conflicts thanks
// to the odd stride) and leaves the block's step size in shared memory, and all
// threads update the tile's elements from shared memory and write m and p back
// with coalesced 16-byte stores.  g is read from HBM once.
//
// The wait on the mbarrier is bounded like those of the streaming kernels.
#ifndef ADAMMINI_KERNELS_TILE_CUH_
#define ADAMMINI_KERNELS_TILE_CUH_

#include <cuda_runtime.h>

#include "adammini_internal.h"
#include "kernels_basic.cuh"
#include "kernels_stream.cuh"

namespace am {

constexpr int kTileElems = 4096;         // elements per tile ...
constexpr int kTileMaxBlocks = 1024;     // ... and at most this many blocks
constexpr int kTileWords = 5120;         // >= blocks * (L | 1) for every L <= kSmallMaxL
// shared memory: m, p, the raw gradients, the padded gradient rows, the step sizes, the mbarrier
constexpr int kTileSmemBytes = (3 * kTileElems + kTileWords + kTileMaxBlocks) * 4 + 16;
constexpr int kTileTimeoutCode = 7;

// Blocks per tile: a multiple of eight, so that every tile starts on a 16-byte
// boundary whatever the block length and the gradient type.
__host__ __device__ inline int tile_blocks(int64_t L) {
    int64_t nb = kTileElems / L;
    if (nb > kTileMaxBlocks) nb = kTileMaxBlocks;
    return static_cast<int>(nb & ~int64_t(7));
}

template <int GD>
__device__ __forceinline__ void tile_body(const DevTensor &t, int64_t tile, float *__restrict__ v,
                                          const SmallScalars &sc, int *error_word, float *sm, float *sp,
                                          unsigned char *sraw, float *sg, float *sstep, unsigned long long *bar) {
    constexpr int gsz = GD == AM_BF16 ? 2 : 4;
    const int L = static_cast<int>(t.L), Ls = L | 1;
    const int per_tile = tile_blocks(L);
    const int64_t b0 = tile * per_tile;
    const int64_t left = t.n_blocks - b0;
    const int nb = static_cast<int>(left < per_tile ? left : per_tile);
    const int64_t e0 = b0 * L;                   // a multiple of eight elements
    const int n = nb * L;
    const int nbulk = n & ~7;                    // a ragged last tile ends with up to seven single elements
    const float lr_wd = t.wd ? sc.lr_wd : 0.f;
    const float gscale = effective_gscale(sc.gscale, sc.gscale_dev);
    float *mg = t.m + e0, *pg = t.p + e0;
    const unsigned char *gg = static_cast<const unsigned char *>(t.g) + e0 * gsz;

    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (nbulk > 0) {
            mbar_arrive_expect_tx(bar, static_cast<uint32_t>(nbulk) * (gsz + 8));
            bulk_load(sraw, gg, nbulk * gsz, bar);
            bulk_load(sm, mg, nbulk * 4, bar);
            bulk_load(sp, pg, nbulk * 4, bar);
        }
    }
    // the ragged end, by plain loads
    for (int i = nbulk + threadIdx.x; i < n; i += kThreads) {
        sm[i] = mg[i];
        sp[i] = pg[i];
        if (GD == AM_BF16) reinterpret_cast<uint16_t *>(sraw)[i] = reinterpret_cast<const uint16_t *>(gg)[i];
        else reinterpret_cast<float *>(sraw)[i] = reinterpret_cast<const float *>(gg)[i];
    }
    // the old v of this thread's blocks, fetched while the copies fly
    float *vt = v + t.v_offset + b0;
    float v_old[kTileMaxBlocks / kThreads];
#pragma unroll
    for (int r = 0; r < kTileMaxBlocks / kThreads; ++r) {
        const int b = threadIdx.x + r * kThreads;
        v_old[r] = b < nb ? vt[b] : 0.f;
    }
    __syncthreads();                             // the barrier exists; the ragged end is in place
    if (nbulk > 0) {
        // bounded wait for the copies (phase 0 of the barrier)
        unsigned spins = 0;
        unsigned long long last = 0, waited = 0;
        bool ok = true;
        while (!mbar_try_wait(bar, 0)) {
            if ((++spins & 255u) == 0) {
                const unsigned long long now = global_ns();
                if (last != 0) {
                    const unsigned long long gap = now - last;
                    waited += gap < kWaitGapCapNs ? gap : kWaitGapCapNs;
                }
                last = now;
                if (waited > kWaitTimeoutNs) { ok = false; break; }
            }
        }
        if (!ok) {
            // give up: report, let the copies land (again bounded) before the CTA's memory is released, leave
            *reinterpret_cast<volatile int *>(error_word) = kTileTimeoutCode;
            const unsigned long long t0 = global_ns();
            while (!mbar_try_wait(bar, 0) && global_ns() - t0 < kDrainTimeoutNs) {}
            return;
        }
    }

    // gradients, widened and scaled -> rows of odd stride: block b of the tile at sg[b * Ls ...]
    for (int i = threadIdx.x * 4; i < n; i += kThreads * 4) {
        float x[4];
        if (i + 3 < n) {
            const float4 g = lds_g4<GD>(sraw, i);
            x[0] = g.x; x[1] = g.y; x[2] = g.z; x[3] = g.w;
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j)
                x[j] = i + j < n ? (GD == AM_BF16 ? __uint_as_float(static_cast<uint32_t>(reinterpret_cast<const uint16_t *>(sraw)[i + j]) << 16)
                                                  : reinterpret_cast<const float *>(sraw)[i + j])
                                 : 0.f;
        }
        int b = i / L, k = i - b * L;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (i + j < n) sg[b * Ls + k] = x[j] * gscale;
            if (++k == L) { k = 0; ++b; }
        }
    }
    __syncthreads();

    // one thread per block: statistic, v and the block's step size
#pragma unroll
    for (int r = 0; r < kTileMaxBlocks / kThreads; ++r) {
        const int b = threadIdx.x + r * kThreads;
        if (b >= nb) break;
        const float *row = sg + b * Ls;
        float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
        int k = 0;
        for (; k + 3 < L; k += 4) {
            s0 = fmaf(row[k], row[k], s0); s1 = fmaf(row[k + 1], row[k + 1], s1);
            s2 = fmaf(row[k + 2], row[k + 2], s2); s3 = fmaf(row[k + 3], row[k + 3], s3);
        }
        for (; k < L; ++k) s0 = fmaf(row[k], row[k], s0);
        const float sum = (s0 + s1) + (s2 + s3);
        float stat = L == 1 ? sum : __fdiv_rn(sum, static_cast<float>(L));
        if (sc.statistic != 0) {
            // ablation statistics of g*g: max, min, 1-norm, 2-norm
            double acc = stat_identity(sc.statistic);
            for (k = 0; k < L; ++k) acc = stat_combine(acc, stat_term(row[k], sc.statistic), sc.statistic);
            stat = static_cast<float>(stat_finish(acc, static_cast<double>(L), sc.statistic));
        }
        float vn;
        sstep[b] = small_block_step(stat, v_old[r], sc, &vn);
        vt[b] = vn;
    }
    __syncthreads();

    // elementwise update from shared memory, coalesced stores
    const int nvec = n & ~3;
    for (int i = threadIdx.x * 4; i < nvec; i += kThreads * 4) {
        float4 m = *reinterpret_cast<const float4 *>(sm + i);
        float4 p = *reinterpret_cast<const float4 *>(sp + i);
        float *mm[4] = {&m.x, &m.y, &m.z, &m.w}, *pp[4] = {&p.x, &p.y, &p.z, &p.w};
        int b = i / L, k = i - b * L;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            update_one(sg[b * Ls + k], *mm[j], *pp[j], sc.beta1, sc.omb1, lr_wd, sstep[b]);
            if (++k == L) { k = 0; ++b; }
        }
        *reinterpret_cast<float4 *>(mg + i) = m;
        *reinterpret_cast<float4 *>(pg + i) = p;
        if (t.p_bf16) store_bf16x4(t.p_bf16 + e0 + i, p);
    }
    for (int i = nvec + threadIdx.x; i < n; i += kThreads) {
        const int b = i / L;
        float m = sm[i], p = sp[i];
        update_one(sg[b * Ls + (i - b * L)], m, p, sc.beta1, sc.omb1, lr_wd, sstep[b]);
        mg[i] = m;
        pg[i] = p;
        if (t.p_bf16) store_bf16(t.p_bf16 + e0 + i, p);
    }
}

__global__ void __launch_bounds__(kThreads)
tile_kernel(const DevTensor *__restrict__ tensors, const Seg *__restrict__ segs, int n_segs,
            float *__restrict__ v, SmallScalars sc, int *error_word) {
    extern __shared__ __align__(128) unsigned char tile_smem[];      // kTileSmemBytes
    float *sm = reinterpret_cast<float *>(tile_smem);
    float *sp = sm + kTileElems;
    unsigned char *sraw = reinterpret_cast<unsigned char *>(sp + kTileElems);
    float *sg = reinterpret_cast<float *>(sraw) + kTileElems;
    float *sstep = sg + kTileWords;
    unsigned long long *bar = reinterpret_cast<unsigned long long *>(sstep + kTileMaxBlocks);
    if (step_skipped(sc.skip_flag)) return;
    const int64_t unit = blockIdx.x;
    const Seg seg = segs[find_seg(segs, n_segs, unit)];
    const DevTensor &t = tensors[seg.tensor];
    if (t.gdtype == AM_BF16) tile_body<AM_BF16>(t, unit - seg.unit_begin, v, sc, error_word, sm, sp, sraw, sg, sstep, bar);
    else tile_body<AM_F32>(t, unit - seg.unit_begin, v, sc, error_word, sm, sp, sraw, sg, sstep, bar);
}

}  // namespace am

#endif  // ADAMMINI_KERNELS_TILE_CUH_
