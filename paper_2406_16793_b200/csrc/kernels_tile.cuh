// Blocks that the streaming kernels do not take: short ones (block length
// <= 64) and those of up to 4096 elements whose length breaks the 16-byte
// alignment of block starts.  float32 scalars throughout.
//
// A CTA handles one tile: a run of whole blocks of one tensor, up to 4096
// elements, starting wherever the first block starts.  One thread starts three
// bulk asynchronous copies (the 32-byte aligned middle of the tile's g, m and p;
// completion counted on an mbarrier), so that about 50 KB per CTA are in flight
// without holding a register; the up to seven elements before and after the
// aligned middle come by plain loads, and every thread fetches the old v of its
// blocks meanwhile.  Then the block sums (Algorithm 1: v = (1-beta2) mean(g*g) +
// beta2 v):
//   L <= 64: the gradients are first widened and scaled into float rows padded to
//            an odd stride (no bank conflicts), then one thread adds up a block;
//   L  > 64: eight lanes per block (up to 256 elements); beyond, one to eight
//            warps per block, each adding a slice, so that every warp is busy.
//            Lanes walk a block with stride one, so they read the gradients as
//            they arrived (widened and scaled on the fly): no second copy in
//            shared memory and one barrier less than for short blocks.
// The block's step size stays in shared memory, and all threads update the
// tile's elements from shared memory and write m and p back with coalesced
// 16-byte stores (single elements up to the first 16-byte boundary and after the
// last).  g is read from HBM once.
//
// The wait on the mbarrier is bounded like those of the streaming kernels.
#ifndef ADAMMINI_KERNELS_TILE_CUH_
#define ADAMMINI_KERNELS_TILE_CUH_

#include <cuda_runtime.h>

#include "adammini_internal.h"
#include "kernels_basic.cuh"
#include "kernels_stream.cuh"

namespace am {

constexpr int kTileElems = 4096;         // elements per tile of blocks longer than kSmallMaxL ...
constexpr int kTileShortElems = 3072;    // ... and of shorter ones,
constexpr int kTileMaxBlocks = 1024;     // with at most this many blocks
constexpr int kTileMaxL = 4096;          // longest block the kernel takes
constexpr int kTileLinear = kTileElems + 8;            // a tile in shared memory, shifted by up to 7 elements
constexpr int kTileShortLinear = kTileShortElems + 8;
constexpr int kTileWords = 3840;         // >= blocks * (L | 1) for every tile of blocks of up to kSmallMaxL elements
// Shared memory: m, p and the gradients as they arrive (`linear` words each), the step sizes, the
// mbarrier and, last, the widened gradient rows that only blocks of up to kSmallMaxL elements use.
// Tiles of short and of longer blocks are launched separately, each kind with what it needs, so
// that four CTAs fit an SM.
constexpr int kTileSmemLongBytes = (3 * kTileLinear + kTileMaxBlocks) * 4 + 16;
constexpr int kTileSmemShortBytes = (3 * kTileShortLinear + kTileMaxBlocks + kTileWords) * 4 + 16;
constexpr int kTileSmemBytes = kTileSmemShortBytes > kTileSmemLongBytes ? kTileSmemShortBytes : kTileSmemLongBytes;
constexpr int kTileTimeoutCode = 7;

// Blocks per tile.  Short blocks: a multiple of eight, so that every tile starts
// on a 32-byte boundary; longer ones: as many as fit.
__host__ __device__ inline int tile_blocks(int64_t L) {
    if (L > kSmallMaxL) return static_cast<int>(kTileElems / L < 1 ? 1 : kTileElems / L);
    int64_t nb = kTileShortElems / L;
    if (nb > kTileMaxBlocks) nb = kTileMaxBlocks;
    return static_cast<int>(nb & ~int64_t(7));
}

// i / L for 0 <= i < 2^32 / L by one multiplication: magic = floor((2^32 - 1) / L) + 1 (L >= 2).
// Exact because i * (magic * L - 2^32) < 2^32 for every index of a tile.
__device__ __forceinline__ int tile_div(int i, int L, uint32_t magic) {
    return L == 1 ? i : static_cast<int>(__umulhi(static_cast<uint32_t>(i), magic));
}

template <int GD>
__device__ __forceinline__ float tile_raw_at(const unsigned char *sraw, int j) {
    if (GD == AM_BF16) return __uint_as_float(static_cast<uint32_t>(reinterpret_cast<const uint16_t *>(sraw)[j]) << 16);
    return reinterpret_cast<const float *>(sraw)[j];
}

template <int GD, bool LONG>
__device__ __forceinline__ void tile_body(const DevTensor &t, int64_t tile, float *__restrict__ v,
                                          const SmallScalars &sc, int *error_word, float *sm, float *sp,
                                          unsigned char *sraw, float *sg, float *sstep, unsigned long long *bar) {
    constexpr int gsz = GD == AM_BF16 ? 2 : 4;
    const int L = static_cast<int>(t.L);
    constexpr bool short_rows = !LONG;           // LONG: L > kSmallMaxL
    const int Ls = L | 1;                        // row stride of the widened gradients (short blocks only)
    const int per_tile = tile_blocks(L);
    const int64_t b0 = tile * per_tile;
    const int64_t left = t.n_blocks - b0;
    const int nb = static_cast<int>(left < per_tile ? left : per_tile);
    const int64_t e0 = b0 * L;
    const int n = nb * L;
    // element i of the tile sits at index i + shift of the linear arrays, so that the
    // 32-byte aligned part of global memory lands 32-byte aligned in shared memory
    const int shift = static_cast<int>(e0 & 7);
    const int head = min(n, (8 - shift) & 7);            // elements before the first 32-byte boundary
    const int nbulk = (n - head) & ~7;                   // the aligned middle
    const int lead = min(n, (4 - static_cast<int>(e0 & 3)) & 3);   // elements before the first 16-byte boundary
    const int nvec = (n - lead) & ~3;                    // elements updated four at a time
    const float lr_wd = t.wd ? sc.lr_wd : 0.f;
    const float gscale = effective_gscale(sc.gscale, sc.gscale_dev);
    float *mg = t.m + e0, *pg = t.p + e0;
    const unsigned char *gg = static_cast<const unsigned char *>(t.g) + e0 * gsz;
    // long rows: 8 lanes add up a block of up to 256 elements, a whole warp a longer one
    const int glanes = L <= 256 ? 8 : 32, groups = kThreads / glanes;
    const uint32_t magic = L == 1 ? 0u : 0xffffffffu / static_cast<uint32_t>(L) + 1u;

    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (nbulk > 0) {
            mbar_arrive_expect_tx(bar, static_cast<uint32_t>(nbulk) * (gsz + 8));
            if (!sc.stall) {        // (test hook: bytes announced that never arrive make the wait below run out)
                bulk_load(sraw + (shift + head) * gsz, gg + head * gsz, nbulk * gsz, bar);
                bulk_load(sm + shift + head, mg + head, nbulk * 4, bar);
                bulk_load(sp + shift + head, pg + head, nbulk * 4, bar);
            }
        }
    }
    // the ends, by plain loads
    for (int i = threadIdx.x; i < n - nbulk; i += kThreads) {
        const int k = i < head ? i : i + nbulk;
        sm[k + shift] = mg[k];
        sp[k + shift] = pg[k];
        if (GD == AM_BF16) reinterpret_cast<uint16_t *>(sraw)[k + shift] = reinterpret_cast<const uint16_t *>(gg)[k];
        else reinterpret_cast<float *>(sraw)[k + shift] = reinterpret_cast<const float *>(gg)[k];
    }
    // the old v of this thread's (short rows) or this warp's blocks, fetched while the copies fly
    float *vt = v + t.v_offset + b0;
    float v_old[kTileMaxBlocks / kThreads];
#pragma unroll
    for (int r = 0; r < kTileMaxBlocks / kThreads; ++r) v_old[r] = 0.f;
    if (short_rows) {
#pragma unroll
        for (int r = 0; r < kTileMaxBlocks / kThreads; ++r) {
            const int b = threadIdx.x + r * kThreads;
            if (b < nb) v_old[r] = vt[b];
        }
    } else if (glanes == 8) {
        // a group of eight lanes per block; the group's lane r holds the old v of the group's r-th block
        const int b = threadIdx.x / glanes + (threadIdx.x % glanes) * groups;
        if (b < nb) v_old[0] = vt[b];
    } else if (threadIdx.x < nb) {
        v_old[0] = vt[threadIdx.x];              // at most 15 blocks of more than 256 elements: thread b finishes block b
    }
    __syncthreads();                             // the barrier exists; the ends are in place
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
                if (waited > sc.wait_limit_ns) { ok = false; break; }
            }
        }
        if (!ok) {
            // give up: report, let the copies land (again bounded) before the CTA's memory is released, leave
            *reinterpret_cast<volatile int *>(error_word) = kTileTimeoutCode;
            const unsigned long long t0 = global_ns();
            const unsigned long long drain = sc.wait_limit_ns < kDrainTimeoutNs ? sc.wait_limit_ns : kDrainTimeoutNs;
            while (!mbar_try_wait(bar, 0) && global_ns() - t0 < drain) {}
            return;
        }
    }

    // element k of the tile's block b, widened and scaled, straight from the gradients as they arrived
    auto graw = [&](int b, int k) { return tile_raw_at<GD>(sraw, b * L + k + shift) * gscale; };
    if (short_rows) {
        // gradients, widened and scaled -> rows: block b of the tile at sg[b * Ls ...]
        for (int i = threadIdx.x; i < lead; i += kThreads) {
            const int b = tile_div(i, L, magic);
            sg[b * Ls + (i - b * L)] = tile_raw_at<GD>(sraw, i + shift) * gscale;
        }
        for (int i = lead + threadIdx.x * 4; i < lead + nvec; i += kThreads * 4) {
            const float4 g = lds_g4<GD>(sraw, i + shift);            // (i + shift) is a multiple of four
            const float x[4] = {g.x, g.y, g.z, g.w};
            int b = tile_div(i, L, magic), k = i - b * L;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                sg[b * Ls + k] = x[j] * gscale;
                if (++k == L) { k = 0; ++b; }
            }
        }
        for (int i = lead + nvec + threadIdx.x; i < n; i += kThreads) {
            const int b = tile_div(i, L, magic);
            sg[b * Ls + (i - b * L)] = tile_raw_at<GD>(sraw, i + shift) * gscale;
        }
        __syncthreads();
    }

    // block statistics, v and the blocks' step sizes
    if (short_rows) {
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
    } else if (glanes == 8) {
        const int gid = threadIdx.x / glanes, gl = threadIdx.x % glanes;
        const int rounds = (nb + groups - 1) / groups;            // the same for every thread: shuffles stay converged
        for (int r = 0; r < rounds; ++r) {
            const int b = gid + r * groups;
            const bool live = b < nb;
            const int rb = live ? b : 0;
            const float vo = __shfl_sync(0xffffffffu, v_old[0], r, glanes);
            double tot;
            if (sc.statistic == 0 || sc.statistic == 3) {
                // per lane at most 128 terms over four accumulators, then double
                float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
                int k = gl;
                for (; k + 3 * glanes < L; k += 4 * glanes) {
                    const float x0 = graw(rb, k), x1 = graw(rb, k + glanes);
                    const float x2 = graw(rb, k + 2 * glanes), x3 = graw(rb, k + 3 * glanes);
                    s0 = fmaf(x0, x0, s0); s1 = fmaf(x1, x1, s1);
                    s2 = fmaf(x2, x2, s2); s3 = fmaf(x3, x3, s3);
                }
                for (; k < L; k += glanes) { const float x = graw(rb, k); s0 = fmaf(x, x, s0); }
                tot = (static_cast<double>(s0) + static_cast<double>(s1)) + (static_cast<double>(s2) + static_cast<double>(s3));
                for (int o = glanes >> 1; o > 0; o >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, o);
            } else {
                tot = stat_identity(sc.statistic);
                for (int k = gl; k < L; k += glanes) tot = stat_combine(tot, stat_term(graw(rb, k), sc.statistic), sc.statistic);
                for (int o = glanes >> 1; o > 0; o >>= 1)
                    tot = stat_combine(tot, __shfl_xor_sync(0xffffffffu, tot, o), sc.statistic);
            }
            if (live && gl == 0) {
                const float stat = static_cast<float>(stat_finish(tot, static_cast<double>(L), sc.statistic));
                float vn;
                sstep[b] = small_block_step(stat, vo, sc, &vn);
                vt[b] = vn;
            }
        }
    } else {
        // few long blocks: every warp adds up a slice of a block (1, 2, 4 or 8 warps per block, so that
        // all eight warps are busy), then thread b adds the slices of block b in order
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        const int wpb = nb >= 8 ? 1 : nb >= 4 ? 2 : nb >= 2 ? 4 : 8;
        const int slots = nb * wpb, per = (L + wpb - 1) / wpb;
        double *spart = reinterpret_cast<double *>(sstep + 64);          // slots <= 15 partial sums
        const bool plain_sum = sc.statistic == 0 || sc.statistic == 3;
        for (int slot = warp; slot < slots; slot += kThreads / 32) {
            const int b = slot / wpb, sl = slot - b * wpb;
            const int k1 = min(L, (sl + 1) * per);
            double tot;
            if (plain_sum) {
                // per lane at most 128 terms over four accumulators, then double
                float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
                int k = sl * per + lane;
                for (; k + 96 < k1; k += 128) {
                    const float x0 = graw(b, k), x1 = graw(b, k + 32), x2 = graw(b, k + 64), x3 = graw(b, k + 96);
                    s0 = fmaf(x0, x0, s0); s1 = fmaf(x1, x1, s1);
                    s2 = fmaf(x2, x2, s2); s3 = fmaf(x3, x3, s3);
                }
                for (; k < k1; k += 32) { const float x = graw(b, k); s0 = fmaf(x, x, s0); }
                tot = warp_sum((static_cast<double>(s0) + static_cast<double>(s1)) +
                               (static_cast<double>(s2) + static_cast<double>(s3)));
            } else {
                tot = stat_identity(sc.statistic);
                for (int k = sl * per + lane; k < k1; k += 32) tot = stat_combine(tot, stat_term(graw(b, k), sc.statistic), sc.statistic);
                tot = warp_stat(tot, sc.statistic);
            }
            if (lane == 0) spart[slot] = tot;
        }
        __syncthreads();
        if (threadIdx.x < nb) {
            const int b = threadIdx.x;
            double tot = spart[b * wpb];
            for (int j = 1; j < wpb; ++j) tot = stat_combine(tot, spart[b * wpb + j], sc.statistic);
            const float stat = static_cast<float>(stat_finish(tot, static_cast<double>(L), sc.statistic));
            float vn;
            sstep[b] = small_block_step(stat, v_old[0], sc, &vn);
            vt[b] = vn;
        }
    }
    __syncthreads();

    // elementwise update from shared memory; 16-byte stores where global memory allows
    for (int i = threadIdx.x; i < lead; i += kThreads) {
        const int b = tile_div(i, L, magic);
        float m = sm[i + shift], p = sp[i + shift];
        update_one(short_rows ? sg[b * Ls + (i - b * L)] : graw(0, i), m, p, sc.beta1, sc.omb1, lr_wd, sstep[b]);
        mg[i] = m;
        pg[i] = p;
        if (t.p_bf16) store_bf16(t.p_bf16 + e0 + i, p);
    }
    for (int i = lead + threadIdx.x * 4; i < lead + nvec; i += kThreads * 4) {
        float4 m = *reinterpret_cast<const float4 *>(sm + i + shift);
        float4 p = *reinterpret_cast<const float4 *>(sp + i + shift);
        float *mm[4] = {&m.x, &m.y, &m.z, &m.w}, *pp[4] = {&p.x, &p.y, &p.z, &p.w};
        int b = tile_div(i, L, magic), k = i - b * L;
        float x[4] = {0.f, 0.f, 0.f, 0.f};
        if (!short_rows) {
            const float4 g = lds_g4<GD>(sraw, i + shift);            // (i + shift) is a multiple of four
            x[0] = g.x * gscale; x[1] = g.y * gscale; x[2] = g.z * gscale; x[3] = g.w * gscale;
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            update_one(short_rows ? sg[b * Ls + k] : x[j], *mm[j], *pp[j], sc.beta1, sc.omb1, lr_wd, sstep[b]);
            if (++k == L) { k = 0; ++b; }
        }
        *reinterpret_cast<float4 *>(mg + i) = m;
        *reinterpret_cast<float4 *>(pg + i) = p;
        if (t.p_bf16) store_bf16x4(t.p_bf16 + e0 + i, p);
    }
    for (int i = lead + nvec + threadIdx.x; i < n; i += kThreads) {
        const int b = tile_div(i, L, magic);
        float m = sm[i + shift], p = sp[i + shift];
        update_one(short_rows ? sg[b * Ls + (i - b * L)] : graw(0, i), m, p, sc.beta1, sc.omb1, lr_wd, sstep[b]);
        mg[i] = m;
        pg[i] = p;
        if (t.p_bf16) store_bf16(t.p_bf16 + e0 + i, p);
    }
}

__global__ void __launch_bounds__(kThreads)
tile_kernel(const DevTensor *__restrict__ tensors, const Seg *__restrict__ segs, int n_segs,
            float *__restrict__ v, SmallScalars sc, int *error_word, int linear, int64_t first_unit) {
    // linear: kTileLinear (kTileSmemLongBytes, no sg) or kTileShortLinear (kTileSmemShortBytes); the grid covers
    // the tiles from first_unit on
    extern __shared__ __align__(128) unsigned char tile_smem[];
    float *sm = reinterpret_cast<float *>(tile_smem);
    float *sp = sm + linear;
    unsigned char *sraw = reinterpret_cast<unsigned char *>(sp + linear);
    float *sstep = reinterpret_cast<float *>(sraw) + linear;
    unsigned long long *bar = reinterpret_cast<unsigned long long *>(sstep + kTileMaxBlocks);
    float *sg = reinterpret_cast<float *>(bar + 2);
    if (step_skipped(sc.skip_flag)) return;
    const int64_t unit = first_unit + blockIdx.x;
    const Seg seg = segs[find_seg_warp(segs, n_segs, unit)];
    const DevTensor &t = tensors[seg.tensor];
    const int64_t tile = unit - seg.unit_begin;
    if (t.L > kSmallMaxL) {
        if (t.gdtype == AM_BF16) tile_body<AM_BF16, true>(t, tile, v, sc, error_word, sm, sp, sraw, sg, sstep, bar);
        else tile_body<AM_F32, true>(t, tile, v, sc, error_word, sm, sp, sraw, sg, sstep, bar);
    } else {
        if (t.gdtype == AM_BF16) tile_body<AM_BF16, false>(t, tile, v, sc, error_word, sm, sp, sraw, sg, sstep, bar);
        else tile_body<AM_F32, false>(t, tile, v, sc, error_word, sm, sp, sraw, sg, sstep, bar);
    }
}

}  // namespace am

#endif  // ADAMMINI_KERNELS_TILE_CUH_
