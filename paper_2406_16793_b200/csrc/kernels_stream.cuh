// The single-read streaming kernels.
//
// One persistent CTA per SM.  A producer thread takes work items (one at a
// time from a global counter, so that all CTAs stay on one neighbourhood of
// memory and share open DRAM pages; or from a fixed range of its own) and
// moves gradients, first moments, parameters and the blocks' old v from HBM
// into a ring of shared-memory stages with bulk asynchronous copies
// (cp.async.bulk, completion counted on an mbarrier).  The consumer warps,
// in one or two groups that own alternate work items, wait for a stage, reduce
// g*g over each block (Algorithm 1: v = (1-beta2) mean(g*g) + beta2 v), turn
// the block's new v into a step size and apply the elementwise update,
// writing m and p back with 16-byte stores.
//
// Three kinds of stage:
//   PACKED  whole blocks (block_len <= kStageElems) with their g, m and p: g is
//           read from HBM exactly once.
//   SUM     gradients only, for a block longer than a stage: consumers add up
//           g*g; the last SUM stage of a block ends with the reduction (across
//           the CTAs of a cluster through distributed shared memory when the
//           block is split over a cluster).
//   APPLY   g, m, p of one chunk of that block: g is fetched a second time, a
//           few microseconds after the first, and is served by L2.
//
// A block is always reduced in one fixed order (per thread, per warp, per
// group, per cluster rank), whichever CTA or group gets it, so results do not
// depend on the number of CTAs or groups or on how the work was handed out; the
// threads per group and the cluster size fix that order and so can change the
// last bit of a sum.
//
// Blocks longer than a stage whose starts are off the 16-byte grid run in a
// launch of their own (template argument EDGES): the aligned middle of every
// chunk is staged, the few elements either side come from global memory.
//
// Every wait is bounded: a wait that gives up sets the abort flag and the
// handle's error word, and all roles leave through the common exit.
#ifndef ADAMMINI_KERNELS_STREAM_CUH_
#define ADAMMINI_KERNELS_STREAM_CUH_

#include <cuda_runtime.h>

#include <algorithm>
#include <vector>

#include "adammini_internal.h"
#include "kernels_basic.cuh"

namespace am {

constexpr int kStageElems = 4096;                 // elements of g, m, p per PACKED/APPLY stage
constexpr int kWarpBlockMaxL = 1024;              // blocks up to this length are reduced by one warp
constexpr int kCtrlBytes = 2048;                  // barriers, stage descriptors, reduction slots
constexpr int kVAreaFloats = 272;                 // per stage: the old v of the stage's blocks (16-byte windows)
constexpr int kMaxStages = 8;
constexpr int kMaxConsumerWarps = 16;              // over all consumer groups
constexpr int kMaxGroups = 2;                     // consumer groups; each owns every n-th work item
constexpr int kExchangeSlots = 4;                 // slots of the cluster exchange, used in turn by consecutive long blocks
constexpr int kMaxCluster = 8;
constexpr int kItemSlots = 8;                     // block indices in flight from a cluster's first CTA to its peers
constexpr int kStaticRanges = 1000000;            // AM_OPT_STREAM_CHUNK value that selects static ranges
constexpr int kMaxStreamCtas = 4096;              // most persistent CTAs AM_OPT_STREAM_CTAS accepts
constexpr int64_t kStreamMaxBlockBytes = 256 << 10;   // longest block one CTA handles alone (bytes of g)
constexpr int64_t kClusterMaxBlockBytes = 4 << 20;    // longest block a cluster handles (bytes of g)
constexpr unsigned long long kWaitTimeoutNs = 2000000000ull;   // 2 s
constexpr unsigned long long kDrainTimeoutNs = 50000000ull;    // 50 ms
constexpr unsigned long long kWaitGapCapNs = 1000000ull;       // 1 ms: the most one gap between polls adds to a wait

enum StageKind : int32_t { STAGE_PACKED = 0, STAGE_SUM = 1, STAGE_APPLY = 2, STAGE_DONE = 3 };
enum StageFlag : int32_t { SF_BF16 = 1, SF_WD = 2, SF_LAST = 4, SF_WRITE_V = 8, SF_V_STAGED = 16 };

struct StageMeta {          // written by the producer, read by the consumers
    float *m;               // global destination of this stage's first element
    float *p;
    float *v;               // v of the stage's first block
    double inv_L;           // 1 / block length
    int32_t n;              // elements in the stage
    int32_t L;              // block length (PACKED)
    int32_t kind;
    int32_t flags;
    int32_t v_shift;        // SF_V_STAGED: the first block's v sits at this index of the stage's v area
    int32_t group;          // consumer group that processes this stage
    uint16_t *pb;           // bf16 copy of the updated parameters (nullptr: none)
};
static_assert(sizeof(StageMeta) == 64, "stage descriptor is 64 bytes");

// A run of work items of one tensor.  Items are addressed in "slots": an item
// takes as many consecutive slots as it has stages, so that a range of slots is
// about the same amount of work whatever kind of item it holds; the item whose
// first slot lies in a CTA's range belongs to that CTA.
struct StreamSeg {
    int64_t item_begin;     // first slot of the segment
    int32_t tensor;
    int32_t bpi;            // blocks per item (PACKED); 0: one long block per item
    int32_t slots;          // slots per item (1 for PACKED items and for cluster launches)
    int32_t pad;
};

struct StreamParams {
    const DevTensor *tensors;
    const StreamSeg *segs;      // n_segs entries plus a sentinel
    const int64_t *bounds;      // item range of CTA (or cluster) k is [bounds[k], bounds[k+1])
    float *v;
    int *error_word;
    StepScalars sc;
    int32_t n_segs;
    int32_t n_stages;
    int32_t stage_bytes;
    int32_t g_region_bytes;     // m starts here inside a stage; p follows kStageElems floats later
    int32_t consumer_threads;   // per consumer group
    int32_t n_groups;
    int32_t chunk;              // > 0: items are handed out `chunk` at a time from *counter
    unsigned long long *counter;
    unsigned long long *counter_next;   // the counter of this launch shape's NEXT launch: set to zero here (the two alternate)
    int64_t total_items;
    int64_t v_len;              // floats in v (staging never reads past it)
    unsigned long long wait_limit_ns;   // polling time after which a wait gives up
    int32_t stall_after;        // test hook: > 0: the producer withholds its n-th and later stages (n = stall_after)
    int32_t pad;
};

// Long blocks whose starts are off the 16-byte grid: a stage carries the aligned middle of its
// chunk; the up to seven elements before the first stage's chunk and after the last one's do
// not pass through shared memory, the consumers fetch them from global memory.
struct EdgeMeta {
    const void *g;          // global address of the stage's first gradient
    int32_t head, tail;     // elements before / after the stage's chunk that belong to the block (0..7)
};

struct Control {            // first kCtrlBytes of dynamic shared memory
    unsigned long long full[kMaxStages];     // producer -> consumers: the stage's copies have landed
    unsigned long long empty[kMaxStages];    // consumers -> producer: every consumer warp is done with the stage
    unsigned long long redbar[kMaxGroups];   // barrier of one consumer group (an mbarrier, so that waits are bounded)
    unsigned long long xbar[kExchangeSlots]; // cluster exchange: all CTAs' partial sums of a block have arrived
    double red[kMaxGroups][2][kMaxConsumerWarps];   // per-warp partial sums of a group, double buffered
    double xpart[kExchangeSlots][kMaxCluster];      // partial sums of the cluster's CTAs, by rank
    float redv[kMaxGroups][2];               // old v of the block being reduced, broadcast to the group
    int abort_flag;                          // raised by a wait that gave up; every wait polls it
    int pad;
    unsigned long long ibar[kItemSlots];     // cluster launches: "the next block index has arrived"
    long long next_item[kItemSlots];
    StageMeta meta[kMaxStages];
    EdgeMeta edge[kMaxStages];               // launches of unaligned long blocks only
};
static_assert(sizeof(Control) <= kCtrlBytes, "control block fits its reservation");

// ------------------------------- PTX wrappers -------------------------------
__device__ __forceinline__ uint32_t smem_addr(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(void *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(void *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(void *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(void *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_addr(bar)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_try_wait_cluster(void *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_addr(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bulk asynchronous copy global -> shared; bytes and both addresses are multiples of 16.
__device__ __forceinline__ void bulk_load(void *dst_smem, const void *src_gmem, uint32_t bytes, void *bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(smem_addr(dst_smem)), "l"(src_gmem), "r"(bytes), "r"(smem_addr(bar)) : "memory");
}
// The same with an L2 eviction-priority hint (a policy from createpolicy).
__device__ __forceinline__ void bulk_load_hint(void *dst_smem, const void *src_gmem, uint32_t bytes, void *bar,
                                               unsigned long long policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(smem_addr(dst_smem)), "l"(src_gmem), "r"(bytes), "r"(smem_addr(bar)), "l"(policy) : "memory");
}
__device__ __forceinline__ unsigned long long l2_policy_evict_last() {
    unsigned long long p; asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p)); return p;
}
__device__ __forceinline__ unsigned long long l2_policy_evict_first() {
    unsigned long long p; asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p)); return p;
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r;
}
__device__ __forceinline__ uint32_t cluster_nctarank() {
    uint32_t r; asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r)); return r;
}
__device__ __forceinline__ uint32_t cluster_id_x() {
    uint32_t r; asm volatile("mov.u32 %0, %%clusterid.x;" : "=r"(r)); return r;
}
__device__ __forceinline__ uint32_t map_to_rank(uint32_t local_smem_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_smem_addr), "r"(rank));
    return r;
}
// Asynchronous 8-byte store into a peer CTA's shared memory that counts as 8 bytes of
// complete_tx on that CTA's mbarrier: value and signal travel together, no fence on the sender's
// side (a release there waits for every global store the thread still has in flight).
__device__ __forceinline__ void st_async_cluster_b64(uint32_t cluster_addr, unsigned long long bits, uint32_t cluster_bar) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.b64 [%0], %1, [%2];"
                 ::"r"(cluster_addr), "l"(bits), "r"(cluster_bar) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release;\n\tbarrier.cluster.wait.acquire;" ::: "memory");
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t;
}

// Bounded wait on an mbarrier phase.  Returns false (after raising the abort
// flag) if the phase did not complete within the limit or another thread of
// the CTA already gave up.
template <bool CLUSTER_ACQUIRE>
__device__ __forceinline__ bool wait_phase_one(void *bar, uint32_t parity, Control *ctl, int *error_word,
                                               int code, unsigned long long limit_ns) {
    uint32_t spins = 0;
    unsigned long long last = 0, waited = 0;
    for (;;) {
        const bool ok = CLUSTER_ACQUIRE ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity);
        if (ok) return true;
        if ((++spins & 255u) == 0) {
            if (*reinterpret_cast<volatile int *>(&ctl->abort_flag)) return false;
            // Only time spent polling counts: a gap between two checks is capped, so a kernel
            // that was switched out for a while (time slicing, a debugger) does not give up.
            const unsigned long long now = global_ns();
            if (last != 0) {
                const unsigned long long gap = now - last;
                waited += gap < kWaitGapCapNs ? gap : kWaitGapCapNs;
            }
            last = now;
            if (waited > limit_ns) {
                *reinterpret_cast<volatile int *>(&ctl->abort_flag) = 1;
                *reinterpret_cast<volatile int *>(error_word) = code;
                return false;
            }
        }
    }
}
// The same for a whole warp that waits together (the consumers): the lanes agree on the
// outcome, so a warp never splits between going on and giving up.
template <bool CLUSTER_ACQUIRE>
__device__ __forceinline__ bool wait_phase(void *bar, uint32_t parity, Control *ctl, int *error_word,
                                           int code, unsigned long long limit_ns) {
    const bool ok = wait_phase_one<CLUSTER_ACQUIRE>(bar, parity, ctl, error_word, code, limit_ns);
    return __all_sync(0xffffffffu, ok) != 0;
}

// ------------------------- consumer-side building blocks -------------------------
template <int GD>
__device__ __forceinline__ float4 lds_g4(const unsigned char *gs, int i) {
    if (GD == AM_BF16) {
        const uint2 u = *reinterpret_cast<const uint2 *>(gs + 2 * i);
        return make_float4(bf16_lo(u.x), bf16_hi(u.x), bf16_lo(u.y), bf16_hi(u.y));
    } else {
        return *reinterpret_cast<const float4 *>(gs + 4 * i);
    }
}

// Per-block scalars in float (one per block; the sum arrives as a double).
__device__ __forceinline__ float stream_block_step(double sum_sq, double inv_L, float v_old,
                                                   const StepScalars &s, float *v_new) {
    const float mean = static_cast<float>(sum_sq * inv_L);
    const float vn = fmaf(static_cast<float>(s.omb2), mean, static_cast<float>(s.beta2) * v_old);
    *v_new = vn;
    const float denom = __fsqrt_rn(vn * static_cast<float>(s.inv_bc2)) + static_cast<float>(s.eps);
    return __fdiv_rn(static_cast<float>(s.lr_over_bc1), denom);
}

// Elementwise update of n elements (n % 4 == 0) by `nthr` cooperating threads.
// The gradient scale is folded into `omb1` (= (1-beta1) * scale) by the caller.
// CS: write m and p with streaming (evict-first) stores.  Measured: the cluster kernel is faster with
// them (its second fetch of g must still find the first in L2), the row kernel with plain stores.
template <int GD, bool BF16_COPY, bool CS>
__device__ __forceinline__ void apply_span_impl(const unsigned char *gs, const float *ms, const float *ps,
                                                float *mg, float *pg, uint16_t *pb, int first, int n, int tid,
                                                int nthr, float beta1, float omb1, float lr_wd, float step) {
#pragma unroll 2
    for (int i = first + tid * 4; i < first + n; i += nthr * 4) {
        const float4 g = lds_g4<GD>(gs, i);
        float4 m = *reinterpret_cast<const float4 *>(ms + i);
        float4 p = *reinterpret_cast<const float4 *>(ps + i);
        update_four(g, m, p, beta1, omb1, lr_wd, step);
        if (CS) {
            __stcs(reinterpret_cast<float4 *>(mg + i), m);
            __stcs(reinterpret_cast<float4 *>(pg + i), p);
        } else {
            *reinterpret_cast<float4 *>(mg + i) = m;
            *reinterpret_cast<float4 *>(pg + i) = p;
        }
        if (BF16_COPY) store_bf16x4(pb + i, p);
    }
}

template <int GD, bool COPY, bool CS>
__device__ __forceinline__ void apply_span(const unsigned char *gs, const float *ms, const float *ps,
                                           float *mg, float *pg, uint16_t *pb, int first, int n, int tid, int nthr,
                                           float beta1, float omb1, float lr_wd, float step) {
    if (COPY && pb) apply_span_impl<GD, true, CS>(gs, ms, ps, mg, pg, pb, first, n, tid, nthr, beta1, omb1, lr_wd, step);
    else apply_span_impl<GD, false, CS>(gs, ms, ps, mg, pg, pb, first, n, tid, nthr, beta1, omb1, lr_wd, step);
}

// The reduction a launch runs over the g*g of a block.  Algorithm 1 needs the sum (for the mean);
// the ablation of the paper's appendix replaces the mean by the max, the min, the 1-norm (the sum
// again, not divided) or the 2-norm (root of the sum of (g*g)^2) of the vector g*g.
enum StatOp : int { ST_SUM = 0, ST_MAX = 1, ST_MIN = 2, ST_SUM4 = 3 };

__host__ __device__ inline int stat_op_of(int statistic) {      // am_option AM_OPT_STATISTIC -> StatOp
    return statistic == 1 ? ST_MAX : statistic == 2 ? ST_MIN : statistic == 4 ? ST_SUM4 : ST_SUM;
}

// Per-thread accumulator: float, except for the sum of fourth powers, whose terms
// (down to 1e-40 for gradients of 1e-10) are below float's normal range.
template <int ST> struct StatAcc { typedef float T; };
template <> struct StatAcc<ST_SUM4> { typedef double T; };

template <int ST>
__device__ __forceinline__ typename StatAcc<ST>::T stat_acc_init() {
    return ST == ST_MIN ? static_cast<typename StatAcc<ST>::T>(__int_as_float(0x7f800000)) : static_cast<typename StatAcc<ST>::T>(0);
}
template <int ST>
__device__ __forceinline__ void stat_acc_add(typename StatAcc<ST>::T &a, float g) {
    if (ST == ST_SUM) a = fmaf(g, g, a);
    else if (ST == ST_MAX) a = fmaxf(a, g * g);
    else if (ST == ST_MIN) a = fminf(a, g * g);
    else { const double sq = static_cast<double>(g * g); a = static_cast<typename StatAcc<ST>::T>(fma(sq, sq, static_cast<double>(a))); }
}
// Two partial results of the same statistic.
template <int ST>
__device__ __forceinline__ double stat_op_combine(double a, double b) {
    if (ST == ST_MAX) return a > b ? a : b;
    if (ST == ST_MIN) return a < b ? a : b;
    return a + b;
}
// From the reduced value to the statistic's numerator: the block step divides a
// sum by the block length for the mean and takes everything else as it is.
template <int ST>
__device__ __forceinline__ double stat_op_finish(double acc) { return ST == ST_SUM4 ? sqrt(acc) : acc; }

template <int GD, int ST>
__device__ __forceinline__ void sum_span(const unsigned char *gs, int first, int n, int tid, int nthr,
                                         typename StatAcc<ST>::T &a0, typename StatAcc<ST>::T &a1,
                                         typename StatAcc<ST>::T &a2, typename StatAcc<ST>::T &a3) {
#pragma unroll 2
    for (int i = first + tid * 4; i < first + n; i += nthr * 4) {
        const float4 g = lds_g4<GD>(gs, i);
        stat_acc_add<ST>(a0, g.x); stat_acc_add<ST>(a1, g.y);
        stat_acc_add<ST>(a2, g.z); stat_acc_add<ST>(a3, g.w);
    }
}

template <int ST, typename A>
__device__ __forceinline__ double fold4(A a0, A a1, A a2, A a3) {
    return stat_op_combine<ST>(stat_op_combine<ST>(static_cast<double>(a0), static_cast<double>(a1)),
                               stat_op_combine<ST>(static_cast<double>(a2), static_cast<double>(a3)));
}

template <int ST>
__device__ __forceinline__ double warp_combine(double x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x = stat_op_combine<ST>(x, __shfl_xor_sync(0xffffffffu, x, o));
    return x;
}

// State of the consumer group's own barrier (an mbarrier so that it is bounded).
struct GroupSync {
    uint32_t parity;
    int buf;
};

// Combine `mine` over the threads of one consumer group in a fixed order; also
// broadcasts v_old read by the group's first thread.  Returns false on abort.
template <int ST>
__device__ __forceinline__ bool group_reduce(Control *ctl, GroupSync &gs, int *error_word, unsigned long long limit_ns,
                                             int group, int gtid, int n_warps, double mine, const float *v_ptr,
                                             double *total, float *v_old) {
    const double w = warp_combine<ST>(mine);
    const int lane = gtid & 31;
    if (lane == 0) {
        ctl->red[group][gs.buf][gtid >> 5] = w;
        if (gtid == 0) ctl->redv[group][gs.buf] = *v_ptr;
        mbar_arrive(&ctl->redbar[group]);
    }
    if (!wait_phase<false>(&ctl->redbar[group], gs.parity, ctl, error_word, 3, limit_ns)) return false;
    double s = ctl->red[group][gs.buf][0];
    for (int k = 1; k < n_warps; ++k) s = stat_op_combine<ST>(s, ctl->red[group][gs.buf][k]);
    *total = s;
    *v_old = ctl->redv[group][gs.buf];
    gs.parity ^= 1;
    gs.buf ^= 1;
    return true;
}

// ------------------------------------ kernel ------------------------------------
// Template parameters keep the code of one launch small (the consumer loop is
// sensitive to instruction-cache misses): GDM says which gradient dtypes the
// launch's tensors have, COPY whether any tensor wants a bf16 copy, ST the block
// statistic (StatOp; ST_SUM is Algorithm 1's mean), EDGES that the launch's blocks are
// long ones that start off the 16-byte grid (see EdgeMeta).
enum GradMode : int { GDM_F32 = 0, GDM_BF16 = 1, GDM_MIXED = 2 };

template <bool CLUSTER, int GDM, bool COPY, int ST, bool EDGES>
__global__ void __launch_bounds__(32 + kMaxConsumerWarps * 32, 1)
stream_kernel(const __grid_constant__ StreamParams P) {
    static_assert(!(EDGES && CLUSTER), "unaligned long blocks are handled by single CTAs");
    typedef typename StatAcc<ST>::T Acc;
    extern __shared__ __align__(128) unsigned char smem[];
    // The work counter of the next launch of this shape starts at zero: the launch before this one
    // used it and has ended (launches of one handle are ordered), so no separate clearing is enqueued.
    if (blockIdx.x == 0 && threadIdx.x == 0 && P.counter_next) *P.counter_next = 0ull;
    if (step_skipped(P.sc.skip_flag)) return;      // uniform over the grid: nobody reaches a barrier
    Control *ctl = reinterpret_cast<Control *>(smem);
    unsigned char *stages = smem + kCtrlBytes;
    float *v_areas = reinterpret_cast<float *>(stages + static_cast<size_t>(P.n_stages) * P.stage_bytes);
    const int tid = threadIdx.x;
    const int n_gwarps = P.consumer_threads >> 5;          // warps of one consumer group
    const int n_cwarps = n_gwarps * P.n_groups;
    const uint32_t crank = CLUSTER ? cluster_ctarank() : 0;
    const uint32_t csize = CLUSTER ? cluster_nctarank() : 1;
    const uint32_t unit = CLUSTER ? cluster_id_x() : blockIdx.x;

    if (tid == 0) {
        for (int s = 0; s < P.n_stages; ++s) {
            mbar_init(&ctl->full[s], 1);
            mbar_init(&ctl->empty[s], n_cwarps);
        }
        for (int k = 0; k < kMaxGroups; ++k) mbar_init(&ctl->redbar[k], n_gwarps);
        for (int k = 0; k < kExchangeSlots; ++k) mbar_init(&ctl->xbar[k], 1);      // armed by its own CTA, completed by the peers' bytes
        for (int k = 0; k < kItemSlots; ++k) mbar_init(&ctl->ibar[k], 1);
        ctl->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (CLUSTER) cluster_sync_all();     // peers' barriers exist before anyone arrives on them

    const int64_t item_lo = P.bounds[unit], item_hi = P.bounds[unit + 1];

    if (tid < 32) {
        // ------------------------------ producer ------------------------------
        if (tid == 0) {
            int stage = 0;
            uint32_t phase = 0;
            int64_t armed = 0;              // stages armed so far
            int32_t item_group = 0;         // consumer group of the current item (items alternate)
            const unsigned long long keep_in_l2 = l2_policy_evict_last(), drop_from_l2 = l2_policy_evict_first();
            bool ok = true;
            int seg = 0;
            if (P.chunk <= 0) {
                int lo = 0, hi = P.n_segs - 1;      // last segment starting at or before item_lo
                while (lo < hi) {
                    const int mid = (lo + hi + 1) >> 1;
                    if (P.segs[mid].item_begin <= item_lo) lo = mid; else hi = mid - 1;
                }
                seg = lo;
            }
            // (test hook: from the stall_after-th stage on the producer behaves as if its wait had
            // failed, without raising the abort flag: it arms nothing more, sends no DONE, lets its
            // copies land and leaves, so that the consumers' next wait runs out)
            auto acquire = [&]() -> bool {
                if (P.stall_after > 0 && armed >= P.stall_after - 1) return false;
                return wait_phase_one<false>(&ctl->empty[stage], phase ^ 1u, ctl, P.error_word, 1, P.wait_limit_ns);
            };
            auto advance = [&]() {
                ++armed;
                if (++stage == P.n_stages) { stage = 0; phase ^= 1u; }
            };
            // Old v of blocks [first, first+count) of v, copied as whole 16-byte
            // windows next to the stage; skipped (consumers then read v from
            // global memory) when the last window would reach past the end of v.
            auto stage_v = [&](StageMeta &mt, int64_t first, int count) -> uint32_t {
                const int64_t w0 = first & ~int64_t(3), w1 = (first + count + 3) & ~int64_t(3);
                if (w1 > P.v_len || w1 - w0 > kVAreaFloats) return 0u;
                mt.flags |= SF_V_STAGED;
                mt.v_shift = static_cast<int32_t>(first - w0);
                return static_cast<uint32_t>(w1 - w0) * 4u;
            };
            // Static mode: the CTA's (or cluster's) own contiguous range.  Dynamic mode:
            // a single CTA takes ranges of `chunk` items from a global counter, the next
            // range requested while the current one is being issued; in a cluster the
            // first CTA takes one block at a time and hands the index to every CTA of the
            // cluster through distributed shared memory, two blocks ahead.
            const bool dynamic = !CLUSTER && P.chunk > 0;
            const bool cdynamic = CLUSTER && P.chunk > 0;
            uint32_t published = 0, taken = 0;
            // The first CTA asks the counter for a block index when it takes one (two blocks ahead of
            // use) and sends it on after the block's first APPLY stage, by which time the counter has
            // answered; the sends are asynchronous stores that complete the peers' barriers themselves.
            long long pub_idx = 0;
            bool pub_pending = false;
            auto publish_begin = [&]() {
                pub_idx = static_cast<long long>(atomicAdd(P.counter, static_cast<unsigned long long>(P.chunk)));
                pub_pending = true;
            };
            auto publish_finish = [&]() {
                const uint32_t slot = published & (kItemSlots - 1);
                ++published;
                pub_pending = false;
                const uint32_t item = smem_addr(&ctl->next_item[slot]), bar = smem_addr(&ctl->ibar[slot]);
                for (uint32_t r = 0; r < csize; ++r)
                    st_async_cluster_b64(map_to_rank(item, r), static_cast<unsigned long long>(pub_idx), map_to_rank(bar, r));
            };
            auto cluster_publish = [&]() {
                publish_begin();
                publish_finish();
            };
            auto cluster_take = [&]() -> int64_t {
                const uint32_t slot = taken & (kItemSlots - 1), par = (taken / kItemSlots) & 1u;
                ++taken;
                mbar_arrive_expect_tx(&ctl->ibar[slot], 8u);     // (the index may have landed already: the byte count is signed)
                if (!wait_phase_one<true>(&ctl->ibar[slot], par, ctl, P.error_word, 5, P.wait_limit_ns)) { ok = false; return P.total_items; }
                return *reinterpret_cast<volatile long long *>(&ctl->next_item[slot]);
            };
            // The segment an item lies in, and what the stages of its tensor need, are looked up when
            // the walk enters a segment and kept in registers: per item the producer only computes
            // offsets (its time per stage counts: a free stage that is not armed at once is
            // bandwidth not asked for).
            StreamSeg sg = {};
            DevTensor t = {};
            int64_t seg_hi = -1;                    // first slot past the cached segment (-1: nothing cached yet)
            int gsz = 4, base_flags = 0;
            double inv_L = 1.0;
            const unsigned char *gbase = nullptr;
            auto load_segment = [&](int64_t item) {
                while (seg + 1 < P.n_segs && P.segs[seg + 1].item_begin <= item) ++seg;
                sg = P.segs[seg];
                seg_hi = P.segs[seg + 1].item_begin;        // (the table ends with a sentinel)
                t = P.tensors[sg.tensor];
                gsz = t.gdtype == AM_BF16 ? 2 : 4;
                base_flags = (t.gdtype == AM_BF16 ? SF_BF16 : 0) | (t.wd ? SF_WD : 0);
                gbase = static_cast<const unsigned char *>(t.g);
                inv_L = P.sc.statistic == 0 ? 1.0 / static_cast<double>(t.L) : 1.0;
            };
            int64_t it = item_lo, hi = item_hi, next = 0;
            if (dynamic) {
                it = static_cast<int64_t>(atomicAdd(P.counter, static_cast<unsigned long long>(P.chunk)));
                hi = it + P.chunk < P.total_items ? it + P.chunk : P.total_items;
                next = static_cast<int64_t>(atomicAdd(P.counter, static_cast<unsigned long long>(P.chunk)));
            } else if (cdynamic) {
                if (crank == 0) { cluster_publish(); cluster_publish(); }
                it = hi = 0;                    // the loop's first test takes the first block
            }
            for (; ok; ++it) {
                if (it >= hi) {
                    if (cdynamic) {
                        if (pub_pending) publish_finish();
                        it = cluster_take();
                        if (!ok || it >= P.total_items) break;
                        hi = it + P.chunk < P.total_items ? it + P.chunk : P.total_items;
                        if (crank == 0) publish_begin();
                    } else {
                        if (!dynamic || next >= P.total_items) break;
                        it = next;
                        hi = it + P.chunk < P.total_items ? it + P.chunk : P.total_items;
                        next = static_cast<int64_t>(atomicAdd(P.counter, static_cast<unsigned long long>(P.chunk)));
                    }
                }
                if (it >= seg_hi) load_segment(it);     // (items only move forward)
                int64_t local = it - sg.item_begin;
                if (sg.slots > 1) {
                    const int64_t rem = local % sg.slots;
                    if (rem != 0) {             // inside an item that began in somebody else's range
                        it += sg.slots - rem - 1;
                        continue;
                    }
                    local /= sg.slots;
                }
                if (sg.bpi > 0) {
                    const int64_t b0 = local * sg.bpi;
                    const int64_t left = t.n_blocks - b0;
                    const int nb = static_cast<int>(left < sg.bpi ? left : sg.bpi);
                    const int64_t e0 = b0 * t.L;
                    const int n = nb * static_cast<int>(t.L);
                    if (!(ok = acquire())) break;
                    StageMeta &mt = ctl->meta[stage];
                    mt.m = t.m + e0; mt.p = t.p + e0; mt.v = P.v + t.v_offset + b0;
                    mt.pb = t.p_bf16 ? t.p_bf16 + e0 : nullptr; mt.group = item_group;
                    mt.inv_L = inv_L;
                    mt.n = n; mt.L = static_cast<int>(t.L); mt.kind = STAGE_PACKED; mt.flags = base_flags | SF_WRITE_V;
                    const uint32_t vbytes = stage_v(mt, t.v_offset + b0, nb);
                    unsigned char *st = stages + static_cast<size_t>(stage) * P.stage_bytes;
                    mbar_arrive_expect_tx(&ctl->full[stage], static_cast<uint32_t>(n) * (gsz + 8) + vbytes);
                    if (vbytes)
                        bulk_load(v_areas + stage * kVAreaFloats, P.v + ((t.v_offset + b0) & ~int64_t(3)), vbytes,
                                  &ctl->full[stage]);
                    bulk_load(st, gbase + e0 * gsz, n * gsz, &ctl->full[stage]);
                    bulk_load(st + P.g_region_bytes, t.m + e0, n * 4, &ctl->full[stage]);
                    bulk_load(st + P.g_region_bytes + kStageElems * 4, t.p + e0, n * 4, &ctl->full[stage]);
                    advance();
                } else {
                    // one long block; a cluster splits it evenly over its CTAs where the slices then start
                    // on 16-byte boundaries, else (cluster sizes that are no power of two) in multiples of 16 elements
                    // (handing the CTAs of a cluster the block's chunks in turn instead, so that they walk it
                    // side by side, was measured: bf16 heads of 1 MB unchanged, float32 heads of 2 MB 1 % slower)
                    int64_t slice = t.L / csize, begin = crank * slice;
                    if (slice * csize != t.L || slice % (16 / gsz) != 0) {
                        const int64_t q = t.L / 16;
                        begin = q * crank / csize * 16;
                        slice = (crank + 1 == csize ? t.L : q * (crank + 1) / csize * 16) - begin;
                    }
                    int head = 0, tail = 0;
                    if (EDGES) {
                        // the aligned middle travels through the stages: 8 elements are 16 bytes of
                        // bf16 gradients and 32 bytes of float32
                        head = static_cast<int>((8 - ((local * t.L) & 7)) & 7);
                        begin = head;
                        slice = (t.L - head) & ~int64_t(7);
                        tail = static_cast<int>(t.L - head - slice);
                    }
                    const int64_t e0 = local * t.L + begin;
                    const int sum_cap = P.stage_bytes / gsz;
                    for (int64_t off = 0; off < slice && ok; off += sum_cap) {
                        const int c = static_cast<int>(slice - off < sum_cap ? slice - off : sum_cap);
                        const bool last = off + c == slice;
                        if (!(ok = acquire())) break;
                        if (EDGES) {
                            EdgeMeta &em = ctl->edge[stage];
                            em.g = gbase + (e0 + off) * gsz;
                            em.head = off == 0 ? head : 0;
                            em.tail = last ? tail : 0;
                        }
                        StageMeta &mt = ctl->meta[stage];
                        mt.m = nullptr; mt.p = nullptr; mt.v = P.v + t.v_offset + local; mt.pb = nullptr; mt.group = item_group;
                        mt.inv_L = inv_L;
                        mt.n = c; mt.L = 0; mt.kind = STAGE_SUM;
                        mt.flags = base_flags | (last ? SF_LAST : 0) | (crank == 0 ? SF_WRITE_V : 0);
                        const uint32_t vbytes = last ? stage_v(mt, t.v_offset + local, 1) : 0u;
                        unsigned char *st = stages + static_cast<size_t>(stage) * P.stage_bytes;
                        mbar_arrive_expect_tx(&ctl->full[stage], static_cast<uint32_t>(c) * gsz + vbytes);
                        if (vbytes)
                            bulk_load(v_areas + stage * kVAreaFloats, P.v + ((t.v_offset + local) & ~int64_t(3)), vbytes,
                                      &ctl->full[stage]);
                        // a head's gradients are fetched twice: keep the first copy in L2 ...
                        if (CLUSTER) bulk_load_hint(st, gbase + (e0 + off) * gsz, c * gsz, &ctl->full[stage], keep_in_l2);
                        else bulk_load(st, gbase + (e0 + off) * gsz, c * gsz, &ctl->full[stage]);
                        advance();
                    }
                    for (int64_t off = 0; off < slice && ok; off += kStageElems) {
                        const int c = static_cast<int>(slice - off < kStageElems ? slice - off : kStageElems);
                        if (!(ok = acquire())) break;
                        if (EDGES) {
                            EdgeMeta &em = ctl->edge[stage];
                            em.g = gbase + (e0 + off) * gsz;
                            em.head = off == 0 ? head : 0;
                            em.tail = off + c == slice ? tail : 0;
                        }
                        StageMeta &mt = ctl->meta[stage];
                        mt.m = t.m + e0 + off; mt.p = t.p + e0 + off; mt.v = nullptr;
                        mt.pb = t.p_bf16 ? t.p_bf16 + e0 + off : nullptr; mt.group = item_group;
                        mt.inv_L = 0.0;
                        mt.n = c; mt.L = 0; mt.kind = STAGE_APPLY; mt.flags = base_flags;
                        unsigned char *st = stages + static_cast<size_t>(stage) * P.stage_bytes;
                        mbar_arrive_expect_tx(&ctl->full[stage], static_cast<uint32_t>(c) * (gsz + 8));
                        // ... and let go of it at the second fetch (measured: head kernel 3.00 ms against 3.10 ms)
                        if (CLUSTER) bulk_load_hint(st, gbase + (e0 + off) * gsz, c * gsz, &ctl->full[stage], drop_from_l2);
                        else bulk_load(st, gbase + (e0 + off) * gsz, c * gsz, &ctl->full[stage]);
                        bulk_load(st + P.g_region_bytes, t.m + e0 + off, c * 4, &ctl->full[stage]);
                        bulk_load(st + P.g_region_bytes + kStageElems * 4, t.p + e0 + off, c * 4, &ctl->full[stage]);
                        advance();
                        if (CLUSTER && pub_pending) publish_finish();
                    }
                }
                if (++item_group == P.n_groups) item_group = 0;
                it += sg.slots - 1;             // the loop's increment then lands on the next item
            }
            // One index more than the cluster takes is always on its way (the first CTA runs two ahead
            // and the last take is the one that finds nothing left): wait for it, so that no store is
            // still travelling towards this CTA's shared memory when it retires.
            if (cdynamic && ok) (void)cluster_take();
            if (ok && acquire()) {
                ctl->meta[stage].kind = STAGE_DONE;
                mbar_arrive(&ctl->full[stage]);
            } else {
                // gave up: let copies that are still in flight land before the CTA retires
                const int64_t back = armed < P.n_stages ? armed : P.n_stages;
                int s = stage;
                uint32_t ph = phase;
                for (int64_t k = 0; k < back; ++k) {
                    if (--s < 0) { s = P.n_stages - 1; ph ^= 1u; }
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(&ctl->full[s], ph) && global_ns() - t0 < kDrainTimeoutNs) {}
                }
            }
        }
        if (CLUSTER) __syncwarp();       // the producer's warp reaches the cluster's exit barrier together
    } else {
        // ------------------------------ consumers ------------------------------
        // The consumer warps form P.n_groups groups.  Every group follows the ring in order and
        // reads every stage's descriptor, but only the owning group (descriptor's `group`; work
        // items alternate between the groups) processes the stage, so the reduce / barrier /
        // apply latencies of one item overlap with the other group's work on the next item.
        // All warps arrive on a stage's `empty` barrier: owners after processing, the others
        // at once (which also keeps the producer from rewriting a descriptor somebody still reads).
        const int ctid = tid - 32;
        const int nthr = P.consumer_threads;
        const int group = ctid / nthr;
        const int gtid = ctid - group * nthr;
        const int lane = gtid & 31, warp = gtid >> 5;
        if (group < P.n_groups) {
            // the gradient scale s enters as (1-beta1)*s in the first moment and as s*s on the
            // sums of squares, so the per-element work is the same with or without it
            const float gscale = effective_gscale(P.sc.gscale, P.sc.gscale_dev);
            const float beta1 = P.sc.beta1, omb1 = P.sc.omb1 * gscale;
            const double gscale_sq = static_cast<double>(gscale) * static_cast<double>(gscale);
            int stage = 0;
            uint32_t phase = 0;
            GroupSync gsync{0u, 0};
            Acc a0 = stat_acc_init<ST>(), a1 = a0, a2 = a0, a3 = a0;   // running statistic of a long block
            float long_step = 0.f;
            uint32_t long_seen = 0;      // long blocks seen by this CTA, whoever owns them (exchange slot/parity)
            for (;;) {
                if (!wait_phase<false>(&ctl->full[stage], phase, ctl, P.error_word, 2, P.wait_limit_ns)) break;
                const StageMeta mt = ctl->meta[stage];
                if (mt.kind == STAGE_DONE) break;
                const bool last_sum = mt.kind == STAGE_SUM && (mt.flags & SF_LAST);
                if (mt.group != group) {
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&ctl->empty[stage]);
                    if (last_sum) ++long_seen;
                    if (++stage == P.n_stages) { stage = 0; phase ^= 1u; }
                    continue;
                }
                const unsigned char *gs = stages + static_cast<size_t>(stage) * P.stage_bytes;
                const float *ms = reinterpret_cast<const float *>(gs + P.g_region_bytes);
                const float *ps = ms + kStageElems;
                const bool bf16 = GDM == GDM_MIXED ? (mt.flags & SF_BF16) != 0 : GDM == GDM_BF16;
                // where the old v of the stage's blocks is read from
                const float *v_src = (mt.flags & SF_V_STAGED) ? v_areas + stage * kVAreaFloats + mt.v_shift : mt.v;
                const float lr_wd = (mt.flags & SF_WD) ? P.sc.lr_wd : 0.f;
                bool alive = true;

                if (mt.kind == STAGE_PACKED) {
                    const int L = mt.L, nb = mt.n / mt.L;
                    if (L <= kWarpBlockMaxL) {
                        for (int b = warp; b < nb; b += n_gwarps) {
                            const int e = b * L;
                            Acc s0 = stat_acc_init<ST>(), s1 = s0, s2 = s0, s3 = s0;
                            if (bf16) sum_span<AM_BF16, ST>(gs, e, L, lane, 32, s0, s1, s2, s3);
                            else sum_span<AM_F32, ST>(gs, e, L, lane, 32, s0, s1, s2, s3);
                            double wtot;
                            if (ST == ST_SUM) {
                                // at most 8 terms per accumulator and a 5-level tree: float is enough
                                float tot = (static_cast<float>(s0) + static_cast<float>(s1)) + (static_cast<float>(s2) + static_cast<float>(s3));
#pragma unroll
                                for (int o = 16; o > 0; o >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, o);
                                wtot = static_cast<double>(tot);
                            } else {
                                wtot = stat_op_finish<ST>(warp_combine<ST>(fold4<ST>(s0, s1, s2, s3)));
                            }
                            float v_old = lane == 0 ? v_src[b] : 0.f;
                            v_old = __shfl_sync(0xffffffffu, v_old, 0);
                            float vn;
                            const float step = stream_block_step(wtot * gscale_sq, mt.inv_L, v_old, P.sc, &vn);
                            if (lane == 0) mt.v[b] = vn;
                            if (bf16) apply_span<AM_BF16, COPY, CLUSTER>(gs, ms, ps, mt.m, mt.p, mt.pb, e, L, lane, 32, beta1, omb1, lr_wd, step);
                            else apply_span<AM_F32, COPY, CLUSTER>(gs, ms, ps, mt.m, mt.p, mt.pb, e, L, lane, 32, beta1, omb1, lr_wd, step);
                        }
                    } else {
                        for (int b = 0; b < nb && alive; ++b) {
                            const int e = b * L;
                            Acc s0 = stat_acc_init<ST>(), s1 = s0, s2 = s0, s3 = s0;
                            if (bf16) sum_span<AM_BF16, ST>(gs, e, L, gtid, nthr, s0, s1, s2, s3);
                            else sum_span<AM_F32, ST>(gs, e, L, gtid, nthr, s0, s1, s2, s3);
                            double tot;
                            float v_old;
                            alive = group_reduce<ST>(ctl, gsync, P.error_word, P.wait_limit_ns, group, gtid, n_gwarps, fold4<ST>(s0, s1, s2, s3),
                                                     v_src + b, &tot, &v_old);
                            if (!alive) break;
                            float vn;
                            const float step = stream_block_step(stat_op_finish<ST>(tot) * gscale_sq, mt.inv_L, v_old, P.sc, &vn);
                            if (gtid == 0) mt.v[b] = vn;
                            if (bf16) apply_span<AM_BF16, COPY, CLUSTER>(gs, ms, ps, mt.m, mt.p, mt.pb, e, L, gtid, nthr, beta1, omb1, lr_wd, step);
                            else apply_span<AM_F32, COPY, CLUSTER>(gs, ms, ps, mt.m, mt.p, mt.pb, e, L, gtid, nthr, beta1, omb1, lr_wd, step);
                        }
                    }
                    if (!alive) break;
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&ctl->empty[stage]);
                } else if (mt.kind == STAGE_SUM) {
                    // (unaligned blocks: the block's elements either side of the staged chunks come from
                    // global memory; their loads are issued first, so that the pass over the stage covers
                    // their latency)
                    bool edge_mine = false;
                    float edge_g = 0.f;
                    if (EDGES) {
                        const EdgeMeta em = ctl->edge[stage];
                        const bool is_head = gtid < em.head, is_tail = gtid >= 8 && gtid < 8 + em.tail;
                        edge_mine = is_head || is_tail;
                        if (edge_mine) {
                            const int64_t k = is_head ? gtid - em.head : mt.n + (gtid - 8);
                            edge_g = bf16 ? load_g1<AM_BF16>(em.g, k, 1.f) : load_g1<AM_F32>(em.g, k, 1.f);
                        }
                    }
                    if (bf16) sum_span<AM_BF16, ST>(gs, 0, mt.n, gtid, nthr, a0, a1, a2, a3);
                    else sum_span<AM_F32, ST>(gs, 0, mt.n, gtid, nthr, a0, a1, a2, a3);
                    if (EDGES && edge_mine) stat_acc_add<ST>(a0, edge_g);
                    if (!last_sum) {
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&ctl->empty[stage]);
                    } else {
                        double tot;
                        float v_old;
                        if (!group_reduce<ST>(ctl, gsync, P.error_word, P.wait_limit_ns, group, gtid, n_gwarps, fold4<ST>(a0, a1, a2, a3), v_src, &tot, &v_old))
                            break;
                        __syncwarp();                       // the stage (and its v area) has been read
                        if (lane == 0) mbar_arrive(&ctl->empty[stage]);
                        a0 = a1 = a2 = a3 = stat_acc_init<ST>();
                        if (CLUSTER) {
                            // Exchange the CTAs' sums through distributed shared memory.  Every CTA of
                            // the cluster walks the same blocks in the same order, so block number
                            // long_seen names the same block (and the same owning group) everywhere.
                            // Four slots: a group reuses a slot only two of its own blocks later, after
                            // a group barrier of every peer has ordered the earlier reads before it.
                            const uint32_t slot = long_seen & (kExchangeSlots - 1);
                            if (gtid == 0) {
                                mbar_arrive_expect_tx(&ctl->xbar[slot], 8u * csize);    // this CTA's turn of the slot: one sum per CTA
                                const uint32_t part = smem_addr(&ctl->xpart[slot][crank]);
                                const uint32_t bar = smem_addr(&ctl->xbar[slot]);
                                for (uint32_t r = 0; r < csize; ++r)
                                    st_async_cluster_b64(map_to_rank(part, r), static_cast<unsigned long long>(__double_as_longlong(tot)),
                                                         map_to_rank(bar, r));
                            }
                            if (!wait_phase<true>(&ctl->xbar[slot], (long_seen / kExchangeSlots) & 1u, ctl, P.error_word, 4, P.wait_limit_ns)) break;
                            tot = ctl->xpart[slot][0];
                            for (uint32_t r = 1; r < csize; ++r) tot = stat_op_combine<ST>(tot, ctl->xpart[slot][r]);
                        }
                        ++long_seen;
                        float vn;
                        long_step = stream_block_step(stat_op_finish<ST>(tot) * gscale_sq, mt.inv_L, v_old, P.sc, &vn);
                        if (gtid == 0 && (mt.flags & SF_WRITE_V)) *mt.v = vn;
                    }
                } else {   // STAGE_APPLY
                    bool edge_mine = false;
                    int64_t edge_k = 0;
                    float edge_g = 0.f, edge_m = 0.f, edge_p = 0.f;
                    if (EDGES) {        // edge elements: loads first, update and stores after the pass over the stage
                        const EdgeMeta em = ctl->edge[stage];
                        const bool is_head = gtid < em.head, is_tail = gtid >= 8 && gtid < 8 + em.tail;
                        edge_mine = is_head || is_tail;
                        if (edge_mine) {
                            edge_k = is_head ? gtid - em.head : mt.n + (gtid - 8);
                            edge_g = bf16 ? load_g1<AM_BF16>(em.g, edge_k, 1.f) : load_g1<AM_F32>(em.g, edge_k, 1.f);
                            edge_m = mt.m[edge_k];
                            edge_p = mt.p[edge_k];
                        }
                    }
                    if (bf16) apply_span<AM_BF16, COPY, CLUSTER>(gs, ms, ps, mt.m, mt.p, mt.pb, 0, mt.n, gtid, nthr, beta1, omb1, lr_wd, long_step);
                    else apply_span<AM_F32, COPY, CLUSTER>(gs, ms, ps, mt.m, mt.p, mt.pb, 0, mt.n, gtid, nthr, beta1, omb1, lr_wd, long_step);
                    if (EDGES && edge_mine) {
                        update_one(edge_g, edge_m, edge_p, beta1, omb1, lr_wd, long_step);
                        mt.m[edge_k] = edge_m;
                        mt.p[edge_k] = edge_p;
                        if (COPY && mt.pb) store_bf16(mt.pb + edge_k, edge_p);
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&ctl->empty[stage]);
                }
                if (++stage == P.n_stages) { stage = 0; phase ^= 1u; }
            }
        }
    }
    // common exit: nobody leaves a cluster while a peer may still write into it
    if (CLUSTER) {
        __syncwarp();
        cluster_sync_all();
    }
}

// ------------------------------- host-side planning -------------------------------
// What planning needs to know about the device (queried when a handle is created).
struct DeviceCaps {
    int sm_count = 0;
    size_t smem_optin = 0;                  // most dynamic shared memory a CTA may ask for
    int64_t l2_bytes = 0;
    int resident[kMaxCluster + 1] = {};     // resident[c]: clusters of c CTAs of the streaming kernel the device
                                            // keeps resident at once (0: such clusters cannot run)
};

struct StreamPlanInput {
    DeviceCaps caps;
    int ctas = 0, cluster_size = 0, threads = 0, groups = 0, chunk = 0, cluster_chunk = 0;
    struct Item { int tensor; am_table_row row; };
    std::vector<Item> stream_tensors, cluster_tensors, edge_tensors;
};

// Which path a tensor with block length L (> 64) takes; *edges: its blocks start off the 16-byte
// grid and run in the streaming kernel's launch for such blocks.
inline int stream_classify(int64_t L, int32_t gdtype, bool cluster_ok, bool *edges) {
    const int64_t gsz = gdtype == AM_BF16 ? 2 : 4;
    const int64_t vec = 16 / gsz;                     // elements per 16 bytes of g
    *edges = false;
    if (L % vec != 0) {                               // block starts are not 16-byte aligned
        if (L > kStageElems && L * gsz <= kStreamMaxBlockBytes) { *edges = true; return PATH_STREAM; }
        return PATH_TWOPASS;                          // (up to kStageElems elements the tile kernel takes them)
    }
    if (L * gsz <= kStreamMaxBlockBytes) return PATH_STREAM;
    if (cluster_ok && L * gsz <= kClusterMaxBlockBytes && L % (kMaxCluster * vec) == 0) return PATH_CLUSTER;
    return PATH_TWOPASS;
}

inline void stream_add_tensor(StreamPlanInput &in, int index, const am_table_row &r, int path, bool edges) {
    (path == PATH_CLUSTER ? in.cluster_tensors : edges ? in.edge_tensors : in.stream_tensors).push_back({index, r});
}

typedef void (*StreamKernelFn)(const StreamParams);

// One instantiation per use keeps the mean's consumer loop small; the ablation
// statistics are compiled with the bf16-copy path in (taken only where a tensor has a copy).
template <bool CLUSTER, int ST>
inline StreamKernelFn stream_kernel_for(int gdm, bool copy) {
    if (ST != ST_SUM) copy = true;
    switch (gdm * 2 + (copy ? 1 : 0)) {
    case 0: return stream_kernel<CLUSTER, GDM_F32, ST != ST_SUM, ST, false>;
    case 1: return stream_kernel<CLUSTER, GDM_F32, true, ST, false>;
    case 2: return stream_kernel<CLUSTER, GDM_BF16, ST != ST_SUM, ST, false>;
    case 3: return stream_kernel<CLUSTER, GDM_BF16, true, ST, false>;
    case 4: return stream_kernel<CLUSTER, GDM_MIXED, ST != ST_SUM, ST, false>;
    default: return stream_kernel<CLUSTER, GDM_MIXED, true, ST, false>;
    }
}
template <bool CLUSTER>
inline StreamKernelFn stream_kernel_for(int gdm, bool copy, int st) {
    switch (st) {
    case ST_MAX: return stream_kernel_for<CLUSTER, ST_MAX>(gdm, copy);
    case ST_MIN: return stream_kernel_for<CLUSTER, ST_MIN>(gdm, copy);
    case ST_SUM4: return stream_kernel_for<CLUSTER, ST_SUM4>(gdm, copy);
    default: return stream_kernel_for<CLUSTER, ST_SUM>(gdm, copy);
    }
}
inline StreamKernelFn stream_kernel_for(bool cluster, int gdm, bool copy, int st) {
    return cluster ? stream_kernel_for<true>(gdm, copy, st) : stream_kernel_for<false>(gdm, copy, st);
}
// Unaligned long blocks: one instantiation per statistic, any gradient dtype, bf16 copies where asked for.
inline StreamKernelFn stream_edge_kernel_for(int st) {
    switch (st) {
    case ST_MAX: return stream_kernel<false, GDM_MIXED, true, ST_MAX, true>;
    case ST_MIN: return stream_kernel<false, GDM_MIXED, true, ST_MIN, true>;
    case ST_SUM4: return stream_kernel<false, GDM_MIXED, true, ST_SUM4, true>;
    default: return stream_kernel<false, GDM_MIXED, true, ST_SUM, true>;
    }
}

struct StreamLaunch {
    std::vector<StreamSeg> segs;     // with sentinel
    std::vector<int64_t> bounds;
    int grid = 0, cluster = 1, n_stages = 0, stage_bytes = 0, g_region_bytes = 0, threads = 0, groups = 1, chunk = 0;
    int gdm = GDM_MIXED;
    bool edges = false;              // the launch of unaligned long blocks
    unsigned long long *d_counter = nullptr;      // two counters, 64 bytes apart, used by alternate launches
    mutable int counter_parity = 0;
    const StreamSeg *d_segs = nullptr;
    const int64_t *d_bounds = nullptr;
    bool active() const { return grid > 0; }
    size_t smem_bytes() const { return kCtrlBytes + static_cast<size_t>(n_stages) * (stage_bytes + kVAreaFloats * 4); }
};

struct StreamPlan {
    StreamLaunch main, clus, edge;

    size_t table_bytes() const {
        return (main.segs.size() + clus.segs.size() + edge.segs.size()) * sizeof(StreamSeg) + 384 +
               (main.bounds.size() + clus.bounds.size() + edge.bounds.size()) * sizeof(int64_t) + 384 + 768;
    }
    int launches() const { return (main.active() ? 1 : 0) + (clus.active() ? 1 : 0) + (edge.active() ? 1 : 0); }

    cudaError_t upload(char *base) {
        size_t off = 0;
        for (StreamLaunch *L : {&main, &clus, &edge}) {
            if (!L->active()) continue;
            cudaError_t e = cudaMemcpy(base + off, L->segs.data(), L->segs.size() * sizeof(StreamSeg), cudaMemcpyHostToDevice);
            if (e != cudaSuccess) return e;
            L->d_segs = reinterpret_cast<const StreamSeg *>(base + off);
            off += (L->segs.size() * sizeof(StreamSeg) + 127) / 128 * 128;
            e = cudaMemcpy(base + off, L->bounds.data(), L->bounds.size() * sizeof(int64_t), cudaMemcpyHostToDevice);
            if (e != cudaSuccess) return e;
            L->d_bounds = reinterpret_cast<const int64_t *>(base + off);
            off += (L->bounds.size() * sizeof(int64_t) + 127) / 128 * 128;
            L->d_counter = reinterpret_cast<unsigned long long *>(base + off);
            L->counter_parity = 0;
            e = cudaMemset(base + off, 0, 128);
            if (e != cudaSuccess) return e;
            off += 128;
        }
        return cudaSuccess;
    }

    int64_t v_len = 0;
    bool bf16_copies = false;      // set per step: some tensor has a bf16 copy to write
    unsigned long long wait_limit_ns = kWaitTimeoutNs;
    int stall_after = 0;

    cudaError_t launch_one(const StreamLaunch &L, bool cluster, const DevTensor *tensors, float *v,
                           const StepScalars &sc, int *error_word, cudaStream_t stream) const {
        StreamParams P;
        P.tensors = tensors; P.segs = L.d_segs; P.bounds = L.d_bounds; P.v = v; P.error_word = error_word;
        P.sc = sc; P.n_segs = static_cast<int>(L.segs.size()) - 1; P.n_stages = L.n_stages;
        P.stage_bytes = L.stage_bytes; P.g_region_bytes = L.g_region_bytes; P.consumer_threads = L.threads;
        P.n_groups = L.groups;
        P.v_len = v_len;
        P.wait_limit_ns = wait_limit_ns; P.stall_after = stall_after; P.pad = 0;
        P.chunk = L.chunk; P.total_items = L.bounds.empty() ? 0 : L.bounds.back();
        P.counter = L.d_counter + 8 * L.counter_parity;
        P.counter_next = L.d_counter + 8 * (L.counter_parity ^ 1);
        L.counter_parity ^= 1;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(L.grid);
        cfg.blockDim = dim3(32 + L.threads * L.groups);
        cfg.dynamicSmemBytes = L.smem_bytes();
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        if (cluster) {
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = L.cluster;
            attr[0].val.clusterDim.y = 1;
            attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
        }
        const int st = stat_op_of(sc.statistic);
        return cudaLaunchKernelEx(&cfg, L.edges ? stream_edge_kernel_for(st) : stream_kernel_for(cluster, L.gdm, bf16_copies, st), P);
    }

    cudaError_t launch_main(const DevTensor *tensors, float *v, const StepScalars &sc, int *error_word,
                            cudaStream_t stream) const {
        return main.active() ? launch_one(main, false, tensors, v, sc, error_word, stream) : cudaSuccess;
    }
    cudaError_t launch_cluster(const DevTensor *tensors, float *v, const StepScalars &sc, int *error_word,
                               cudaStream_t stream) const {
        return clus.active() ? launch_one(clus, true, tensors, v, sc, error_word, stream) : cudaSuccess;
    }
    cudaError_t launch_edge(const DevTensor *tensors, float *v, const StepScalars &sc, int *error_word,
                            cudaStream_t stream) const {
        return edge.active() ? launch_one(edge, false, tensors, v, sc, error_word, stream) : cudaSuccess;
    }
};

// Shared-memory layout of a launch: a stage holds kStageElems gradients (2 or 4 bytes each), first
// moments and parameters; as many stages as the CTA's shared memory allows.
inline void stream_stage_layout(bool any_f32, size_t smem_optin, int *g_region_bytes, int *stage_bytes, int *n_stages) {
    *g_region_bytes = kStageElems * (any_f32 ? 4 : 2);
    *stage_bytes = *g_region_bytes + kStageElems * 8;
    const size_t per_stage = static_cast<size_t>(*stage_bytes) + kVAreaFloats * 4;
    *n_stages = smem_optin > kCtrlBytes ? std::min<int>(kMaxStages, static_cast<int>((smem_optin - kCtrlBytes) / per_stage)) : 0;
}

// Build segment tables and balanced item ranges for one launch.
inline void stream_build_launch(const std::vector<StreamPlanInput::Item> &tensors, bool cluster, int workers,
                                size_t smem_optin, StreamLaunch *out) {
    out->segs.clear();
    out->bounds.clear();
    out->grid = 0;
    if (tensors.empty() || workers <= 0) return;
    bool any_f32 = false, any_bf16 = false;
    for (const auto &it : tensors) {
        any_f32 |= it.row.grad_dtype == AM_F32;
        any_bf16 |= it.row.grad_dtype == AM_BF16;
    }
    out->gdm = any_f32 && any_bf16 ? GDM_MIXED : (any_bf16 ? GDM_BF16 : GDM_F32);
    stream_stage_layout(any_f32, smem_optin, &out->g_region_bytes, &out->stage_bytes, &out->n_stages);

    std::vector<double> item_cost;      // per segment
    int64_t slots = 0, n_items = 0;
    for (const auto &it : tensors) {
        const am_table_row &r = it.row;
        const int gsz = r.grad_dtype == AM_BF16 ? 2 : 4;
        StreamSeg s;
        s.item_begin = slots;
        s.tensor = it.tensor;
        s.pad = 0;
        int64_t seg_items;
        if (!cluster && r.block_len <= kStageElems) {
            s.bpi = static_cast<int32_t>(kStageElems / r.block_len);
            s.slots = 1;
            seg_items = (r.n_blocks + s.bpi - 1) / s.bpi;
            item_cost.push_back(static_cast<double>(s.bpi) * r.block_len * (gsz + 16));
        } else {
            s.bpi = 0;
            const int64_t sum_cap = out->stage_bytes / gsz;
            s.slots = cluster ? 1 : static_cast<int32_t>((r.block_len + sum_cap - 1) / sum_cap +
                                                         (r.block_len + kStageElems - 1) / kStageElems);
            seg_items = r.n_blocks;
            item_cost.push_back(static_cast<double>(r.block_len) * (2 * gsz + 16));
        }
        slots += seg_items * s.slots;
        n_items += seg_items;
        out->segs.push_back(s);
    }
    StreamSeg sentinel;
    sentinel.item_begin = slots;
    sentinel.tensor = -1;
    sentinel.bpi = 0;
    sentinel.slots = 1;
    sentinel.pad = 0;
    out->segs.push_back(sentinel);

    // contiguous ranges of (nearly) equal cost, cut at item starts
    double total = 0.0;
    auto seg_items_of = [&](size_t k) {
        return (out->segs[k + 1].item_begin - out->segs[k].item_begin) / out->segs[k].slots;
    };
    for (size_t k = 0; k + 1 < out->segs.size(); ++k) total += item_cost[k] * static_cast<double>(seg_items_of(k));
    workers = static_cast<int>(std::min<int64_t>(workers, n_items));
    out->bounds.assign(workers + 1, 0);
    out->bounds[workers] = slots;
    size_t k = 0;
    double before = 0.0;                // cost of the segments before k
    for (int w = 1; w < workers; ++w) {
        const double target = total * w / workers;
        for (;;) {
            const double seg_cost = item_cost[k] * static_cast<double>(seg_items_of(k));
            if (before + seg_cost >= target || k + 2 >= out->segs.size()) break;
            before += seg_cost;
            ++k;
        }
        int64_t item = static_cast<int64_t>((target - before) / item_cost[k] + 0.5);
        item = std::min(item, seg_items_of(k));
        int64_t idx = out->segs[k].item_begin + item * out->segs[k].slots;
        idx = std::max(idx, out->bounds[w - 1]);
        idx = std::min(idx, slots);
        out->bounds[w] = idx;
    }
    out->grid = workers;
}

// How many clusters of every size the device keeps resident at once, for CTAs of
// `block_threads` threads with the larger of the two stage layouts.
inline void stream_probe_clusters(DeviceCaps *caps, int block_threads) {
    int g_region, stage_bytes, n_stages;
    stream_stage_layout(true, caps->smem_optin, &g_region, &stage_bytes, &n_stages);
    const size_t smem = kCtrlBytes + static_cast<size_t>(n_stages) * (stage_bytes + kVAreaFloats * 4);
    for (int cs = 1; cs <= kMaxCluster; ++cs) {
        caps->resident[cs] = 0;
        if (n_stages < 2) continue;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(std::max(caps->sm_count / cs, 1) * cs);
        cfg.blockDim = dim3(block_threads);
        cfg.dynamicSmemBytes = smem;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = cs;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, stream_kernel<true, GDM_MIXED, true, ST_SUM, false>, &cfg) == cudaSuccess && n > 0)
            caps->resident[cs] = n;
        else
            (void)cudaGetLastError();
    }
}

// Cluster size for head-sized blocks whose gradients take `block_bytes`.
//
// A cluster reads a block's gradients twice (to reduce them, then to apply the
// update), and the second read should find them in L2.  Every resident cluster
// has one block between its two reads, so resident[c] * block_bytes is what L2
// must keep besides the m and p streaming through it.  Smaller clusters mean
// more clusters, which use more SMs but keep more in L2: the choice is the
// smallest size whose in-flight gradients stay within kL2ShareForHeads of L2,
// or the largest size that can run when none does.  A size that keeps no more
// clusters resident than a larger one is passed over (it only idles SMs).
//
// kL2ShareForHeads is a measured boundary, not a derived one (B200, 126 MB of
// L2 in two halves, resident = 148/74/45/33/26/22/15/15 for sizes 1..8).  With
// the exchange done by asynchronous stores a larger cluster costs nothing extra,
// and fewer clusters that hold less in L2 beat many: on 1 MB blocks 22 clusters
// of 6 and 15 of 8 run at 1.00-1.02 of the copy bandwidth against 0.98 for 33 of
// 4 and 0.93 for 74 of 2 (in long runs under the power cap 6 is ahead of 8 by
// 1 %, in short ones 8 by as much); 2 MB blocks reach 1.02 with 15 of 8 against
// 0.98 with 22 of 6; blocks of 0.3 to 0.5 MB run at 1.02-1.05 with 3 to 6 CTAs.
constexpr double kL2ShareForHeads = 0.18;

inline int choose_cluster_size(const int *resident, int64_t l2_bytes, int64_t block_bytes) {
    int largest = 0;
    for (int c = 1; c <= kMaxCluster; ++c)
        if (resident[c] > 0) largest = c;
    if (largest == 0) return 0;
    const double room = kL2ShareForHeads * static_cast<double>(l2_bytes);
    for (int c = 1; c < largest; ++c) {
        if (resident[c] <= 0) continue;
        bool passed_over = false;
        for (int d = c + 1; d <= largest; ++d) passed_over |= resident[d] >= resident[c];
        if (passed_over) continue;
        if (static_cast<double>(resident[c]) * static_cast<double>(block_bytes) <= room) return c;
    }
    return largest;
}

// Consumer groups and threads per group of a launch (0 = defaults: two groups of 256).
inline void stream_consumer_shape(int threads_opt, int groups_opt, int *threads, int *groups) {
    *groups = groups_opt > 0 ? std::min(groups_opt, kMaxGroups) : kMaxGroups;
    *threads = threads_opt > 0 ? threads_opt : 256;
    while (*threads * *groups > kMaxConsumerWarps * 32) *threads -= 32;
}

// Number of work items of a launch whose segment table is still in slots.
inline int64_t stream_count_items(const StreamLaunch &L) {
    int64_t n = 0;
    for (size_t k = 0; k + 1 < L.segs.size(); ++k) n += (L.segs[k + 1].item_begin - L.segs[k].item_begin) / L.segs[k].slots;
    return n;
}

// Renumber a launch's items 0, 1, 2, ... (one slot each): the addressing of launches that take their
// work from the shared counter.
inline void stream_use_item_ordinals(StreamLaunch *L) {
    if (L->segs.empty()) return;
    std::vector<int64_t> count(L->segs.size() - 1);
    for (size_t k = 0; k + 1 < L->segs.size(); ++k)
        count[k] = (L->segs[k + 1].item_begin - L->segs[k].item_begin) / L->segs[k].slots;
    int64_t next = 0;
    for (size_t k = 0; k + 1 < L->segs.size(); ++k) {
        L->segs[k].item_begin = next;
        L->segs[k].slots = 1;
        next += count[k];
    }
    L->segs.back().item_begin = next;
    // (the per-CTA ranges are not used by such a launch; their last entry is its number of items)
    for (int64_t &b : L->bounds) b = std::min(b, next);
    L->bounds.back() = next;
}

inline void stream_finish_plan(const StreamPlanInput &in, StreamPlan *plan) {
    int threads, groups;
    stream_consumer_shape(in.threads, in.groups, &threads, &groups);
    const int ctas = in.ctas > 0 ? in.ctas : in.caps.sm_count;
    for (StreamLaunch *L : {&plan->main, &plan->edge}) {
        stream_build_launch(L == &plan->main ? in.stream_tensors : in.edge_tensors, false, ctas, in.caps.smem_optin, L);
        L->edges = L == &plan->edge;
        L->threads = threads;
        L->groups = groups;
        L->cluster = 1;
        // work distribution: ranges of `chunk` items from a shared counter unless static ranges were asked for
        if (in.chunk == kStaticRanges) L->chunk = 0;
        else if (in.chunk > 0) L->chunk = in.chunk;
        else {
            // One item per grab keeps the CTAs within a few stages of one another, so that they work on
            // one neighbourhood of every array and share DRAM pages.  Measured on Llama-2-7B rows, per
            // grab: 64 stages 15.17 ms, 16: 15.02, 8: 14.93, 4: 14.75, 2: 14.73, one item: 14.62; the same
            // 3-5 % on flat tensors of 128- to 8192-element blocks and on long rows.  (A workload of a
            // couple of items per CTA gains nothing from the counter.)
            L->chunk = stream_count_items(*L) <= 2 * static_cast<int64_t>(ctas) ? 0 : 1;
        }
        // The shared counter hands out ITEMS (a stage of packed blocks, or one long block with all its
        // stages): slots, which weigh an item by its stages, are for cutting fixed ranges of equal cost.
        // (Grabs counted in slots leave some grabs without an item's start when items have several:
        // a trip to the counter for nothing.  Rows of 4104 elements, three slots each: 0.75 of measured
        // with grabs of two slots, 0.95 with grabs of one item.)
        if (L->chunk > 0) stream_use_item_ordinals(L);
    }
    plan->clus = StreamLaunch();
    if (in.cluster_tensors.empty()) return;
    // Launch shape for head-sized blocks: the cluster size follows from the largest block, the L2
    // size and how many clusters of each size fit the device (choose_cluster_size), unless the
    // caller fixed it (then the largest size up to the caller's that can run).  Clusters take one
    // block at a time from the shared counter (fixed ranges, which keep every cluster in a region
    // of its own, ran 7 % slower on Llama-2-7B's heads).
    int64_t max_block_bytes = 0;
    for (const auto &it : in.cluster_tensors)
        max_block_bytes = std::max(max_block_bytes, it.row.block_len * (it.row.grad_dtype == AM_BF16 ? 2 : 4));
    int cluster_size = 0;
    if (in.cluster_size > 0) {
        for (int c = std::min(in.cluster_size, kMaxCluster); c >= 1 && cluster_size == 0; --c)
            if (in.caps.resident[c] > 0) cluster_size = c;
    } else {
        cluster_size = choose_cluster_size(in.caps.resident, in.caps.l2_bytes, max_block_bytes);
    }
    if (cluster_size == 0) return;
    int chunk = in.cluster_chunk;
    if (chunk == 0) chunk = 1;
    stream_build_launch(in.cluster_tensors, true, in.caps.resident[cluster_size], in.caps.smem_optin, &plan->clus);
    plan->clus.grid *= cluster_size;          // bounds are per cluster
    plan->clus.cluster = cluster_size;
    plan->clus.threads = threads;
    plan->clus.groups = in.groups > 0 ? groups : 1;     // measured: a second group does not help the head kernel
    plan->clus.chunk = chunk == kStaticRanges ? 0 : chunk;
}

inline cudaError_t stream_configure_kernels(size_t smem_optin) {
    for (int cluster = 0; cluster < 2; ++cluster)
        for (int gdm = 0; gdm < 3; ++gdm)
            for (int copy = 0; copy < 2; ++copy)
                for (int st = 0; st < 4; ++st) {
                    const cudaError_t e = cudaFuncSetAttribute(stream_kernel_for(cluster != 0, gdm, copy != 0, st),
                                                               cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                               static_cast<int>(smem_optin));
                    if (e != cudaSuccess) return e;
                }
    for (int st = 0; st < 4; ++st) {
        const cudaError_t e = cudaFuncSetAttribute(stream_edge_kernel_for(st), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                   static_cast<int>(smem_optin));
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace am

#endif  // ADAMMINI_KERNELS_STREAM_CUH_
