// A copy through a ring of shared-memory stages with no arithmetic in between:
// bulk asynchronous loads global -> shared (the streaming kernel's loads) and
// bulk asynchronous stores shared -> global, one persistent CTA per SM, items
// handed out one at a time from a shared counter.  It measures what this
// device's memory system gives a kernel that reads `load_bytes` and writes
// `store_bytes` per item: the ceiling for the update's own mix (10 bytes read,
// 8 written per parameter with bf16 gradients), which is lower than for reads
// or writes alone.  A measurement aid: no step of Algorithm 1 runs here.
#ifndef ADAMMINI_KERNELS_PROBE_CUH_
#define ADAMMINI_KERNELS_PROBE_CUH_

#include "kernels_stream.cuh"

namespace am {

constexpr int kProbeStageBytes = 40960;
constexpr int kProbeThreads = 64;        // thread 0 loads, thread 32 stores

__device__ __forceinline__ void bulk_store(void *dst_gmem, const void *src_smem, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst_gmem), "r"(smem_addr(src_smem)), "r"(bytes)
                 : "memory");
}

__global__ void __launch_bounds__(kProbeThreads, 1)
ring_copy_kernel(const unsigned char *src, unsigned char *dst, long long n_items, int load_bytes, int store_bytes, int n_stages,
                 unsigned long long *counter, int *error_word, unsigned long long limit_ns) {
    extern __shared__ __align__(128) unsigned char smem[];
    Control *ctl = reinterpret_cast<Control *>(smem);
    unsigned char *stages = smem + kCtrlBytes;
    if (threadIdx.x == 0) {
        for (int s = 0; s < n_stages; ++s) {
            mbar_init(&ctl->full[s], 1);
            mbar_init(&ctl->empty[s], 1);
        }
        ctl->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int stage = 0;
        uint32_t phase = 0;
        long long armed = 0;
        bool ok = true;
        for (;;) {
            const long long it = static_cast<long long>(atomicAdd(counter, 1ull));
            if (!(ok = wait_phase_one<false>(&ctl->empty[stage], phase ^ 1u, ctl, error_word, 1, limit_ns))) break;
            ctl->next_item[stage] = it < n_items ? it : -1;
            if (it >= n_items) {                 // tells the storing thread that nothing follows
                mbar_arrive(&ctl->full[stage]);
                break;
            }
            if (load_bytes > 0) {
                mbar_arrive_expect_tx(&ctl->full[stage], static_cast<uint32_t>(load_bytes));
                bulk_load(stages + static_cast<size_t>(stage) * kProbeStageBytes, src + it * load_bytes, load_bytes, &ctl->full[stage]);
            } else {
                mbar_arrive(&ctl->full[stage]);
            }
            ++armed;
            if (++stage == n_stages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) {      // gave up: let copies that are still in flight land before the CTA retires
            const long long back = armed < n_stages ? armed : n_stages;
            int s = stage;
            uint32_t ph = phase;
            for (long long k = 0; k < back; ++k) {
                if (--s < 0) { s = n_stages - 1; ph ^= 1u; }
                const unsigned long long t0 = global_ns();
                while (!mbar_try_wait(&ctl->full[s], ph) && global_ns() - t0 < kDrainTimeoutNs) {}
            }
        }
    } else if (threadIdx.x == 32) {
        int stage = 0;
        uint32_t phase = 0;
        for (;;) {
            if (!wait_phase_one<false>(&ctl->full[stage], phase, ctl, error_word, 2, limit_ns)) break;
            const long long it = ctl->next_item[stage];
            if (it < 0) break;
            if (store_bytes > 0) {
                bulk_store(dst + it * store_bytes, stages + static_cast<size_t>(stage) * kProbeStageBytes, store_bytes);
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");     // the stage has been read: it may be refilled
            }
            mbar_arrive(&ctl->empty[stage]);
            if (++stage == n_stages) { stage = 0; phase ^= 1u; }
        }
        asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");                  // the stores have landed
    }
}

}  // namespace am

#endif  // ADAMMINI_KERNELS_PROBE_CUH_
