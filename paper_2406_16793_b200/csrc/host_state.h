// The optimizer handle.
#ifndef ADAMMINI_HOST_STATE_H_
#define ADAMMINI_HOST_STATE_H_

#include <cuda_runtime.h>

#include <vector>

#include "adammini_internal.h"
#include "kernels_stream.cuh"

struct HostStepState;   // staging for adammini_step_host, created on first use

struct am_handle {
    int device = 0;
    int sm_count = 0;
    std::vector<am_table_row> rows;
    int64_t total_blocks = 0;
    int64_t total_elems = 0;
    am_hparams hp{};
    int64_t opt[11] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0};

    // launch plan
    bool planned = false;
    std::vector<int32_t> path;
    std::vector<am::DevTensor> host_tensors;
    void *arena = nullptr;
    size_t arena_bytes = 0;
    am::DevTensor *d_tensors = nullptr;
    am::Seg *d_small_segs = nullptr, *d_piece_segs = nullptr, *d_block_segs = nullptr;
    int n_small_segs = 0, n_piece_segs = 0, n_block_segs = 0;
    int64_t small_units = 0, piece_units = 0, block_units = 0;
    int64_t small_units_by_len[4] = {0, 0, 0, 0};   // units of the register kernel for block lengths 1, 2, 3 (index 0 unused)
    am::Seg *d_tile_segs = nullptr;      // short blocks handled a tile at a time
    int n_tile_segs = 0;
    int64_t tile_units = 0;
    int64_t tile_short_units = 0;        // the first so many tiles hold blocks of up to kSmallMaxL elements, the rest longer ones
    am::Seg *d_wide_segs = nullptr;      // two-pass tensors whose blocks have many partial sums
    int n_wide_segs = 0;
    int64_t wide_units = 0;
    am::Seg *d_part_segs = nullptr;      // pieces of the tensors that are parts of blocks (AM_PART)
    int32_t *d_part_tensors = nullptr;
    int n_parts = 0;
    int64_t part_units = 0;
    double *d_partials = nullptr;
    unsigned long long *d_probe_counter = nullptr;   // work counter of adammini_probe_ring_copy
    float *d_block_steps = nullptr;
    am::StreamPlan stream;
    am::DeviceCaps caps;                 // SMs, shared memory, L2, resident clusters per cluster size
    int launches = 0;
    int64_t elems_by_path[4] = {0, 0, 0, 0};
    int64_t algorithmic_bytes = 0;
    int64_t bytes_by_path[4] = {0, 0, 0, 0};
    std::vector<cudaEvent_t> prof_ev;    // AM_OPT_PROFILE: 5 events per recorded step, a ring of `opt` steps
    int64_t prof_steps = 0;              // steps recorded since profiling was switched on

    // pinned staging of the tensor table, double buffered
    am::DevTensor *pinned[2] = {nullptr, nullptr};
    cudaEvent_t ev[2] = {nullptr, nullptr};
    bool ev_pending[2] = {false, false};
    int next_pinned = 0;
    bool ptrs_valid = false;

    int *error_word = nullptr;   // pinned; kernels write a code here when a bounded wait gives up
    int last_cuda_error = 0;

    HostStepState *host_step = nullptr;
};

void host_step_release(am_handle *h);

#endif  // ADAMMINI_HOST_STATE_H_
