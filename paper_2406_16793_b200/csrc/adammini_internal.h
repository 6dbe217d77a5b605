// Internal declarations shared by the host code and the kernels.
#ifndef ADAMMINI_INTERNAL_H_
#define ADAMMINI_INTERNAL_H_

#include <cstdint>
#include <vector>

#include "adammini.h"

struct am_partition {
    std::vector<am_table_row> rows;
    int64_t total_blocks = 0;
};

namespace am {

// Which kernel family updates a tensor.
enum Path : int32_t {
    PATH_SMALL = 0,    // block_len <= 64, or <= 4096 with unaligned block starts: small_kernel / tile_kernel
    PATH_STREAM = 1,   // blocks that fit a shared-memory stage, and rows re-read from L2
    PATH_CLUSTER = 2,  // head-sized blocks: one thread-block cluster per block
    PATH_TWOPASS = 3   // everything else: partial sums, finalize, update (g read twice)
};

// Per-tensor record in device memory.  The three data pointers are refreshed
// whenever the caller passes different ones; the rest is fixed at planning.
struct DevTensor {
    const void *g;
    float *m;
    float *p;
    uint16_t *p_bf16;   // optional bf16 copy of the updated parameters (nullptr: none)
    int64_t numel;
    int64_t L;          // block length
    int64_t n_blocks;
    int64_t v_offset;   // first block's index in v
    int32_t gdtype;     // am_dtype
    int32_t wd;         // apply the decay line
    // two-pass path bookkeeping
    int64_t piece_len;        // elements per partial sum (last piece of a block may be shorter)
    int64_t pieces_per_block;
    int64_t piece_base;       // first partial of this tensor in the scratch array
    int64_t block_base;       // first per-block step size of this tensor in the scratch array
    int64_t mean_len;         // divisor of the block mean (the whole block's length for a part of a block)
    int32_t part_index;       // >= 0: this tensor is a part of a block; index of its externally supplied sum
    int32_t pad2;
};

// A run of work units that belong to one tensor; units are numbered
// consecutively over the segments of one kernel.
struct Seg {
    int64_t unit_begin;
    int32_t tensor;
    int32_t aux;
};

// Scalars of one step, computed on the host in double.
struct StepScalars {
    double beta2, omb2;     // beta2, 1-beta2
    double inv_bc2;         // 1 / (1-beta2^t)
    double lr_over_bc1;     // eta_t / (1-beta1^t)
    double eps;
    float beta1, omb1;      // beta1, 1-beta1
    float lr_wd;            // eta_t * lambda
    float gscale;           // gradients are multiplied by this on load (1 = off) ...
    const float *gscale_dev;  // ... and by this device scalar when not null
    const float *skip_flag;   // device scalar; non-zero: the step leaves everything untouched
    int32_t statistic;        // block statistic: 0 mean, 1 max, 2 min, 3 one-norm, 4 two-norm of g*g
    int32_t pad;
    const double *part_sums;  // whole-block sums of g*g for tensors that are parts of blocks
};

}  // namespace am

#endif  // ADAMMINI_INTERNAL_H_
