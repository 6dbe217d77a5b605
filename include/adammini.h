/*
 * adammini.h -- C ABI of the B200 Adam-mini optimizer-step library.
 *
 * The library performs, on one GPU, the per-step update of Adam-mini
 * (Algorithm 1 of the paper, "Adam-mini (General form)"; the boxed v_b rule of
 * the introduction) over all parameter tensors of a model:
 *
 *   for every block b (L contiguous elements of one tensor), at step t >= 1:
 *     v_b   <- (1-beta2) * mean(g_b * g_b) + beta2 * v_b          one scalar per block
 *     p_i   <- p_i - eta_t * lambda * p_i                          decoupled decay
 *     m_i   <- (1-beta1) * g_i + beta1 * m_i
 *     p_i   <- p_i - eta_t * (m_i / (1-beta1^t)) / (sqrt(v_b / (1-beta2^t)) + eps)
 *
 * Blocks follow the paper's partition rules (Algorithm 2, "Partition for
 * non-Transformers"; Algorithm 3, "Partition for Transformers"): token rows for
 * embedding/output, heads for query/key, output neurons for value /
 * attention projection / MLP, the whole tensor otherwise.
 *
 * Conventions
 *   - Weights are [out_features, in_features], row-major, contiguous.  Layouts
 *     that are transposed or flattened differently (the paper's appendix notes
 *     that they need re-ordering) are the caller's to re-order: the library
 *     sees only rows x cols.
 *   - Parameters (master copy), m and v are float32; gradients are float32 or
 *     bfloat16 per tensor.  m and v must be zero before step 1.
 *   - Every function returns an am_status (0 = success, negative = error) and
 *     never throws or aborts.  Pointers marked "device" are device addresses
 *     on the GPU that was current when adammini_create ran; "host" pointers
 *     are ordinary host addresses.
 *   - The caller owns params, grads, m, v.  The library owns its handle, the
 *     device copy of the block table and a small scratch area.
 */
#ifndef ADAMMINI_H_
#define ADAMMINI_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* How a tensor is cut into blocks (Algorithm 3 branches). */
typedef enum {
    AM_WHOLE  = 0,  /* one block: the ELSE branch of Algorithm 3, and Algorithm 2 */
    AM_ROWS   = 1,  /* value, attn.proj, mlp: one block per output neuron (row)    */
    AM_HEADS  = 2,  /* query, key: one block per head = rows/n_heads rows          */
    AM_TOKENS = 3,  /* embed, output: one block per token row                      */
    AM_FIXED  = 4,  /* explicit block length (any divisor of numel)                */
    AM_PART   = 5   /* a contiguous PART of one block whose other parts are held elsewhere (a flat
                       shard that cuts a block between data-parallel ranks): rows = 1, cols = the
                       local length, fixed_block_len = the length of the whole block.  The sum of
                       g*g over the whole block is supplied to the step (see am_step_extras)      */
} am_kind;

typedef enum { AM_F32 = 0, AM_BF16 = 1 } am_dtype;

typedef enum {
    AM_OK                   =  0,
    AM_ERR_INVALID_ARGUMENT = -1,  /* null pointer, step < 1, eps <= 0, beta outside [0,1), ... */
    AM_ERR_SHAPE            = -2,  /* rows/cols <= 0, rows % n_heads != 0, numel % block_len != 0 */
    AM_ERR_MISALIGNED       = -3,  /* a device pointer is not 16-byte aligned */
    AM_ERR_CUDA             = -4,  /* a CUDA call failed; see adammini_last_cuda_error */
    AM_ERR_TIMEOUT          = -5,  /* a bounded device-side wait gave up (reported by adammini_sync_status) */
    AM_ERR_ALLOC            = -6,  /* host or device allocation failed */
    AM_ERR_TOO_LARGE        = -7   /* a size exceeds what the entry point supports */
} am_status;

/* One parameter tensor as the caller describes it.  1-D tensors: rows = 1. */
typedef struct am_tensor_desc {
    int64_t rows, cols;
    int32_t kind;               /* am_kind */
    int32_t n_heads;            /* AM_HEADS only; rows % n_heads == 0 */
    int64_t fixed_block_len;    /* AM_FIXED: block length, (rows*cols) % fixed_block_len == 0;
                                   AM_PART: length of the whole block, >= rows*cols */
    int32_t grad_dtype;         /* am_dtype of this tensor's gradient */
    int32_t apply_weight_decay; /* 0: skip the decay line for this tensor */
} am_tensor_desc;

/* One row of the flat block table (one per tensor, caller's order).  Block b of
 * the tensor is elements [b*block_len, (b+1)*block_len); its second moment is
 * v[v_offset + b]. */
typedef struct am_table_row {
    int64_t numel, block_len, n_blocks, v_offset;
    int32_t kind, grad_dtype, wd, pad;
    int64_t mean_len;           /* divisor of the block mean: block_len, except for AM_PART (whole block's length) */
} am_table_row;

/* eta, beta1, beta2, eps, lambda of Algorithm 1.  Doubles, so the caller's
 * values reach the library unrounded; the kernels compute in float32. */
typedef struct am_hparams {
    double lr, beta1, beta2, eps, weight_decay;
} am_hparams;

typedef struct am_partition am_partition;
typedef struct am_handle am_handle;

/* ---- partitioner (host only; Algorithm 2 / Algorithm 3) ------------------------
 * Builds the flat block table from `n_tensors` descriptors (host array, read
 * during the call only).  On success *out owns the table; free it with
 * adammini_partition_free.  AM_ERR_SHAPE if a descriptor does not divide (or its
 * rows * cols overflows int64), AM_ERR_TOO_LARGE if the element count of the whole
 * table does, AM_ERR_INVALID_ARGUMENT for an unknown kind or dtype. */
int adammini_partition_build(const am_tensor_desc *descs, int32_t n_tensors, am_partition **out);

/* Number of tensors in the table. */
int32_t adammini_partition_num_tensors(const am_partition *part);

/* Copies the table into `rows` (host array of n_tensors entries, may be NULL)
 * and the total number of blocks (= length of v) into *total_blocks (may be NULL). */
int adammini_partition_export(const am_partition *part, am_table_row *rows, int64_t *total_blocks);

void adammini_partition_free(am_partition *part);

/* Algorithm 3's name tests in its order of precedence: "embed"/"output" ->
 * AM_TOKENS, "query"/"key" -> AM_HEADS, "value"/"attn.proj"/"mlp" -> AM_ROWS,
 * anything else AM_WHOLE.  `name` is a host C string.  Returns the am_kind. */
int32_t adammini_kind_from_name(const char *name);

/* ---- optimizer handle ----------------------------------------------------------
 * Creates a handle on the current CUDA device: copies the table (the partition
 * may be freed afterwards), plans the kernel launches, uploads the device
 * tables and allocates scratch.  Hyper-parameters are validated:
 * lr >= 0, 0 <= beta < 1, eps > 0, weight_decay >= 0. */
int adammini_create(const am_partition *part, const am_hparams *hp, am_handle **out);

/* eta_t of Algorithm 1 is time-varying: set it before the step it applies to. */
int adammini_set_lr(am_handle *h, double lr);
int adammini_set_hparams(am_handle *h, const am_hparams *hp);

/* One Adam-mini step (Algorithm 1) over every tensor of the table.
 *   params, grads, m : host arrays of n_tensors DEVICE pointers, in table order;
 *                      tensor i holds rows*cols contiguous elements
 *                      (params/m float32, grads of the tensor's grad_dtype).
 *                      All must be 16-byte aligned (AM_PART tensors: aligned to their element
 *                      size, since a shard may cut a block anywhere).  grads are only read.
 *   v                : DEVICE pointer, float32[total_blocks], 16-byte aligned.
 *   step             : t, 1-based.
 *   cuda_stream      : a cudaStream_t (NULL = the legacy default stream).
 * Asynchronous: work is enqueued on the stream and the call returns without
 * synchronising.  params, m and v are updated in place.  Calls on one handle
 * must be issued from one thread at a time and ordered on one stream (or
 * otherwise serialised), because they share the handle's scratch.
 * A step cannot be recorded into a CUDA graph (t and the hyper-parameters are
 * kernel arguments, and successive launches take turns on two work counters,
 * so a replay would repeat a stale step): a stream that is capturing is refused
 * with AM_ERR_INVALID_ARGUMENT and nothing is enqueued. */
int adammini_step(am_handle *h, void *const *params, const void *const *grads, void *const *m,
                  float *v, int64_t step, void *cuda_stream);

/* Optional extras of a step: trainer-side operations that sit next to
 * optimizer.step() in mixed-precision training and cost nothing when fused
 * into the same pass (the paper's Algorithm 1 is silent on them).
 *   params_bf16       host array of n_tensors DEVICE pointers (entries may be NULL), 16-byte
 *                     aligned: the updated parameter is also written there rounded to bfloat16
 *                     (round to nearest even) -- the working copy of a bf16 model.  NULL: none.
 *   grad_scale        every gradient is multiplied by this before use (1.0 = off): the inverse
 *                     loss scale and/or a global-norm clip coefficient known on the host.
 *   grad_scale_device optional DEVICE float multiplied in as well (a clip coefficient computed
 *                     on the device).  NULL: none.
 *   skip_flag         optional DEVICE float; if it is non-zero when the kernels run, the step
 *                     changes nothing (found-inf skip of dynamic loss scaling).  NULL: never skip. */
typedef struct am_step_extras {
    void *const *params_bf16;
    double grad_scale;
    const float *grad_scale_device;
    const float *skip_flag;
    const double *part_sums;   /* required when the table has AM_PART tensors: DEVICE array with one entry
                                  per AM_PART tensor, in table order: the sum of g*g (unscaled gradients)
                                  over the WHOLE block, i.e. the parts' sums from adammini_part_sums added
                                  up over all holders (an all-reduce between data-parallel ranks) */
} am_step_extras;

/* adammini_step with extras (`ex` may be NULL, which is adammini_step). */
int adammini_step_ex(am_handle *h, void *const *params, const void *const *grads, void *const *m,
                     float *v, int64_t step, void *cuda_stream, const am_step_extras *ex);

/* Sums of g*g of the table's AM_PART tensors (this holder's parts only), written to
 * `out` (DEVICE array, one double per AM_PART tensor in table order), asynchronously on
 * the stream.  grads: as for adammini_step (only the AM_PART entries are read).  The
 * caller adds the parts of every block over all its holders and passes the totals to
 * adammini_step_ex as am_step_extras.part_sums. */
int adammini_part_sums(am_handle *h, const void *const *grads, double *out, void *cuda_stream);

/* The same step for callers whose state lives in HOST memory (offloaded
 * optimizer state): params, grads, m are host arrays of HOST pointers, v is a
 * HOST pointer.  The library streams groups of tensors through device staging
 * buffers (host->device copies, the kernels above, device->host copies) on
 * internal streams and returns after everything has landed back in host
 * memory.  Pinned host memory gives full copy bandwidth; pageable works.
 * Every group runs with the launch shape this handle resolved, so the result
 * equals adammini_step's on the same handle bit for bit.
 * `staging_bytes` bounds the device memory used for staging (0 = default: 3 GiB, or three times
 * the largest tensor's p + m + g if that is more).  Tables with AM_PART tensors are not supported
 * here (AM_ERR_INVALID_ARGUMENT): their step needs the exchange of part sums in between. */
int adammini_step_host(am_handle *h, void *const *params, const void *const *grads, void *const *m,
                       float *v, int64_t step, int64_t staging_bytes);

/* One Adam-mini step on ONE tensor without any allocation.  (The paper has no
 * counterpart: this entry point exists for callers that must not allocate.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a
 * framework's memory-pool callback or a training loop whose allocator owns the
 * whole device, in a process that has handed all free memory to another
 * library, or in latency-critical sections where an allocation's implicit
 * synchronisation is not acceptable.  adammini_create allocates device tables
 * and scratch; this call allocates nothing, neither on the device nor through
 * any library: its scratch (partial sums of g*g and per-block step sizes) is a
 * fixed array compiled into the library, AM_NOALLOC_SCRATCH_BYTES of device
 * memory that every GPU holds from the moment the library is loaded on it
 * until the process exits.
 *
 *   param, m : DEVICE float32[numel], updated in place; grad: DEVICE, numel
 *              elements of grad_dtype, read only; v: DEVICE float32[numel/block_len],
 *              updated in place.  All 16-byte aligned.  m, v zero before step 1.
 *   block_len must divide numel.  Limits: numel/block_len <= AM_NOALLOC_MAX_BLOCKS
 *   and the number of partial sums, (numel/block_len) * ceil(block_len/32768)
 *   (pieces grow beyond 32768 elements only for blocks over 2^29 elements),
 *   <= AM_NOALLOC_MAX_PIECES; larger requests return AM_ERR_TOO_LARGE and do
 *   nothing.
 *
 * The arithmetic is that of adammini_step's two-pass path, and so are the bits
 * as long as a block has fewer than 256 partial sums (beyond that the other
 * path adds a block's partial sums in a different order).  cuda_stream must
 * belong to the device that is current at the call: that device's array is
 * used.  The first call on a device looks up the array's device address (once
 * per device, with that device current); make that first call outside any
 * stream capture.  Every call on a device shares the one array, which keeps whatever
 * the previous call left there: each call overwrites the entries it uses before
 * it reads them, so nothing needs clearing, but two calls whose kernels overlap
 * on the GPU (different streams, or different threads or processes' streams on
 * one context) race on it -- keep such calls on one stream or order them with
 * events.  Asynchronous on cuda_stream like adammini_step. */
#define AM_NOALLOC_MAX_BLOCKS 32768
#define AM_NOALLOC_MAX_PIECES 32768
#define AM_NOALLOC_SCRATCH_BYTES (AM_NOALLOC_MAX_PIECES * 8 + AM_NOALLOC_MAX_BLOCKS * 4)
int adammini_step_tensor_noalloc(void *param, const void *grad, void *m, float *v, int64_t numel,
                                 int64_t block_len, int32_t grad_dtype, int32_t apply_weight_decay,
                                 const am_hparams *hp, int64_t step, void *cuda_stream);

/* Waits for the stream and returns AM_OK, or AM_ERR_TIMEOUT if a device-side
 * bounded wait gave up during any step since the last call, or AM_ERR_CUDA. */
int adammini_sync_status(am_handle *h, void *cuda_stream);

/* Options and queries (keys below).  Unknown keys: AM_ERR_INVALID_ARGUMENT. */
typedef enum {
    AM_OPT_PATH           = 0, /* 0 = automatic; 1 = force the two-pass path for every tensor with
                                  block_len > 16 (correctness anchor: a second implementation of every
                                  other kernel family's work) */
    AM_OPT_STREAM_CTAS    = 1, /* persistent CTAs of the streaming kernel (0 = one per SM; at most 4096) */
    AM_OPT_CLUSTER_SIZE   = 2, /* CTAs per cluster for head-sized blocks: 1 to 8, lowered to the next size the
                                  device can run (0 = chosen by adammini_choose_cluster_size) */
    AM_OPT_STREAM_THREADS = 3, /* threads per consumer group of the streaming kernels, a multiple of 32
                                  from 64 to 512 (0 = default 256; anything else is rejected);
                                  groups x threads is capped at 512 */
    AM_OPT_PROFILE        = 4, /* n > 0: record CUDA events around each kernel family of every step (one
                                  at the start, one behind every family that launches something), keeping
                                  the latest n steps (n <= 4096); read them with adammini_get_profile.
                                  Setting the option again, or an option that changes the launch plan,
                                  restarts the record */
    AM_OPT_STREAM_CHUNK   = 5, /* how the streaming kernel's CTAs share the work: 0 = automatic (CTAs take one
                                  work item at a time -- a stage of packed blocks, or one long block -- from
                                  a shared counter: this evens out bandwidth differences between SMs and
                                  keeps all CTAs on one neighbourhood of memory; fixed ranges for tiny
                                  workloads); 1..4096 = that many items at a time; 1000000 = every CTA
                                  walks its own fixed, cost-balanced range.  Results are bit-identical in
                                  every mode */
    AM_OPT_CLUSTER_CHUNK  = 6, /* the same for the cluster kernel, in blocks handed to a cluster at a time */
    AM_OPT_STATISTIC      = 7, /* block statistic that feeds v: 0 = mean(g*g), Algorithm 1.  The ablation
                                  of the paper's appendix ("Ablation Studies on the Design of Adam-mini"),
                                  which it reports to train worse: 1 = max, 2 = min, 3 = 1-norm (sum),
                                  4 = 2-norm of the vector g*g.  Every kernel family takes the statistic
                                  as a parameter of its block reduction (g is still read once).  Blocks
                                  that hold a NaN gradient: their max / min is unspecified.  Tables with
                                  AM_PART tensors support the mean only */
    AM_OPT_STREAM_GROUPS  = 8, /* consumer groups per CTA of the streaming kernel, which own alternate
                                  work items: 1 or 2 (0 = default: 2; the cluster kernel runs one) */
    AM_OPT_WAIT_LIMIT_US  = 9, /* how long a device-side wait (for a staged copy, a barrier of a consumer
                                  group, a cluster exchange) polls before it gives up, in microseconds:
                                  100 to 60 000 000 (0 = default: 2 s).  A wait that gives up ends its
                                  kernel through the normal exit; adammini_sync_status then returns
                                  AM_ERR_TIMEOUT and the tensors of that step are partly updated */
    AM_OPT_TEST_STALL     = 10 /* for tests of that error path: n > 0 makes the thread that stages data
                                  withhold its n-th and later stages in every CTA of the streaming
                                  kernels (the tile kernel announces its copies without issuing them),
                                  so that the waits above run out.  Nothing faults and nothing waits
                                  without a limit.  0 = off */
} am_option;
int adammini_set_option(am_handle *h, int32_t key, int64_t value);

typedef enum {
    AM_Q_LAUNCHES_PER_STEP = 0, /* kernels one adammini_step enqueues */
    AM_Q_SCRATCH_BYTES     = 1, /* device scratch owned by the handle */
    AM_Q_TOTAL_BLOCKS      = 2,
    AM_Q_TOTAL_ELEMENTS    = 3,
    AM_Q_ELEMENTS_SMALL    = 4, /* elements routed to the short-block kernels (block_len <= 64, and blocks of
                                   up to 4096 elements whose starts are not 16-byte aligned) */
    AM_Q_ELEMENTS_STREAM   = 5, /* ... to the streaming kernel (its launch for rows, and the one for blocks of more
                                   than 4096 elements, up to 256 KB of gradients, whose starts are not 16-byte
                                   aligned) */
    AM_Q_ELEMENTS_CLUSTER  = 6, /* ... to the cluster kernel (head-sized blocks) */
    AM_Q_ELEMENTS_TWOPASS  = 7, /* ... to the two-pass path (blocks beyond on-chip/L2 reach: more than 4 MB of
                                   gradients, or more than 256 KB with unaligned starts; parts of blocks) */
    AM_Q_ALGORITHMIC_BYTES = 8, /* bytes one step must move: per tensor g once (twice for blocks beyond
                                   on-chip/L2 reach), m and p read+written, v read+written */
    AM_Q_BYTES_SMALL       = 9, /* the same, split by the kernel family that handles the tensor */
    AM_Q_BYTES_STREAM      = 10,
    AM_Q_BYTES_CLUSTER     = 11,
    AM_Q_BYTES_TWOPASS     = 12,
    AM_Q_STREAM_CTAS       = 13, /* launch shape of the streaming kernel */
    AM_Q_CLUSTER_SIZE      = 14,
    AM_Q_CLUSTER_COUNT     = 15,
    AM_Q_PART_TENSORS      = 16, /* number of AM_PART tensors in the table */
    AM_Q_L2_BYTES          = 17, /* what planning read from the device: L2 size, */
    AM_Q_SMEM_BYTES        = 18, /* most dynamic shared memory a CTA may ask for, */
    AM_Q_RESIDENT_CLUSTERS = 19  /* and, at 19 + (c - 1) for c = 1..8, how many clusters of c CTAs of the
                                    streaming kernel fit the device at once (with the handle's current
                                    threads per CTA): the inputs of adammini_choose_cluster_size */
} am_query;
int adammini_query(const am_handle *h, int32_t what, int64_t *value);

/* The planning rule behind AM_Q_CLUSTER_SIZE, as a function of what a handle reads from its
 * device (host only; no CUDA call): the CTAs per cluster chosen for head-sized blocks whose
 * gradients take `block_bytes`, on a device with `l2_bytes` of L2 that keeps
 * resident_clusters[c] clusters of c CTAs of the streaming kernel resident at once
 * (host array of 9 entries, c = 1..8; entry 0 is ignored; 0 = clusters of that size cannot
 * run).  A cluster reads a block's gradients twice and the second read should hit L2, so the
 * rule takes the smallest size (most clusters, most SMs busy) whose resident clusters keep no
 * more than a fixed share of L2 in flight, the largest size that can run otherwise, and 0 when
 * no cluster can run (such blocks then take the two-pass kernels).  Negative: am_status. */
int32_t adammini_choose_cluster_size(const int32_t *resident_clusters, int64_t l2_bytes, int64_t block_bytes);

/* With AM_OPT_PROFILE set: waits for the recorded steps and writes the mean device time in
 * milliseconds per step of each kernel family to ms[0..3] (host array): short-block
 * kernels, streaming kernel, cluster kernel, two-pass kernels (0 where none ran).  *n_steps
 * (may be NULL) receives the number of steps averaged. */
int adammini_get_profile(am_handle *h, float *ms, int32_t *n_steps);

/* Measurement aid (no step of Algorithm 1 runs here): a copy through the streaming kernel's
 * ring of shared-memory stages with nothing in between -- bulk asynchronous loads, bulk
 * asynchronous stores, one persistent CTA per SM, items handed out one at a time.  Item i reads
 * load_bytes at src + i * load_bytes and writes store_bytes (the first store_bytes of what it
 * read) at dst + i * store_bytes.  Timed by the caller with events on the stream, n_items *
 * (load_bytes + store_bytes) / time is what this device's memory gives a kernel with that mix
 * of reads and writes: the ceiling for the update's 10 bytes read and 8 written per parameter.
 *   src, dst : DEVICE, 16-byte aligned, at least n_items * load_bytes / store_bytes long
 *              (either may be NULL when its byte count is 0).
 *   load_bytes, store_bytes : multiples of 16 from 0 to 40960, not both 0; when both are
 *              set, store_bytes <= load_bytes.
 * Asynchronous on cuda_stream (which must not be capturing); waits inside are bounded like a
 * step's, and a wait that gives up is reported by adammini_sync_status.  Uses the handle's
 * device only, none of its tensors. */
int adammini_probe_ring_copy(am_handle *h, const void *src, void *dst, int64_t n_items, int32_t load_bytes,
                             int32_t store_bytes, void *cuda_stream);

/* The CUDA error code (cudaError_t as int) of the last AM_ERR_CUDA on this handle; with
 * h == NULL, of the calling thread's last adammini_create that failed with AM_ERR_CUDA. */
int adammini_last_cuda_error(const am_handle *h);

int adammini_destroy(am_handle *h);

/* Static string for a status code. */
const char *adammini_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* ADAMMINI_H_ */
