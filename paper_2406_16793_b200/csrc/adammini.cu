// Host side of the Adam-mini step library: handle, launch planning, C ABI.
// Every step of Algorithm 1 of the paper runs in the kernels of
// kernels_basic.cuh and kernels_stream.cuh; this file only validates, plans
// and launches.
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "adammini_internal.h"
#include "kernels_basic.cuh"
#include "kernels_stream.cuh"
#include "kernels_tile.cuh"
#include "kernels_probe.cuh"
#include "host_state.h"

using namespace am;

namespace {

constexpr int kNumOptions = 11;

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

int cuda_fail(am_handle *h, cudaError_t e) {
    if (h) h->last_cuda_error = static_cast<int>(e);
    return AM_ERR_CUDA;
}

#define AM_CUDA(h, call)                                   \
    do {                                                   \
        cudaError_t e__ = (call);                          \
        if (e__ != cudaSuccess) return cuda_fail((h), e__); \
    } while (0)

int validate_hparams(const am_hparams *hp) {
    if (!hp) return AM_ERR_INVALID_ARGUMENT;
    const double vals[5] = {hp->lr, hp->beta1, hp->beta2, hp->eps, hp->weight_decay};
    for (double x : vals)
        if (!std::isfinite(x)) return AM_ERR_INVALID_ARGUMENT;
    if (hp->lr < 0.0 || hp->weight_decay < 0.0 || hp->eps <= 0.0) return AM_ERR_INVALID_ARGUMENT;
    if (hp->beta1 < 0.0 || hp->beta1 >= 1.0 || hp->beta2 < 0.0 || hp->beta2 >= 1.0)
        return AM_ERR_INVALID_ARGUMENT;
    return AM_OK;
}

void release_plan(am_handle *h) {
    if (h->arena) cudaFree(h->arena);
    h->arena = nullptr;
    h->arena_bytes = 0;
    h->planned = false;
    h->ptrs_valid = false;
}

// Decide the kernel family of every tensor, build the unit tables and the
// device arena.  Called at creation and after an option changes.
int build_plan(am_handle *h) {
    release_plan(h);
    const int n = static_cast<int>(h->rows.size());
    h->path.assign(n, PATH_TWOPASS);
    h->host_tensors.assign(n, DevTensor{});
    std::vector<Seg> small_segs, tile_segs, piece_segs, block_segs, part_segs, wide_segs;
    int64_t tile_units = 0;
    int64_t wide_units = 0;
    std::vector<int32_t> part_tensors;
    int64_t part_units = 0;
    int64_t small_units = 0, piece_units = 0, block_units = 0;
    for (int k = 0; k < 4; ++k) h->elems_by_path[k] = h->bytes_by_path[k] = 0;
    h->algorithmic_bytes = 0;

    StreamPlanInput sin;
    sin.ctas = static_cast<int>(h->opt[AM_OPT_STREAM_CTAS]);
    sin.cluster_size = static_cast<int>(h->opt[AM_OPT_CLUSTER_SIZE]);
    sin.threads = static_cast<int>(h->opt[AM_OPT_STREAM_THREADS]);
    sin.groups = static_cast<int>(h->opt[AM_OPT_STREAM_GROUPS]);
    sin.chunk = static_cast<int>(h->opt[AM_OPT_STREAM_CHUNK]);
    sin.cluster_chunk = static_cast<int>(h->opt[AM_OPT_CLUSTER_CHUNK]);

    {
        int threads, groups;
        stream_consumer_shape(sin.threads, sin.groups, &threads, &groups);
        stream_probe_clusters(&h->caps, 32 + threads * groups);
        sin.caps = h->caps;
    }
    bool clusters_ok = false;
    for (int c = 1; c <= kMaxCluster; ++c) clusters_ok |= h->caps.resident[c] > 0;
    bool stream_ok;         // the ring needs at least two stages of the larger layout
    {
        int g_region, stage_bytes, n_stages;
        stream_stage_layout(true, h->caps.smem_optin, &g_region, &stage_bytes, &n_stages);
        stream_ok = n_stages >= 2;
    }

    for (int i = 0; i < n; ++i) {
        const am_table_row &r = h->rows[i];
        DevTensor &t = h->host_tensors[i];
        t.numel = r.numel;
        t.L = r.block_len;
        t.n_blocks = r.n_blocks;
        t.v_offset = r.v_offset;
        t.gdtype = r.grad_dtype;
        t.wd = r.wd;
        t.mean_len = r.mean_len;
        t.part_index = -1;
        const int64_t gsz = r.grad_dtype == AM_BF16 ? 2 : 4;

        int path;
        bool edges = false;
        if (r.kind == AM_PART) path = PATH_TWOPASS;          // its sum of squares comes from outside
        else if (r.block_len <= kSmallMaxL && !(h->opt[AM_OPT_PATH] == 1 && r.block_len > 16)) path = PATH_SMALL;
        else if (h->opt[AM_OPT_PATH] == 1) path = PATH_TWOPASS;
        else {
            path = stream_ok ? stream_classify(r.block_len, r.grad_dtype, clusters_ok, &edges) : PATH_TWOPASS;
            // block starts off the 16-byte grid: the tile kernel copes, up to its tile size
            if (path == PATH_TWOPASS && r.block_len <= kTileMaxL) path = PATH_SMALL;
        }
        h->path[i] = path;
        h->elems_by_path[path] += r.numel;

        // bytes the update must move: g once if a block can stay on chip / in
        // L2 between its reduction and its update, twice otherwise
        const int64_t g_reads = r.block_len * gsz > kClusterMaxBlockBytes ? 2 : 1;
        const int64_t tensor_bytes = r.numel * (g_reads * gsz + 16) + r.n_blocks * 8;
        h->algorithmic_bytes += tensor_bytes;
        h->bytes_by_path[path] += tensor_bytes;

        if (path == PATH_SMALL) {
            Seg s;
            s.tensor = i;
            s.aux = small_vec_ok(r.block_len, r.numel, r.v_offset) ? 1 : 0;
            if (s.aux) {                // blocks of one to three elements, aligned: straight from registers
                s.unit_begin = small_units;
                small_units += ceil_div(r.numel, small_vec_unit(r.block_len));
                small_segs.push_back(s);
            } else {                    // tiles of whole blocks staged in shared memory
                s.unit_begin = tile_units;
                tile_units += ceil_div(r.n_blocks, tile_blocks(r.block_len));
                tile_segs.push_back(s);
            }
        } else if (path == PATH_TWOPASS) {
            int64_t piece_len = r.block_len, ppb = 1;
            if (r.block_len > kPieceMax) {
                ppb = std::min<int64_t>(ceil_div(r.block_len, kPieceMax), kMaxPiecesPerBlock);
                piece_len = ceil_div(ceil_div(r.block_len, ppb), 1024) * 1024;
                ppb = ceil_div(r.block_len, piece_len);
            }
            t.piece_len = piece_len;
            t.pieces_per_block = ppb;
            t.piece_base = piece_units;
            t.block_base = block_units;
            Seg s;
            s.unit_begin = piece_units;
            s.tensor = i;
            s.aux = r.kind != AM_PART ? 1 : 0;   // 16-byte accesses; parts may start at any address: single elements
            piece_segs.push_back(s);
            if (r.kind == AM_PART) {
                t.part_index = static_cast<int32_t>(part_tensors.size());
                part_tensors.push_back(i);
                Seg ps = s;
                ps.unit_begin = part_units;
                part_segs.push_back(ps);
                part_units += r.n_blocks * ppb;
            }
            Seg b;
            b.unit_begin = block_units;
            b.tensor = i;
            b.aux = 0;
            block_segs.push_back(b);
            if (ppb >= kWideBlockPieces) {          // finalized by a CTA per block
                Seg ws = b;
                ws.unit_begin = wide_units;
                wide_segs.push_back(ws);
                wide_units += r.n_blocks;
            }
            piece_units += r.n_blocks * ppb;
            block_units += r.n_blocks;
        } else {
            stream_add_tensor(sin, i, r, path, edges);
        }
    }
    if (part_units > 0x7fffffffLL || wide_units > 0x7fffffffLL) return AM_ERR_TOO_LARGE;
    // Segments of the register kernel by block length (one launch per length present).
    int64_t small_units_by_len[kSmallVecMaxL + 1] = {};
    {
        std::vector<Seg> ordered;
        int64_t next = 0;
        for (int len = 1; len <= kSmallVecMaxL; ++len) {
            const int64_t begin = next;
            for (const Seg &sg : small_segs) {
                const am_table_row &r = h->rows[sg.tensor];
                if (r.block_len != len) continue;
                Seg o = sg;
                o.unit_begin = next;
                next += ceil_div(r.numel, small_vec_unit(len));
                ordered.push_back(o);
            }
            small_units_by_len[len] = next - begin;
        }
        small_segs.swap(ordered);
    }
    // Tiles of short blocks first, then those of longer ones: the two kinds are launched
    // separately, each with the shared-memory layout it needs (four CTAs per SM for both).
    int64_t tile_short_units = 0;
    {
        std::vector<Seg> ordered;
        int64_t next = 0;
        for (int pass = 0; pass < 2; ++pass) {
            for (const Seg &sg : tile_segs) {
                const am_table_row &r = h->rows[sg.tensor];
                if ((r.block_len <= kSmallMaxL) != (pass == 0)) continue;
                Seg o = sg;
                o.unit_begin = next;
                next += ceil_div(r.n_blocks, tile_blocks(r.block_len));
                ordered.push_back(o);
            }
            if (pass == 0) tile_short_units = next;
        }
        tile_segs.swap(ordered);
    }
    if (small_units > 0x7fffffffLL || tile_units > 0x7fffffffLL || piece_units > 0x7fffffffLL || ceil_div(block_units, kThreads / 32) > 0x7fffffffLL)
        return AM_ERR_TOO_LARGE;

    StreamPlan &sp = h->stream;
    stream_finish_plan(sin, &sp);
    sp.v_len = h->total_blocks;

    // device arena: tensor table, unit tables, scratch
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = round_up(off + bytes, 256); return o; };
    const size_t o_tensors = take(sizeof(DevTensor) * std::max(n, 1));
    const size_t o_small = take(sizeof(Seg) * std::max<size_t>(small_segs.size(), 1));
    const size_t o_tile = take(sizeof(Seg) * std::max<size_t>(tile_segs.size(), 1));
    const size_t o_piece = take(sizeof(Seg) * std::max<size_t>(piece_segs.size(), 1));
    const size_t o_block = take(sizeof(Seg) * std::max<size_t>(block_segs.size(), 1));
    const size_t o_partials = take(sizeof(double) * std::max<int64_t>(piece_units, 1));
    const size_t o_steps = take(sizeof(float) * std::max<int64_t>(block_units, 1));
    const size_t o_stream = take(std::max<size_t>(sp.table_bytes(), 16));
    const size_t o_wide_segs = take(sizeof(Seg) * std::max<size_t>(wide_segs.size(), 1));
    const size_t o_part_segs = take(sizeof(Seg) * std::max<size_t>(part_segs.size(), 1));
    const size_t o_part_list = take(sizeof(int32_t) * std::max<size_t>(part_tensors.size(), 1));
    const size_t o_probe = take(128);
    h->arena_bytes = off;
    AM_CUDA(h, cudaMalloc(&h->arena, h->arena_bytes));
    char *base = static_cast<char *>(h->arena);
    h->d_tensors = reinterpret_cast<DevTensor *>(base + o_tensors);
    h->d_small_segs = reinterpret_cast<Seg *>(base + o_small);
    h->d_tile_segs = reinterpret_cast<Seg *>(base + o_tile);
    h->n_tile_segs = static_cast<int>(tile_segs.size());
    h->tile_units = tile_units;
    h->tile_short_units = tile_short_units;
    h->d_piece_segs = reinterpret_cast<Seg *>(base + o_piece);
    h->d_block_segs = reinterpret_cast<Seg *>(base + o_block);
    h->d_partials = reinterpret_cast<double *>(base + o_partials);
    h->d_probe_counter = reinterpret_cast<unsigned long long *>(base + o_probe);
    h->d_block_steps = reinterpret_cast<float *>(base + o_steps);
    h->n_small_segs = static_cast<int>(small_segs.size());
    h->n_piece_segs = static_cast<int>(piece_segs.size());
    h->n_block_segs = static_cast<int>(block_segs.size());
    h->d_wide_segs = reinterpret_cast<Seg *>(base + o_wide_segs);
    h->n_wide_segs = static_cast<int>(wide_segs.size());
    h->wide_units = wide_units;
    if (!wide_segs.empty())
        AM_CUDA(h, cudaMemcpy(h->d_wide_segs, wide_segs.data(), sizeof(Seg) * wide_segs.size(), cudaMemcpyHostToDevice));
    h->d_part_segs = reinterpret_cast<Seg *>(base + o_part_segs);
    h->d_part_tensors = reinterpret_cast<int32_t *>(base + o_part_list);
    h->n_parts = static_cast<int>(part_tensors.size());
    h->part_units = part_units;
    if (!part_segs.empty()) {
        AM_CUDA(h, cudaMemcpy(h->d_part_segs, part_segs.data(), sizeof(Seg) * part_segs.size(), cudaMemcpyHostToDevice));
        AM_CUDA(h, cudaMemcpy(h->d_part_tensors, part_tensors.data(), sizeof(int32_t) * part_tensors.size(), cudaMemcpyHostToDevice));
    }
    h->small_units = small_units;
    for (int len = 1; len <= kSmallVecMaxL; ++len) h->small_units_by_len[len] = small_units_by_len[len];
    h->piece_units = piece_units;
    h->block_units = block_units;
    if (!small_segs.empty())
        AM_CUDA(h, cudaMemcpy(h->d_small_segs, small_segs.data(), sizeof(Seg) * small_segs.size(), cudaMemcpyHostToDevice));
    if (!tile_segs.empty())
        AM_CUDA(h, cudaMemcpy(h->d_tile_segs, tile_segs.data(), sizeof(Seg) * tile_segs.size(), cudaMemcpyHostToDevice));
    if (!piece_segs.empty())
        AM_CUDA(h, cudaMemcpy(h->d_piece_segs, piece_segs.data(), sizeof(Seg) * piece_segs.size(), cudaMemcpyHostToDevice));
    if (!block_segs.empty())
        AM_CUDA(h, cudaMemcpy(h->d_block_segs, block_segs.data(), sizeof(Seg) * block_segs.size(), cudaMemcpyHostToDevice));
    {
        cudaError_t e = sp.upload(base + o_stream);
        if (e != cudaSuccess) return cuda_fail(h, e);
    }

    h->prof_steps = 0;       // recorded steps belong to the plan that launched them
    h->launches = (small_units_by_len[1] ? 1 : 0) + (small_units_by_len[2] ? 1 : 0) + (small_units_by_len[3] ? 1 : 0) + (tile_short_units ? 1 : 0) + (tile_units > tile_short_units ? 1 : 0) + (piece_units ? 3 : 0) + (wide_units ? 1 : 0) + sp.launches();
    h->planned = true;
    return AM_OK;
}

// Kernel families in the order a step launches them (and adammini_get_profile reports them):
// short blocks, streaming launches, cluster launch, two-pass kernels.
inline void active_families(const am_handle *h, bool active[4]) {
    active[0] = h->small_units > 0 || h->tile_units > 0;
    active[1] = h->stream.main.active() || h->stream.edge.active();
    active[2] = h->stream.clus.active();
    active[3] = h->piece_units > 0;
}

// Refresh the device tensor table if any data pointer changed.
int refresh_pointers(am_handle *h, void *const *params, const void *const *grads, void *const *m,
                     void *const *params_bf16, cudaStream_t stream) {
    const int n = static_cast<int>(h->rows.size());
    bool changed = !h->ptrs_valid;
    for (int i = 0; i < n; ++i) {
        DevTensor &t = h->host_tensors[i];
        uint16_t *pb = params_bf16 ? static_cast<uint16_t *>(params_bf16[i]) : nullptr;
        if (t.g != grads[i] || t.m != m[i] || t.p != params[i] || t.p_bf16 != pb) {
            t.p_bf16 = pb;
            t.g = grads[i];
            t.m = static_cast<float *>(m[i]);
            t.p = static_cast<float *>(params[i]);
            changed = true;
        }
    }
    if (!changed || n == 0) return AM_OK;
    const int k = h->next_pinned;
    h->next_pinned ^= 1;
    if (h->ev_pending[k]) {
        AM_CUDA(h, cudaEventSynchronize(h->ev[k]));   // the copy that last read this buffer
        h->ev_pending[k] = false;
    }
    std::memcpy(h->pinned[k], h->host_tensors.data(), sizeof(DevTensor) * n);
    AM_CUDA(h, cudaMemcpyAsync(h->d_tensors, h->pinned[k], sizeof(DevTensor) * n, cudaMemcpyHostToDevice, stream));
    AM_CUDA(h, cudaEventRecord(h->ev[k], stream));
    h->ev_pending[k] = true;
    h->ptrs_valid = true;
    return AM_OK;
}

}  // namespace

extern "C" {

// CUDA error of the last adammini_create that failed in this thread (there is no handle to ask then)
static thread_local int g_create_cuda_error = 0;

int adammini_create(const am_partition *part, const am_hparams *hp, am_handle **out) {
    if (!out) return AM_ERR_INVALID_ARGUMENT;
    *out = nullptr;
    if (!part) return AM_ERR_INVALID_ARGUMENT;
    int rc = validate_hparams(hp);
    if (rc != AM_OK) return rc;
    am_handle *h = new (std::nothrow) am_handle();
    if (!h) return AM_ERR_ALLOC;
    try {
        h->rows = part->rows;
    } catch (...) {
        delete h;
        return AM_ERR_ALLOC;
    }
    h->total_blocks = part->total_blocks;
    for (const am_table_row &r : h->rows) h->total_elems += r.numel;
    h->hp = *hp;

    cudaError_t e = cudaGetDevice(&h->device);
    cudaDeviceProp prop;
    if (e == cudaSuccess) e = cudaGetDeviceProperties(&prop, h->device);
    if (e == cudaSuccess) {
        h->sm_count = prop.multiProcessorCount;
        h->caps.sm_count = prop.multiProcessorCount;
        h->caps.smem_optin = prop.sharedMemPerBlockOptin;
        h->caps.l2_bytes = prop.l2CacheSize;
        const size_t n = std::max<size_t>(h->rows.size(), 1);
        for (int k = 0; k < 2 && e == cudaSuccess; ++k) {
            e = cudaMallocHost(&h->pinned[k], sizeof(DevTensor) * n);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev[k], cudaEventDisableTiming);
        }
    }
    if (e == cudaSuccess) e = cudaMallocHost(&h->error_word, sizeof(int));
    if (e == cudaSuccess) *h->error_word = 0;
    if (e == cudaSuccess) e = stream_configure_kernels(h->caps.smem_optin);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(tile_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kTileSmemBytes);
    if (e == cudaSuccess && h->caps.smem_optin >= kCtrlBytes + 2 * static_cast<size_t>(kProbeStageBytes))
        e = cudaFuncSetAttribute(ring_copy_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(h->caps.smem_optin));
    if (e != cudaSuccess) {
        g_create_cuda_error = static_cast<int>(e);
        adammini_destroy(h);
        return AM_ERR_CUDA;
    }
    rc = build_plan(h);
    if (rc != AM_OK) {
        if (rc == AM_ERR_CUDA) g_create_cuda_error = h->last_cuda_error;
        adammini_destroy(h);
        return rc;
    }
    *out = h;
    return AM_OK;
}

int adammini_set_lr(am_handle *h, double lr) {
    if (!h || !std::isfinite(lr) || lr < 0.0) return AM_ERR_INVALID_ARGUMENT;
    h->hp.lr = lr;
    return AM_OK;
}

int adammini_set_hparams(am_handle *h, const am_hparams *hp) {
    if (!h) return AM_ERR_INVALID_ARGUMENT;
    const int rc = validate_hparams(hp);
    if (rc != AM_OK) return rc;
    h->hp = *hp;
    return AM_OK;
}

int adammini_set_option(am_handle *h, int32_t key, int64_t value) {
    if (!h || key < 0 || key >= kNumOptions || value < 0) return AM_ERR_INVALID_ARGUMENT;
    if (key == AM_OPT_PATH && value > 1) return AM_ERR_INVALID_ARGUMENT;
    if ((key == AM_OPT_STREAM_CHUNK || key == AM_OPT_CLUSTER_CHUNK) && value > 4096 && value != kStaticRanges)
        return AM_ERR_INVALID_ARGUMENT;
    if (key == AM_OPT_STATISTIC && value > 4) return AM_ERR_INVALID_ARGUMENT;
    if (key == AM_OPT_STREAM_GROUPS && value > kMaxGroups) return AM_ERR_INVALID_ARGUMENT;
    if (key == AM_OPT_CLUSTER_SIZE && value > kMaxCluster) return AM_ERR_INVALID_ARGUMENT;
    // a consumer group is made of whole warps (its shuffles and barriers count warps)
    if (key == AM_OPT_STREAM_THREADS && value != 0 && (value % 32 != 0 || value < 64 || value > 512))
        return AM_ERR_INVALID_ARGUMENT;
    if (key == AM_OPT_STREAM_CTAS && value > kMaxStreamCtas) return AM_ERR_INVALID_ARGUMENT;
    if (key == AM_OPT_WAIT_LIMIT_US && value != 0 && (value < 100 || value > 60000000)) return AM_ERR_INVALID_ARGUMENT;
    if (key == AM_OPT_WAIT_LIMIT_US || key == AM_OPT_TEST_STALL) {      // read at every launch: nothing to plan again
        h->opt[key] = value;
        if (h->host_step) host_step_release(h);
        return AM_OK;
    }
    if (key == AM_OPT_PROFILE) {
        if (value > 4096) return AM_ERR_INVALID_ARGUMENT;
        for (cudaEvent_t e : h->prof_ev) cudaEventDestroy(e);
        h->prof_ev.clear();
        try {
            h->prof_ev.resize(static_cast<size_t>(value) * 5, nullptr);
        } catch (...) {
            return AM_ERR_ALLOC;
        }
        for (cudaEvent_t &e : h->prof_ev) AM_CUDA(h, cudaEventCreate(&e));
        h->opt[key] = value;
        h->prof_steps = 0;
        return AM_OK;
    }
    if (h->opt[key] == value) return AM_OK;
    AM_CUDA(h, cudaDeviceSynchronize());    // the old tables may still be in use
    const int64_t old = h->opt[key];
    h->opt[key] = value;
    int rc = build_plan(h);
    if (rc != AM_OK) {
        h->opt[key] = old;
        build_plan(h);
    }
    host_step_release(h);                   // its per-group handles were planned with the old options
    return rc;
}

int adammini_query(const am_handle *h, int32_t what, int64_t *value) {
    if (!h || !value) return AM_ERR_INVALID_ARGUMENT;
    switch (what) {
    case AM_Q_LAUNCHES_PER_STEP: *value = h->launches; break;
    case AM_Q_SCRATCH_BYTES: *value = static_cast<int64_t>(h->arena_bytes); break;
    case AM_Q_TOTAL_BLOCKS: *value = h->total_blocks; break;
    case AM_Q_TOTAL_ELEMENTS: *value = h->total_elems; break;
    case AM_Q_ELEMENTS_SMALL: *value = h->elems_by_path[PATH_SMALL]; break;
    case AM_Q_ELEMENTS_STREAM: *value = h->elems_by_path[PATH_STREAM]; break;
    case AM_Q_ELEMENTS_CLUSTER: *value = h->elems_by_path[PATH_CLUSTER]; break;
    case AM_Q_ELEMENTS_TWOPASS: *value = h->elems_by_path[PATH_TWOPASS]; break;
    case AM_Q_ALGORITHMIC_BYTES: *value = h->algorithmic_bytes; break;
    case AM_Q_BYTES_SMALL: *value = h->bytes_by_path[PATH_SMALL]; break;
    case AM_Q_BYTES_STREAM: *value = h->bytes_by_path[PATH_STREAM]; break;
    case AM_Q_BYTES_CLUSTER: *value = h->bytes_by_path[PATH_CLUSTER]; break;
    case AM_Q_BYTES_TWOPASS: *value = h->bytes_by_path[PATH_TWOPASS]; break;
    case AM_Q_STREAM_CTAS: *value = h->stream.main.grid; break;
    case AM_Q_CLUSTER_SIZE: *value = h->stream.clus.active() ? h->stream.clus.cluster : 0; break;
    case AM_Q_PART_TENSORS: *value = h->n_parts; break;
    case AM_Q_CLUSTER_COUNT: *value = h->stream.clus.active() ? h->stream.clus.grid / h->stream.clus.cluster : 0; break;
    case AM_Q_L2_BYTES: *value = h->caps.l2_bytes; break;
    case AM_Q_SMEM_BYTES: *value = static_cast<int64_t>(h->caps.smem_optin); break;
    default:
        if (what >= AM_Q_RESIDENT_CLUSTERS && what < AM_Q_RESIDENT_CLUSTERS + kMaxCluster) {
            *value = h->caps.resident[what - AM_Q_RESIDENT_CLUSTERS + 1];
            break;
        }
        return AM_ERR_INVALID_ARGUMENT;
    }
    return AM_OK;
}

int32_t adammini_choose_cluster_size(const int32_t *resident_clusters, int64_t l2_bytes, int64_t block_bytes) {
    if (!resident_clusters || l2_bytes < 0 || block_bytes < 0) return AM_ERR_INVALID_ARGUMENT;
    int resident[kMaxCluster + 1] = {};
    for (int c = 1; c <= kMaxCluster; ++c) resident[c] = resident_clusters[c];
    return choose_cluster_size(resident, l2_bytes, block_bytes);
}

int adammini_last_cuda_error(const am_handle *h) { return h ? h->last_cuda_error : g_create_cuda_error; }

int adammini_step(am_handle *h, void *const *params, const void *const *grads, void *const *m,
                  float *v, int64_t step, void *cuda_stream) {
    return adammini_step_ex(h, params, grads, m, v, step, cuda_stream, nullptr);
}

int adammini_step_ex(am_handle *h, void *const *params, const void *const *grads, void *const *m,
                     float *v, int64_t step, void *cuda_stream, const am_step_extras *ex) {
    if (!h || !h->planned || step < 1) return AM_ERR_INVALID_ARGUMENT;
    if (ex && !(std::isfinite(ex->grad_scale))) return AM_ERR_INVALID_ARGUMENT;
    const int n = static_cast<int>(h->rows.size());
    if (n == 0) return AM_OK;
    if (!params || !grads || !m || !v) return AM_ERR_INVALID_ARGUMENT;
    for (int i = 0; i < n; ++i) {
        if (!params[i] || !grads[i] || !m[i]) return AM_ERR_INVALID_ARGUMENT;
        if (h->rows[i].kind == AM_PART) {      // a part of a block may start at any element
            const uintptr_t gmask = h->rows[i].grad_dtype == AM_BF16 ? 1u : 3u;
            if ((reinterpret_cast<uintptr_t>(params[i]) & 3u) || (reinterpret_cast<uintptr_t>(m[i]) & 3u) ||
                (reinterpret_cast<uintptr_t>(grads[i]) & gmask))
                return AM_ERR_MISALIGNED;
        } else if (!aligned16(params[i]) || !aligned16(grads[i]) || !aligned16(m[i])) {
            return AM_ERR_MISALIGNED;
        }
    }
    if (!aligned16(v)) return AM_ERR_MISALIGNED;
    if (h->n_parts > 0 && (!ex || !ex->part_sums || h->opt[AM_OPT_STATISTIC] != 0)) return AM_ERR_INVALID_ARGUMENT;
    if (ex && ex->params_bf16)
        for (int i = 0; i < n; ++i)
            if (!aligned16(ex->params_bf16[i])) return AM_ERR_MISALIGNED;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

    int dev = -1;
    AM_CUDA(h, cudaGetDevice(&dev));
    if (dev != h->device) return AM_ERR_INVALID_ARGUMENT;
    // A step is not a replayable graph node: t and the hyper-parameters are kernel arguments, the
    // tensor table is re-uploaded when a pointer changes, and consecutive launches of a shape take
    // turns on two work counters.  A capturing stream is refused before anything is enqueued.
    cudaStreamCaptureStatus capture = cudaStreamCaptureStatusNone;
    AM_CUDA(h, cudaStreamIsCapturing(stream, &capture));
    if (capture != cudaStreamCaptureStatusNone) return AM_ERR_INVALID_ARGUMENT;

    int rc = refresh_pointers(h, params, grads, m, ex ? ex->params_bf16 : nullptr, stream);
    if (rc != AM_OK) return rc;

    // scalars of this step (Algorithm 1: bias corrections use beta^t)
    const am_hparams &hp = h->hp;
    const double bc1 = 1.0 - std::pow(hp.beta1, static_cast<double>(step));
    const double bc2 = 1.0 - std::pow(hp.beta2, static_cast<double>(step));
    StepScalars sc;
    sc.beta2 = hp.beta2;
    sc.omb2 = 1.0 - hp.beta2;
    sc.inv_bc2 = 1.0 / bc2;
    sc.lr_over_bc1 = hp.lr / bc1;
    sc.eps = hp.eps;
    sc.beta1 = static_cast<float>(hp.beta1);
    sc.omb1 = static_cast<float>(1.0 - hp.beta1);
    sc.lr_wd = static_cast<float>(hp.lr * hp.weight_decay);
    sc.gscale = ex ? static_cast<float>(ex->grad_scale) : 1.f;
    sc.gscale_dev = ex ? ex->grad_scale_device : nullptr;
    sc.skip_flag = ex ? ex->skip_flag : nullptr;
    sc.statistic = static_cast<int32_t>(h->opt[AM_OPT_STATISTIC]);
    sc.pad = 0;
    sc.part_sums = ex ? ex->part_sums : nullptr;

    const unsigned long long wait_limit_ns =
        h->opt[AM_OPT_WAIT_LIMIT_US] ? static_cast<unsigned long long>(h->opt[AM_OPT_WAIT_LIMIT_US]) * 1000ull : kWaitTimeoutNs;
    h->stream.wait_limit_ns = wait_limit_ns;
    h->stream.stall_after = static_cast<int>(std::min<int64_t>(h->opt[AM_OPT_TEST_STALL], 1 << 30));
    const bool prof = h->opt[AM_OPT_PROFILE] != 0;
    cudaEvent_t *pev = prof ? &h->prof_ev[(h->prof_steps % h->opt[AM_OPT_PROFILE]) * 5] : nullptr;
    // An event behind every family that launches something (none behind the others: on steps of a
    // few hundred microseconds each event costs a percent).
    bool fam[4] = {false, false, false, false};
    if (prof) {
        active_families(h, fam);
        AM_CUDA(h, cudaEventRecord(pev[0], stream));
    }
    if (h->small_units || h->tile_units) {
        SmallScalars ss;
        ss.beta1 = sc.beta1;
        ss.omb1 = sc.omb1;
        ss.beta2 = static_cast<float>(hp.beta2);
        ss.omb2 = static_cast<float>(1.0 - hp.beta2);
        ss.inv_bc2 = static_cast<float>(sc.inv_bc2);
        ss.lr_over_bc1 = static_cast<float>(sc.lr_over_bc1);
        ss.eps = static_cast<float>(hp.eps);
        ss.lr_wd = sc.lr_wd;
        ss.gscale = sc.gscale;
        ss.gscale_dev = sc.gscale_dev;
        ss.skip_flag = sc.skip_flag;
        ss.statistic = sc.statistic;
        ss.stall = h->opt[AM_OPT_TEST_STALL] != 0;
        ss.wait_limit_ns = wait_limit_ns;
        int64_t first = 0;
        for (int len = 1; len <= kSmallVecMaxL; ++len) {
            const int64_t units = h->small_units_by_len[len];
            if (!units) continue;
            const unsigned grid = static_cast<unsigned>(units);
            if (len == 1) small_kernel<1><<<grid, kThreads, 0, stream>>>(h->d_tensors, h->d_small_segs, h->n_small_segs, v, ss, first);
            else if (len == 2) small_kernel<2><<<grid, kThreads, 0, stream>>>(h->d_tensors, h->d_small_segs, h->n_small_segs, v, ss, first);
            else small_kernel<3><<<grid, kThreads, 0, stream>>>(h->d_tensors, h->d_small_segs, h->n_small_segs, v, ss, first);
            AM_CUDA(h, cudaGetLastError());
            first += units;
        }
        if (h->tile_units) {
            const int64_t n_short = h->tile_short_units, n_long = h->tile_units - n_short;
            if (n_short) {
                tile_kernel<<<static_cast<unsigned>(n_short), kThreads, kTileSmemShortBytes, stream>>>(
                    h->d_tensors, h->d_tile_segs, h->n_tile_segs, v, ss, h->error_word, kTileShortLinear, 0);
                AM_CUDA(h, cudaGetLastError());
            }
            if (n_long) {
                tile_kernel<<<static_cast<unsigned>(n_long), kThreads, kTileSmemLongBytes, stream>>>(
                    h->d_tensors, h->d_tile_segs, h->n_tile_segs, v, ss, h->error_word, kTileLinear, n_short);
                AM_CUDA(h, cudaGetLastError());
            }
        }
    }
    h->stream.bf16_copies = ex && ex->params_bf16;
    if (fam[0]) AM_CUDA(h, cudaEventRecord(pev[1], stream));
    AM_CUDA(h, h->stream.launch_main(h->d_tensors, v, sc, h->error_word, stream));
    AM_CUDA(h, h->stream.launch_edge(h->d_tensors, v, sc, h->error_word, stream));
    if (fam[1]) AM_CUDA(h, cudaEventRecord(pev[2], stream));
    AM_CUDA(h, h->stream.launch_cluster(h->d_tensors, v, sc, h->error_word, stream));
    if (fam[2]) AM_CUDA(h, cudaEventRecord(pev[3], stream));
    if (h->piece_units) {
        twopass_partial_kernel<<<static_cast<unsigned>(h->piece_units), kThreads, 0, stream>>>(
            h->d_tensors, h->d_piece_segs, h->n_piece_segs, h->d_partials, sc.gscale, sc.gscale_dev, sc.skip_flag, sc.statistic);
        AM_CUDA(h, cudaGetLastError());
        const unsigned fin_grid = static_cast<unsigned>(ceil_div(h->block_units, kThreads / 32));
        twopass_finalize_kernel<<<fin_grid, kThreads, 0, stream>>>(
            h->d_tensors, h->d_block_segs, h->n_block_segs, h->block_units, h->d_partials,
            h->d_block_steps, v, sc);
        AM_CUDA(h, cudaGetLastError());
        if (h->wide_units) {
            twopass_finalize_wide_kernel<<<static_cast<unsigned>(h->wide_units), kThreads, 0, stream>>>(
                h->d_tensors, h->d_wide_segs, h->n_wide_segs, h->d_partials, h->d_block_steps, v, sc);
            AM_CUDA(h, cudaGetLastError());
        }
        twopass_update_kernel<<<static_cast<unsigned>(h->piece_units), kThreads, 0, stream>>>(
            h->d_tensors, h->d_piece_segs, h->n_piece_segs, h->d_block_steps, sc);
        AM_CUDA(h, cudaGetLastError());
    }
    if (fam[3]) AM_CUDA(h, cudaEventRecord(pev[4], stream));
    if (prof) ++h->prof_steps;
    return AM_OK;
}

int adammini_get_profile(am_handle *h, float *ms, int32_t *n_steps) {
    if (!h || !ms || h->opt[AM_OPT_PROFILE] == 0 || h->prof_steps == 0) return AM_ERR_INVALID_ARGUMENT;
    const int64_t ring = h->opt[AM_OPT_PROFILE];
    const int64_t n = std::min(h->prof_steps, ring);
    double sum[4] = {0.0, 0.0, 0.0, 0.0};
    bool fam[4];
    active_families(h, fam);
    int last = 0;                       // the last event a step records
    for (int k = 0; k < 4; ++k)
        if (fam[k]) last = k + 1;
    for (int64_t s = 0; s < n; ++s) {
        cudaEvent_t *ev = &h->prof_ev[s * 5];
        AM_CUDA(h, cudaEventSynchronize(ev[last]));
        int before = 0;                 // the event recorded before family k's launches
        for (int k = 0; k < 4; ++k) {
            if (!fam[k]) continue;      // (launches nothing: no time, no event)
            float x = 0.f;
            AM_CUDA(h, cudaEventElapsedTime(&x, ev[before], ev[k + 1]));
            sum[k] += x;
            before = k + 1;
        }
    }
    for (int k = 0; k < 4; ++k) ms[k] = static_cast<float>(sum[k] / static_cast<double>(n));
    if (n_steps) *n_steps = static_cast<int32_t>(n);
    return AM_OK;
}

int adammini_probe_ring_copy(am_handle *h, const void *src, void *dst, int64_t n_items, int32_t load_bytes,
                             int32_t store_bytes, void *cuda_stream) {
    if (!h || !h->planned || n_items < 0) return AM_ERR_INVALID_ARGUMENT;
    if (load_bytes < 0 || store_bytes < 0 || load_bytes > kProbeStageBytes || store_bytes > kProbeStageBytes ||
        load_bytes % 16 != 0 || store_bytes % 16 != 0 || (load_bytes == 0 && store_bytes == 0) ||
        (load_bytes > 0 && store_bytes > load_bytes))
        return AM_ERR_INVALID_ARGUMENT;
    if ((load_bytes > 0 && !src) || (store_bytes > 0 && !dst)) return AM_ERR_INVALID_ARGUMENT;
    if (!aligned16(src) || !aligned16(dst)) return AM_ERR_MISALIGNED;
    if (n_items > (int64_t(1) << 40) / kProbeStageBytes) return AM_ERR_TOO_LARGE;
    const int n_stages = h->caps.smem_optin > kCtrlBytes
                             ? std::min<int>(kMaxStages, static_cast<int>((h->caps.smem_optin - kCtrlBytes) / kProbeStageBytes)) : 0;
    if (n_stages < 2) return AM_ERR_TOO_LARGE;          // the device's shared memory does not hold a ring
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int dev = -1;
    AM_CUDA(h, cudaGetDevice(&dev));
    if (dev != h->device) return AM_ERR_INVALID_ARGUMENT;
    cudaStreamCaptureStatus capture = cudaStreamCaptureStatusNone;
    AM_CUDA(h, cudaStreamIsCapturing(stream, &capture));
    if (capture != cudaStreamCaptureStatusNone) return AM_ERR_INVALID_ARGUMENT;
    if (n_items == 0) return AM_OK;
    AM_CUDA(h, cudaMemsetAsync(h->d_probe_counter, 0, sizeof(unsigned long long), stream));
    const unsigned long long limit_ns =
        h->opt[AM_OPT_WAIT_LIMIT_US] ? static_cast<unsigned long long>(h->opt[AM_OPT_WAIT_LIMIT_US]) * 1000ull : kWaitTimeoutNs;
    const unsigned grid = static_cast<unsigned>(std::min<int64_t>(h->caps.sm_count, n_items));
    const size_t smem = kCtrlBytes + static_cast<size_t>(n_stages) * kProbeStageBytes;
    ring_copy_kernel<<<grid, kProbeThreads, smem, stream>>>(static_cast<const unsigned char *>(src), static_cast<unsigned char *>(dst),
                                                            n_items, load_bytes, store_bytes, n_stages, h->d_probe_counter,
                                                            h->error_word, limit_ns);
    AM_CUDA(h, cudaGetLastError());
    return AM_OK;
}

int adammini_part_sums(am_handle *h, const void *const *grads, double *out, void *cuda_stream) {
    if (!h || !h->planned || !grads) return AM_ERR_INVALID_ARGUMENT;
    if (h->n_parts == 0) return AM_OK;
    if (!out) return AM_ERR_INVALID_ARGUMENT;
    const int n = static_cast<int>(h->rows.size());
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int dev = -1;
    AM_CUDA(h, cudaGetDevice(&dev));
    if (dev != h->device) return AM_ERR_INVALID_ARGUMENT;
    // the kernels read the gradient addresses from the device tensor table: refresh those
    bool changed = !h->ptrs_valid;
    for (int i = 0; i < n; ++i) {
        if (h->rows[i].kind != AM_PART) continue;
        if (!grads[i]) return AM_ERR_INVALID_ARGUMENT;
        if (reinterpret_cast<uintptr_t>(grads[i]) & (h->rows[i].grad_dtype == AM_BF16 ? 1u : 3u)) return AM_ERR_MISALIGNED;
        if (h->host_tensors[i].g != grads[i]) {
            h->host_tensors[i].g = grads[i];
            changed = true;
        }
    }
    if (changed) {
        const int k = h->next_pinned;
        h->next_pinned ^= 1;
        if (h->ev_pending[k]) {
            AM_CUDA(h, cudaEventSynchronize(h->ev[k]));
            h->ev_pending[k] = false;
        }
        std::memcpy(h->pinned[k], h->host_tensors.data(), sizeof(DevTensor) * n);
        AM_CUDA(h, cudaMemcpyAsync(h->d_tensors, h->pinned[k], sizeof(DevTensor) * n, cudaMemcpyHostToDevice, stream));
        AM_CUDA(h, cudaEventRecord(h->ev[k], stream));
        h->ev_pending[k] = true;
        // the other addresses of the table may be stale: the next step uploads it again
        h->ptrs_valid = false;
    }
    twopass_partial_kernel<<<static_cast<unsigned>(h->part_units), kThreads, 0, stream>>>(
        h->d_tensors, h->d_part_segs, h->n_parts, h->d_partials, 1.f, nullptr, nullptr, 0);
    AM_CUDA(h, cudaGetLastError());
    part_sums_kernel<<<static_cast<unsigned>(ceil_div(h->n_parts, kThreads / 32)), kThreads, 0, stream>>>(
        h->d_tensors, h->d_part_tensors, h->n_parts, h->d_partials, out);
    AM_CUDA(h, cudaGetLastError());
    return AM_OK;
}

int adammini_sync_status(am_handle *h, void *cuda_stream) {
    if (!h) return AM_ERR_INVALID_ARGUMENT;
    AM_CUDA(h, cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)));
    if (h->error_word && *h->error_word != 0) {
        *h->error_word = 0;
        return AM_ERR_TIMEOUT;
    }
    return AM_OK;
}

int adammini_destroy(am_handle *h) {
    if (!h) return AM_OK;
    cudaDeviceSynchronize();
    host_step_release(h);
    release_plan(h);
    for (int k = 0; k < 2; ++k) {
        if (h->pinned[k]) cudaFreeHost(h->pinned[k]);
        if (h->ev[k]) cudaEventDestroy(h->ev[k]);
    }
    for (cudaEvent_t e : h->prof_ev)
        if (e) cudaEventDestroy(e);
    if (h->error_word) cudaFreeHost(h->error_word);
    delete h;
    return AM_OK;
}

}  // extern "C"

#include "host_step.inl"

// ---------------------------------------------------------------------------
// adammini_step_tensor_noalloc: the two-pass update of one tensor with its
// scratch in a fixed device array instead of allocated memory.
// ---------------------------------------------------------------------------
namespace {

constexpr int kNoAllocMaxDevices = 64;

// partial sums (double) first, per-block step sizes (float) after them
static __device__ __align__(256) unsigned char g_noalloc_scratch[AM_NOALLOC_SCRATCH_BYTES];

// Device address of the array on each device; the symbol itself is only a
// host-side handle and must never be handed to a kernel.  Atomic: host threads
// may make their first calls on a device at the same time (they all look up
// the same address).
std::atomic<void *> g_noalloc_addr[kNoAllocMaxDevices] = {};

__device__ __forceinline__ PieceRef noalloc_piece(const DevTensor &t, int64_t local, bool vec) {
    PieceRef r;
    r.t = &t;
    r.local = local;
    r.block = local / t.pieces_per_block;
    const int64_t off = (local - r.block * t.pieces_per_block) * t.piece_len;
    r.start = r.block * t.L + off;
    const int64_t left = t.L - off;
    r.n = left < t.piece_len ? left : t.piece_len;
    r.vec = vec;
    return r;
}

__global__ void __launch_bounds__(kThreads)
noalloc_partial_kernel(const __grid_constant__ DevTensor t, int vec, double *__restrict__ partials) {
    __shared__ double warp_part[kThreads / 32];
    const PieceRef r = noalloc_piece(t, blockIdx.x, vec != 0);
    const double w = warp_sum(t.gdtype == AM_BF16 ? piece_sum_sq<AM_BF16>(r, 1.f) : piece_sum_sq<AM_F32>(r, 1.f));
    if ((threadIdx.x & 31) == 0) warp_part[threadIdx.x >> 5] = w;
    __syncthreads();
    if (threadIdx.x == 0) {
        double s = 0.0;
#pragma unroll
        for (int k = 0; k < kThreads / 32; ++k) s += warp_part[k];
        partials[r.local] = s;
    }
}

__global__ void __launch_bounds__(kThreads)
noalloc_finalize_kernel(const __grid_constant__ DevTensor t, const double *__restrict__ partials,
                        float *__restrict__ block_steps, float *__restrict__ v, StepScalars sc) {
    const int64_t b = static_cast<int64_t>(blockIdx.x) * (kThreads / 32) + (threadIdx.x >> 5);
    if (b >= t.n_blocks) return;
    const int lane = threadIdx.x & 31;
    const double *src = partials + b * t.pieces_per_block;
    double s = 0.0;
    for (int64_t j = lane; j < t.pieces_per_block; j += 32) s += src[j];
    s = warp_sum(s);
    if (lane == 0) {
        float vn;
        const float st = block_step(s, static_cast<double>(t.L), v[b], sc, &vn);
        v[b] = vn;
        block_steps[b] = st;
    }
}

__global__ void __launch_bounds__(kThreads)
noalloc_update_kernel(const __grid_constant__ DevTensor t, int vec, const float *__restrict__ block_steps,
                      StepScalars sc) {
    const PieceRef r = noalloc_piece(t, blockIdx.x, vec != 0);
    if (t.gdtype == AM_BF16) twopass_update_body<AM_BF16>(r, block_steps, sc);
    else twopass_update_body<AM_F32>(r, block_steps, sc);
}

}  // namespace

extern "C" int adammini_step_tensor_noalloc(void *param, const void *grad, void *m, float *v, int64_t numel,
                                            int64_t block_len, int32_t grad_dtype, int32_t apply_weight_decay,
                                            const am_hparams *hp, int64_t step, void *cuda_stream) {
    if (!param || !grad || !m || !v || step < 1 || numel < 0) return AM_ERR_INVALID_ARGUMENT;
    if (grad_dtype != AM_F32 && grad_dtype != AM_BF16) return AM_ERR_INVALID_ARGUMENT;
    const int rc = validate_hparams(hp);
    if (rc != AM_OK) return rc;
    if (block_len <= 0 || numel % block_len != 0) return AM_ERR_SHAPE;
    if (!aligned16(param) || !aligned16(grad) || !aligned16(m) || !aligned16(v)) return AM_ERR_MISALIGNED;
    if (numel == 0) return AM_OK;

    DevTensor t{};
    t.g = grad;
    t.m = static_cast<float *>(m);
    t.p = static_cast<float *>(param);
    t.numel = numel;
    t.L = block_len;
    t.n_blocks = numel / block_len;
    t.v_offset = 0;
    t.gdtype = grad_dtype;
    t.wd = apply_weight_decay ? 1 : 0;
    t.piece_len = block_len;
    t.pieces_per_block = 1;
    if (block_len > kPieceMax) {
        int64_t ppb = std::min<int64_t>(ceil_div(block_len, kPieceMax), kMaxPiecesPerBlock);
        t.piece_len = ceil_div(ceil_div(block_len, ppb), 1024) * 1024;
        t.pieces_per_block = ceil_div(block_len, t.piece_len);
    }
    t.piece_base = 0;
    t.block_base = 0;      // block_steps is indexed by block inside the array
    t.mean_len = block_len;
    t.part_index = -1;
    if (t.n_blocks > AM_NOALLOC_MAX_BLOCKS) return AM_ERR_TOO_LARGE;
    const int64_t pieces = t.n_blocks * t.pieces_per_block;
    if (pieces > AM_NOALLOC_MAX_PIECES) return AM_ERR_TOO_LARGE;

    // set-up, once per device: the device address of the static array
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= kNoAllocMaxDevices) return AM_ERR_CUDA;
    void *scratch = g_noalloc_addr[dev].load(std::memory_order_acquire);
    if (!scratch) {
        e = cudaGetSymbolAddress(&scratch, g_noalloc_scratch);
        if (e != cudaSuccess || !scratch) return AM_ERR_CUDA;
        g_noalloc_addr[dev].store(scratch, std::memory_order_release);
    }
    double *partials = static_cast<double *>(scratch);
    float *block_steps = reinterpret_cast<float *>(static_cast<unsigned char *>(scratch) +
                                                   AM_NOALLOC_MAX_PIECES * sizeof(double));

    const double bc1 = 1.0 - std::pow(hp->beta1, static_cast<double>(step));
    const double bc2 = 1.0 - std::pow(hp->beta2, static_cast<double>(step));
    StepScalars sc;
    sc.beta2 = hp->beta2;
    sc.omb2 = 1.0 - hp->beta2;
    sc.inv_bc2 = 1.0 / bc2;
    sc.lr_over_bc1 = hp->lr / bc1;
    sc.eps = hp->eps;
    sc.beta1 = static_cast<float>(hp->beta1);
    sc.omb1 = static_cast<float>(1.0 - hp->beta1);
    sc.lr_wd = static_cast<float>(hp->lr * hp->weight_decay);
    sc.gscale = 1.f;
    sc.gscale_dev = nullptr;
    sc.skip_flag = nullptr;
    sc.statistic = 0;
    sc.pad = 0;
    sc.part_sums = nullptr;

    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int vec = 1;      // every array starts 16-byte aligned (checked above): 16-byte accesses wherever the element index allows
    noalloc_partial_kernel<<<static_cast<unsigned>(pieces), kThreads, 0, stream>>>(t, vec, partials);
    if (cudaGetLastError() != cudaSuccess) return AM_ERR_CUDA;
    noalloc_finalize_kernel<<<static_cast<unsigned>(ceil_div(t.n_blocks, kThreads / 32)), kThreads, 0, stream>>>(
        t, partials, block_steps, v, sc);
    if (cudaGetLastError() != cudaSuccess) return AM_ERR_CUDA;
    noalloc_update_kernel<<<static_cast<unsigned>(pieces), kThreads, 0, stream>>>(t, vec, block_steps, sc);
    if (cudaGetLastError() != cudaSuccess) return AM_ERR_CUDA;
    return AM_OK;
}
