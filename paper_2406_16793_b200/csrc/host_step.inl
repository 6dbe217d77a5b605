// adammini_step_host: the step for optimizer state that lives in host memory
// (offloaded parameters, moments and gradients).  Consecutive tensors are
// grouped so that a group's p, m, g and its slice of v fit one device staging
// slot; groups rotate over three slots, each with its own stream, so that the
// host->device copies of one group, the kernels of the previous one and the
// device->host copies of the one before overlap.  The update itself is the
// same kernels adammini_step launches: every group owns a handle planned for
// its staging addresses.
// (included at the end of adammini.cu)

namespace {

constexpr int kHostSlots = 3;
constexpr size_t kHostDefaultStaging = size_t(3) << 30;   // 1 GiB per slot unless a tensor needs more

struct HostGroup {
    int first = 0, count = 0;
    int64_t v_begin = 0, v_count = 0;
    am_handle *sub = nullptr;
    std::vector<void *> d_p, d_m;
    std::vector<const void *> d_g;
    float *d_v = nullptr;
};

inline size_t tensor_staging_bytes(const am_table_row &r) {
    const size_t gsz = r.grad_dtype == AM_BF16 ? 2 : 4;
    return round_up(r.numel * 4, 256) * 2 + round_up(r.numel * gsz, 256) + round_up(r.n_blocks * 4, 256);
}

}  // namespace

struct HostStepState {
    size_t slot_bytes = 0;
    bool ready = false;          // every group has its handle
    void *slots[kHostSlots] = {nullptr, nullptr, nullptr};
    cudaStream_t streams[kHostSlots] = {nullptr, nullptr, nullptr};
    std::vector<HostGroup> groups;
};

void host_step_release(am_handle *h) {
    HostStepState *s = h->host_step;
    if (!s) return;
    for (HostGroup &g : s->groups)
        if (g.sub) adammini_destroy(g.sub);
    for (int k = 0; k < kHostSlots; ++k) {
        if (s->slots[k]) cudaFree(s->slots[k]);
        if (s->streams[k]) cudaStreamDestroy(s->streams[k]);
    }
    delete s;
    h->host_step = nullptr;
}

namespace {

int host_step_prepare(am_handle *h, int64_t staging_bytes) {
    const int n = static_cast<int>(h->rows.size());
    size_t largest = 0;
    for (const am_table_row &r : h->rows) largest = std::max(largest, tensor_staging_bytes(r));
    const size_t budget = staging_bytes > 0 ? static_cast<size_t>(staging_bytes) : kHostDefaultStaging;
    const size_t slot_bytes = std::max(budget / kHostSlots, largest);
    if (h->host_step && h->host_step->ready && h->host_step->slot_bytes == slot_bytes) return AM_OK;
    host_step_release(h);

    HostStepState *s = new (std::nothrow) HostStepState();
    if (!s) return AM_ERR_ALLOC;
    h->host_step = s;
    s->slot_bytes = slot_bytes;
    for (int k = 0; k < kHostSlots; ++k) {
        AM_CUDA(h, cudaMalloc(&s->slots[k], slot_bytes));
        AM_CUDA(h, cudaStreamCreateWithFlags(&s->streams[k], cudaStreamNonBlocking));
    }
    // consecutive tensors -> groups that fit a slot
    int i = 0;
    while (i < n) {
        HostGroup g;
        g.first = i;
        g.v_begin = h->rows[i].v_offset;
        size_t used = 0;
        while (i < n && used + tensor_staging_bytes(h->rows[i]) <= slot_bytes) {
            used += tensor_staging_bytes(h->rows[i]);
            g.v_count += h->rows[i].n_blocks;
            ++i;
        }
        g.count = i - g.first;
        s->groups.push_back(g);
    }
    // a handle per group, planned for the group's staging addresses
    for (size_t gi = 0; gi < s->groups.size(); ++gi) {
        HostGroup &g = s->groups[gi];
        am_partition part;
        char *base = static_cast<char *>(s->slots[gi % kHostSlots]);
        size_t off = round_up(g.v_count * 4, 256);
        g.d_v = reinterpret_cast<float *>(base);
        for (int k = 0; k < g.count; ++k) {
            am_table_row r = h->rows[g.first + k];
            r.v_offset -= g.v_begin;
            part.rows.push_back(r);
            const size_t gsz = r.grad_dtype == AM_BF16 ? 2 : 4;
            g.d_p.push_back(base + off); off += round_up(r.numel * 4, 256);
            g.d_m.push_back(base + off); off += round_up(r.numel * 4, 256);
            g.d_g.push_back(base + off); off += round_up(r.numel * gsz, 256);
        }
        part.total_blocks = g.v_count;
        const int rc = adammini_create(&part, &h->hp, &g.sub);
        if (rc != AM_OK) return rc;
        for (int key = 0; key < kNumOptions; ++key)
            if (key != AM_OPT_PROFILE && h->opt[key]) adammini_set_option(g.sub, key, h->opt[key]);
        // The order in which a long block's partial sums are added depends on the cluster size, and
        // the automatic choice looks at all tensors of a table: give the group the size this handle
        // resolved, so that the staged step returns the bits adammini_step returns.
        if (h->stream.clus.active() && h->opt[AM_OPT_CLUSTER_SIZE] == 0) {
            const int rc2 = adammini_set_option(g.sub, AM_OPT_CLUSTER_SIZE, h->stream.clus.cluster);
            if (rc2 != AM_OK) return rc2;
        }
    }
    s->ready = true;
    return AM_OK;
}

}  // namespace

extern "C" int adammini_step_host(am_handle *h, void *const *params, const void *const *grads, void *const *m,
                                  float *v, int64_t step, int64_t staging_bytes) {
    if (!h || !h->planned || step < 1 || staging_bytes < 0) return AM_ERR_INVALID_ARGUMENT;
    const int n = static_cast<int>(h->rows.size());
    if (n == 0) return AM_OK;
    if (h->n_parts > 0) return AM_ERR_INVALID_ARGUMENT;     // parts of blocks need the exchange of their sums
    if (!params || !grads || !m || !v) return AM_ERR_INVALID_ARGUMENT;
    for (int i = 0; i < n; ++i)
        if (!params[i] || !grads[i] || !m[i]) return AM_ERR_INVALID_ARGUMENT;
    int dev = -1;
    AM_CUDA(h, cudaGetDevice(&dev));
    if (dev != h->device) return AM_ERR_INVALID_ARGUMENT;
    int rc;
    try {
        rc = host_step_prepare(h, staging_bytes);      // (its tables grow by push_back)
    } catch (...) {
        rc = AM_ERR_ALLOC;
    }
    if (rc != AM_OK) {
        host_step_release(h);                           // a half-built pipeline is not kept
        return rc;
    }
    HostStepState *s = h->host_step;

    // One exit: whatever fails, the copies already enqueued still read and write the caller's
    // buffers, so the loop is left through the synchronisation of all three streams below.
    int result = AM_OK;
    auto copy = [&](void *dst, const void *src, size_t bytes, cudaMemcpyKind kind, cudaStream_t st) {
        if (result != AM_OK) return;
        const cudaError_t e = cudaMemcpyAsync(dst, src, bytes, kind, st);
        if (e != cudaSuccess) result = cuda_fail(h, e);
    };
    for (size_t gi = 0; gi < s->groups.size() && result == AM_OK; ++gi) {
        HostGroup &g = s->groups[gi];
        cudaStream_t st = s->streams[gi % kHostSlots];
        g.sub->hp = h->hp;
        copy(g.d_v, v + g.v_begin, g.v_count * 4, cudaMemcpyHostToDevice, st);
        for (int k = 0; k < g.count; ++k) {
            const am_table_row &r = h->rows[g.first + k];
            const size_t gsz = r.grad_dtype == AM_BF16 ? 2 : 4;
            copy(const_cast<void *>(g.d_g[k]), grads[g.first + k], r.numel * gsz, cudaMemcpyHostToDevice, st);
            copy(g.d_m[k], m[g.first + k], r.numel * 4, cudaMemcpyHostToDevice, st);
            copy(g.d_p[k], params[g.first + k], r.numel * 4, cudaMemcpyHostToDevice, st);
        }
        if (result != AM_OK) break;
        result = adammini_step(g.sub, g.d_p.data(), g.d_g.data(), g.d_m.data(), g.d_v, step, st);
        if (result != AM_OK) {
            h->last_cuda_error = g.sub->last_cuda_error;
            break;
        }
        for (int k = 0; k < g.count; ++k) {
            const am_table_row &r = h->rows[g.first + k];
            copy(m[g.first + k], g.d_m[k], r.numel * 4, cudaMemcpyDeviceToHost, st);
            copy(params[g.first + k], g.d_p[k], r.numel * 4, cudaMemcpyDeviceToHost, st);
        }
        copy(v + g.v_begin, g.d_v, g.v_count * 4, cudaMemcpyDeviceToHost, st);
    }
    for (int k = 0; k < kHostSlots; ++k) {
        const cudaError_t e = cudaStreamSynchronize(s->streams[k]);
        if (e != cudaSuccess && result == AM_OK) result = cuda_fail(h, e);
    }
    if (result == AM_OK)
        for (HostGroup &g : s->groups)
            if (g.sub->error_word && *g.sub->error_word != 0) {
                *g.sub->error_word = 0;
                result = AM_ERR_TIMEOUT;
            }
    return result;
}
