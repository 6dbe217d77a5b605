// adammini_step_host: the step for optimizer state that lives in host memory.
// (placeholder until the staging pipeline is written)
struct HostStepState {};

void host_step_release(am_handle *h) {
    delete h->host_step;
    h->host_step = nullptr;
}

extern "C" int adammini_step_host(am_handle *h, void *const *params, const void *const *grads, void *const *m,
                                  float *v, int64_t step, int64_t staging_bytes) {
    (void)h; (void)params; (void)grads; (void)m; (void)v; (void)step; (void)staging_bytes;
    return AM_ERR_INVALID_ARGUMENT;
}
