/*
 * Adam-mini oracle -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, single-threaded float64 transcription of the Adam-mini
 * update (paper: Algorithm 1 "Adam-mini (General form)", restated as
 * "Adam-mini in Pytorch style" in the appendix, and the boxed v_b rule of the
 * introduction).  It exists so that tests and the benchmark's CPU baseline
 * have something obviously correct to compare the CUDA library with.  It
 * shares no code, header, table or constant with the CUDA library and must
 * never be linked into, imported by, or called from the product path.
 *
 * Only tests/, the smoke check and the benchmark's cpu_baseline / reference
 * legs may load this file's shared object.
 *
 * Conventions (each is a reading of the paper where it is silent):
 *   - one tensor per call; the tensor is n_blocks * L contiguous elements and
 *     block b is elements [b*L, (b+1)*L)  (Algorithm 3: param[i] views);
 *   - t is 1-based (the bias corrections 1 - beta^t must not vanish);
 *   - state p, m (per element) and v (per block) are kept in float64 by the
 *     caller across steps; m and v start at zero;
 *   - gradients arrive with the bits the GPU sees (float32 or bfloat16) and
 *     are widened exactly;
 *   - "mean" is the arithmetic mean, summed left to right in float64;
 *   - epsilon is added to sqrt(v_hat), outside the root (Algorithm 1, last
 *     line of the loop body);
 *   - the decoupled decay acts on the old parameter first, then the Adam
 *     term is subtracted (order of the loop body of Algorithm 1).
 *
 * Build: gcc -O2 -ffp-contract=off -fno-fast-math -shared -fPIC (see build.py).
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

enum { ORACLE_G_F32 = 0, ORACLE_G_BF16 = 1, ORACLE_G_F64 = 2 };

static double widen_bf16(uint16_t h)
{
    /* bfloat16 is the upper half of an IEEE float32 */
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

static double grad_at(const void *g, int g_dtype, int64_t i)
{
    switch (g_dtype) {
    case ORACLE_G_F32:  return (double)((const float *)g)[i];
    case ORACLE_G_BF16: return widen_bf16(((const uint16_t *)g)[i]);
    default:            return ((const double *)g)[i];
    }
}

/*
 * One Adam-mini step on one tensor (Algorithm 1, loop body, for every block).
 *   p, m : float64[numel]   updated in place
 *   v    : float64[numel/L] updated in place (one scalar per block)
 *   g    : numel gradients of type g_dtype, read only
 *   apply_wd : 0 skips the decay line for this tensor
 * Returns 0, or -1 on an invalid argument.
 */
int oracle_adammini_step(double *p, double *m, double *v, const void *g,
                         int g_dtype, int64_t numel, int64_t L, double lr,
                         double beta1, double beta2, double eps, double wd,
                         int apply_wd, int64_t t)
{
    if (!p || !m || !v || !g || numel < 0 || L <= 0 || numel % L != 0 || t < 1)
        return -1;
    const double bc1 = 1.0 - pow(beta1, (double)t);   /* 1 - beta1^t */
    const double bc2 = 1.0 - pow(beta2, (double)t);   /* 1 - beta2^t */
    const int64_t n_blocks = numel / L;

    for (int64_t b = 0; b < n_blocks; ++b) {
        const int64_t lo = b * L;

        /* v = (1-beta2) * mean(g*g) + beta2 * v      (boxed rule; Alg. 1) */
        double sum_sq = 0.0;
        for (int64_t i = 0; i < L; ++i) {
            const double gi = grad_at(g, g_dtype, lo + i);
            sum_sq = sum_sq + gi * gi;
        }
        const double mean_sq = sum_sq / (double)L;
        v[b] = (1.0 - beta2) * mean_sq + beta2 * v[b];
        const double v_hat = v[b] / bc2;               /* v / (1-beta2^t)  */
        const double denom = sqrt(v_hat) + eps;

        for (int64_t i = 0; i < L; ++i) {
            const int64_t k = lo + i;
            const double gi = grad_at(g, g_dtype, k);
            if (apply_wd)
                p[k] = p[k] - lr * wd * p[k];          /* decoupled decay  */
            m[k] = (1.0 - beta1) * gi + beta1 * m[k];  /* first moment     */
            const double m_hat = m[k] / bc1;           /* m / (1-beta1^t)  */
            p[k] = p[k] - lr * m_hat / denom;          /* parameter update */
        }
    }
    return 0;
}

/*
 * The paper's ablation of the block statistic (appendix "Ablation Studies on
 * the Design of Adam-mini"): instead of the mean of g*g the block's learning
 * rate is built from the max, the min, the 1-norm or the 2-norm.  The paper
 * names the quantities only; the reading taken here is that the statistic of
 * the vector g_b*g_b replaces mean(g_b*g_b) in the v rule, so that v stays
 * one scalar per block:
 *   statistic 0: mean(g*g)   1: max(g*g)   2: min(g*g)
 *   statistic 3: sum(g*g)    (1-norm of a non-negative vector)
 *   statistic 4: sqrt(sum((g*g)^2))   (2-norm)
 * Everything else is Algorithm 1 as above.
 */
int oracle_adammini_step_stat(double *p, double *m, double *v, const void *g,
                              int g_dtype, int64_t numel, int64_t L, double lr,
                              double beta1, double beta2, double eps, double wd,
                              int apply_wd, int64_t t, int statistic)
{
    if (!p || !m || !v || !g || numel < 0 || L <= 0 || numel % L != 0 || t < 1 ||
        statistic < 0 || statistic > 4)
        return -1;
    const double bc1 = 1.0 - pow(beta1, (double)t);
    const double bc2 = 1.0 - pow(beta2, (double)t);
    const int64_t n_blocks = numel / L;

    for (int64_t b = 0; b < n_blocks; ++b) {
        const int64_t lo = b * L;
        double acc = 0.0;
        for (int64_t i = 0; i < L; ++i) {
            const double gi = grad_at(g, g_dtype, lo + i);
            const double sq = gi * gi;
            if (statistic == 0 || statistic == 3) acc = acc + sq;
            else if (statistic == 1) acc = (i == 0 || sq > acc) ? sq : acc;
            else if (statistic == 2) acc = (i == 0 || sq < acc) ? sq : acc;
            else acc = acc + sq * sq;
        }
        double stat = acc;
        if (statistic == 0) stat = acc / (double)L;
        if (statistic == 4) stat = sqrt(acc);
        v[b] = (1.0 - beta2) * stat + beta2 * v[b];
        const double v_hat = v[b] / bc2;
        const double denom = sqrt(v_hat) + eps;

        for (int64_t i = 0; i < L; ++i) {
            const int64_t k = lo + i;
            const double gi = grad_at(g, g_dtype, k);
            if (apply_wd)
                p[k] = p[k] - lr * wd * p[k];
            m[k] = (1.0 - beta1) * gi + beta1 * m[k];
            const double m_hat = m[k] / bc1;
            p[k] = p[k] - lr * m_hat / denom;
        }
    }
    return 0;
}

/* Exact widening helpers so Python callers can build float64 state from the
 * bits handed to the GPU without going through another library. */
void oracle_widen_f32(const float *src, double *dst, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) dst[i] = (double)src[i];
}

void oracle_widen_bf16(const uint16_t *src, double *dst, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) dst[i] = widen_bf16(src[i]);
}
