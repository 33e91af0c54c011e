/*
 * dd_cpu_parallel.c -- the oracle's element loop of the direct-averaging merge split
 * over all host cores with OpenMP.  TEST / BENCHMARK INFRASTRUCTURE ONLY: it exists to
 * report what a CPU syncer (the paper runs its syncer on CPU hosts, Section 4) achieves
 * on the benchmark machine.  It is NOT the checked oracle (that is dd_oracle.c, single
 * thread) and nothing is ever compared against it except in its own consistency test.
 * Participation and weights are taken from the caller (computed by the oracle).
 */
#include <stddef.h>
#include <stdint.h>
#include <string.h>

static double learner_value(const void *base, int is_bf16, size_t i)
{
    if (is_bf16) {
        uint32_t bits = (uint32_t)((const uint16_t *)base)[i] << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
    return (double)((const float *)base)[i];
}

/* Theta, v in place; learners[j], w_hat[j] for the s participants in order.  Returns ||Delta||^2. */
double ddp_merge_fragment(float *Theta, float *v, const void *const *learners, const double *w_hat,
                          int s, int learner_is_bf16, float eta, float mu, int nesterov, size_t n)
{
    const double eta_d = (double)eta, mu_d = (double)mu;
    double delta_sq = 0.0;
    long long i;
#pragma omp parallel for schedule(static) reduction(+ : delta_sq)
    for (i = 0; i < (long long)n; ++i) {
        double T = (double)Theta[i], d = 0.0, vn, u;
        int j;
        for (j = 0; j < s; ++j) d += w_hat[j] * (T - learner_value(learners[j], learner_is_bf16, (size_t)i));
        vn = mu_d * (double)v[i] + d;
        u = nesterov ? d + mu_d * vn : vn;
        v[i] = (float)vn;
        Theta[i] = (float)(T - eta_d * u);
        delta_sq += d * d;
    }
    return delta_sq;
}
