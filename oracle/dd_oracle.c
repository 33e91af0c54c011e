/*
 * dd_oracle.c -- CPU oracle for the Decoupled DiLoCo syncer's per-fragment merge.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, single-threaded
 * statement of what the merge computes, written from the paper's definitions in
 * fp64.  It shares no code, header, table or helper with the CUDA library and
 * must never be reached from the product path: only the test-suite, the smoke
 * check and the benchmark's cpu_baseline / reference legs may build or call it.
 *
 * What it follows:
 *   participation ........ Algorithm 2 step 1 ("at least K" reports; the set M_t),
 *                          Section 3.2; absent learner == weight 0, Section 4
 *                          ("Syncer worker").
 *   weights .............. the Weight display in Section 3.2:
 *                          w = c_tokens * (c_tokens / c_steps).
 *   merge ................ "Direct averaging", weighted form, Appendix
 *                          "Merging methods": sum_m w_m (Theta - theta_m) / sum_m w_m.
 *   radial-directional ... "Radial-directional averaging", same appendix.
 *   outer step ........... Eq. 1 / Eq. 2 + Section 2: OuterOpt is SGD with Nesterov
 *                          momentum; plain averaging is SGD with learning rate 1.
 *   grace window ......... "Adaptive Quorum Window", Section 3.2 (slack equation).
 *
 * Parity pins (tests/test_oracle_*.py): plain mean with equal tokens; mu=0, lr=1
 * gives the token-weighted mean; masked / zero-token learners have no effect;
 * permutation invariance; the two-merge momentum recurrence in closed form;
 * torch.optim.SGD(nesterov=True) as an independent third implementation; brute
 * force over all masks for the participant set; E||Delta||^2 = n sigma^2 sum w^2.
 *
 * Parity unpinned BY THE PAPER (pinned only to library semantics): the exact
 * Nesterov formulation and the values of the outer learning rate / momentum --
 * the paper names the optimizer but prints neither its update rule nor its
 * hyper-parameters.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

#define DDO_MAX_LEARNERS 64

enum {
    DDO_STATUS_OK = 0,
    DDO_STATUS_QUORUM_NOT_MET = 1,
    DDO_STATUS_ZERO_WEIGHT = 2,
    DDO_INVALID = -1
};

enum { DDO_MERGE_AVG = 0, DDO_MERGE_RDA = 1 };

typedef struct {
    int32_t status;
    int32_t n_part;
    uint8_t idx[DDO_MAX_LEARNERS];        /* ascending learner ids            */
    double  w_hat[DDO_MAX_LEARNERS];      /* normalised weights, idx order    */
    double  w_total;                      /* sum of raw weights               */
    double  delta_sq;                     /* ||Delta||^2 of the merged update */
    double  theta_sq;                     /* ||Theta'||^2                     */
    double  mom_sq;                       /* ||v'||^2                         */
    double  delta_m_sq[DDO_MAX_LEARNERS]; /* ||Theta - theta_m||^2, idx order */
} ddo_record;

/* ---- bf16 <-> fp32 ------------------------------------------------------- */

/* bf16 is the upper half of an IEEE binary32, so widening is exact. */
float ddo_bf16_to_f32(uint16_t h)
{
    uint32_t bits = (uint32_t)h << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return f;
}

/* Round-to-nearest, ties-to-even, from binary32 to its upper 16 bits. */
uint16_t ddo_bf16_rne(float x)
{
    uint32_t bits;
    memcpy(&bits, &x, sizeof bits);
    if ((bits & 0x7fffffffu) > 0x7f800000u)          /* NaN: keep sign, make quiet */
        return (uint16_t)((bits >> 16) | 0x0040u);
    {
        uint32_t upper = bits >> 16;
        uint32_t lower = bits & 0xffffu;
        if (lower > 0x8000u || (lower == 0x8000u && (upper & 1u)))
            upper += 1u;                             /* carry may reach Inf: correct */
        return (uint16_t)upper;
    }
}

/* Array form of ddo_bf16_rne. */
void ddo_bf16_rne_array(const float *x, uint16_t *out, size_t n)
{
    size_t i;
    for (i = 0; i < n; ++i) out[i] = ddo_bf16_rne(x[i]);
}

/* ---- participation (Algorithm 2 step 1; Section 4: absent == weight 0) ---- */

/*
 * S = { m < M : mask bit m set and tokens[m] > 0 }, listed ascending.
 * The quorum is met when |S| >= max(K, 1).
 */
int ddo_participants(uint64_t mask, const uint64_t *tokens, int M, int K,
                     uint8_t *idx, int32_t *n_part)
{
    int m, s = 0;
    if (M < 1 || M > DDO_MAX_LEARNERS || K < 0 || K > M) return DDO_INVALID;
    for (m = 0; m < M; ++m) {
        int reported = (int)((mask >> m) & 1u);
        if (reported && tokens[m] > 0) idx[s++] = (uint8_t)m;
    }
    *n_part = s;
    return s >= (K > 1 ? K : 1) ? DDO_STATUS_OK : DDO_STATUS_QUORUM_NOT_MET;
}

/* ---- weights (the Weight display, Section 3.2) ----------------------------- */

/*
 * w_m = tokens_m * (tokens_m / steps_m); when no step counters are supplied the
 * weight is the token count itself (the two agree up to a common factor when
 * every learner uses the same tokens per step, and common factors cancel).
 * w_hat_m = w_m / sum_{m in S} w_m.
 */
int ddo_weights(const uint64_t *tokens, const uint64_t *steps, const uint8_t *idx,
                int s, double *w_hat, double *w_total)
{
    double w[DDO_MAX_LEARNERS];
    double W = 0.0;
    int j;
    if (steps == NULL) {
        uint64_t Wi = 0;
        for (j = 0; j < s; ++j) {
            w[j] = (double)tokens[idx[j]];
            if (Wi + tokens[idx[j]] < Wi) return DDO_INVALID;   /* the exact 64-bit sum would wrap */
            Wi += tokens[idx[j]];
        }
        W = (double)Wi;
    } else {
        for (j = 0; j < s; ++j) {
            double t = (double)tokens[idx[j]];
            if (steps[idx[j]] == 0) return DDO_INVALID;   /* tokens > 0 but no step */
            w[j] = t * t / (double)steps[idx[j]];
            W += w[j];
        }
    }
    *w_total = W;
    if (!(W > 0.0)) return DDO_STATUS_ZERO_WEIGHT;
    for (j = 0; j < s; ++j) w_hat[j] = w[j] / W;
    return DDO_STATUS_OK;
}

/* ---- element access -------------------------------------------------------- */

static double learner_at(const void *base, int is_bf16, size_t i)
{
    if (is_bf16) return (double)ddo_bf16_to_f32(((const uint16_t *)base)[i]);
    return (double)((const float *)base)[i];
}

/* ---- the merge + outer step ------------------------------------------------ */

/*
 * One syncer update of one fragment (Algorithm 2 steps 2-3), in place on
 * Theta and v.  merge_kind selects direct averaging or radial-directional
 * averaging for Delta; the outer step is the same for both:
 *     v'     = mu v + Delta
 *     Theta' = Theta - eta (Delta + mu v')      (Nesterov)
 *     Theta' = Theta - eta v'                   (heavy ball, nesterov == 0)
 * Nothing is written when the quorum is not met or the weights sum to zero.
 * Returns DDO_INVALID for malformed arguments, else 0 (see rec->status).
 */
int ddo_merge_fragment(float *Theta, float *v, const void *const *learners, int M,
                       int learner_is_bf16, const uint64_t *tokens,
                       const uint64_t *steps, uint64_t mask, int K, float eta,
                       float mu, int nesterov, int merge_kind, size_t n,
                       uint16_t *out_bf16, ddo_record *rec)
{
    double w_hat[DDO_MAX_LEARNERS];
    double dir_coef[DDO_MAX_LEARNERS];
    double radial = 0.0, rda_scale = 1.0;
    const double eta_d = (double)eta, mu_d = (double)mu;
    size_t i;
    int j, s, st;

    memset(rec, 0, sizeof *rec);
    st = ddo_participants(mask, tokens, M, K, rec->idx, &rec->n_part);
    if (st == DDO_INVALID) return DDO_INVALID;
    s = rec->n_part;
    if (st != DDO_STATUS_OK) { rec->status = st; return 0; }
    st = ddo_weights(tokens, steps, rec->idx, s, w_hat, &rec->w_total);
    if (st == DDO_INVALID) return DDO_INVALID;
    if (st != DDO_STATUS_OK) { rec->status = st; return 0; }
    for (j = 0; j < s; ++j) {
        rec->w_hat[j] = w_hat[j];
        if (learners[rec->idx[j]] == NULL) return DDO_INVALID;
    }

    /* Per-participant outer-gradient norms ||Theta - theta_m||^2. */
    for (j = 0; j < s; ++j) {
        const void *th = learners[rec->idx[j]];
        double acc = 0.0;
        for (i = 0; i < n; ++i) {
            double d = (double)Theta[i] - learner_at(th, learner_is_bf16, i);
            acc += d * d;
        }
        rec->delta_m_sq[j] = acc;
    }

    if (merge_kind == DDO_MERGE_RDA) {
        /*
         * RDA({v_m, w_m}) = (sum w_m ||v_m|| / sum w_m) * phi(sum w_m phi(v_m) / sum w_m),
         * phi(x) = x / ||x||.  The printed weighted display shows a vector in
         * the first factor; by analogy with the unweighted
         * definition it is read as the weighted mean of the NORMS.  phi is
         * undefined at 0: a participant whose outer gradient is exactly zero
         * contributes its (zero) norm to the radial mean and nothing to the
         * direction; if the mean direction vanishes, Delta = 0.
         */
        double dir_sq = 0.0;
        for (j = 0; j < s; ++j) {
            double nm = sqrt(rec->delta_m_sq[j]);
            radial += w_hat[j] * nm;
            dir_coef[j] = nm > 0.0 ? w_hat[j] / nm : 0.0;
        }
        for (i = 0; i < n; ++i) {
            double T = (double)Theta[i], u = 0.0;
            for (j = 0; j < s; ++j)
                u += dir_coef[j] * (T - learner_at(learners[rec->idx[j]], learner_is_bf16, i));
            dir_sq += u * u;
        }
        rda_scale = dir_sq > 0.0 ? radial / sqrt(dir_sq) : 0.0;
    }

    for (i = 0; i < n; ++i) {
        double T = (double)Theta[i];
        double d = 0.0, vn, u, Tn;
        if (merge_kind == DDO_MERGE_RDA) {
            for (j = 0; j < s; ++j)
                d += dir_coef[j] * (T - learner_at(learners[rec->idx[j]], learner_is_bf16, i));
            d *= rda_scale;
        } else {
            for (j = 0; j < s; ++j)
                d += w_hat[j] * (T - learner_at(learners[rec->idx[j]], learner_is_bf16, i));
        }
        vn = mu_d * (double)v[i] + d;
        u = nesterov ? d + mu_d * vn : vn;
        Tn = T - eta_d * u;
        v[i] = (float)vn;
        Theta[i] = (float)Tn;
        if (out_bf16 != NULL) out_bf16[i] = ddo_bf16_rne((float)Tn);
        rec->delta_sq += d * d;
        rec->theta_sq += (double)Theta[i] * (double)Theta[i];   /* norms of the stored state */
        rec->mom_sq += (double)v[i] * (double)v[i];
    }
    rec->status = DDO_STATUS_OK;
    return 0;
}

/*
 * Radial-directional averaging of a fragment that is cut by element range over several syncer
 * shards.  The paper's sharded syncer all-reduces the norms first and the directions second
 * (appendix "Merging methods"); so one call does ONE stage on this shard's n elements and the
 * caller sums the stage's output over the shards before the next stage:
 *
 *   stage 0  rec->delta_m_sq[j] = sum_i (Theta_i - theta_{j,i})^2 over the shard    -> sum over shards
 *   stage 1  *dir_sq = sum_i u_i^2,  u = sum_j (w_hat_j / ||D_j||) D_j, with ||D_j||
 *            from norms_sq (the summed stage-0 output)                               -> sum over shards
 *   stage 2  Delta = (sum_j w_hat_j ||D_j||) u / sqrt(*dir_sq) with the summed *dir_sq, then the
 *            outer step on the shard; rec->delta_sq, theta_sq, mom_sq are the shard's -> sum over shards
 *
 * Participation and weights are recomputed in every stage (they depend on the counters only).
 * With a single shard the three stages are ddo_merge_fragment(..., DDO_MERGE_RDA).
 */
int ddo_merge_fragment_rda_stage(int stage, float *Theta, float *v, const void *const *learners, int M,
                                 int learner_is_bf16, const uint64_t *tokens, const uint64_t *steps,
                                 uint64_t mask, int K, float eta, float mu, int nesterov, size_t n,
                                 const double *norms_sq, double *dir_sq, uint16_t *out_bf16,
                                 ddo_record *rec)
{
    double w_hat[DDO_MAX_LEARNERS], dir_coef[DDO_MAX_LEARNERS];
    double radial = 0.0, scale;
    const double eta_d = (double)eta, mu_d = (double)mu;
    size_t i;
    int j, s, st;

    memset(rec, 0, sizeof *rec);
    st = ddo_participants(mask, tokens, M, K, rec->idx, &rec->n_part);
    if (st == DDO_INVALID) return DDO_INVALID;
    s = rec->n_part;
    if (st != DDO_STATUS_OK) { rec->status = st; return 0; }
    st = ddo_weights(tokens, steps, rec->idx, s, w_hat, &rec->w_total);
    if (st == DDO_INVALID) return DDO_INVALID;
    if (st != DDO_STATUS_OK) { rec->status = st; return 0; }
    for (j = 0; j < s; ++j) {
        rec->w_hat[j] = w_hat[j];
        if (learners[rec->idx[j]] == NULL) return DDO_INVALID;
    }
    rec->status = DDO_STATUS_OK;

    if (stage == 0) {
        for (j = 0; j < s; ++j) {
            double acc = 0.0;
            for (i = 0; i < n; ++i) {
                double d = (double)Theta[i] - learner_at(learners[rec->idx[j]], learner_is_bf16, i);
                acc += d * d;
            }
            rec->delta_m_sq[j] = acc;
        }
        return 0;
    }
    if (norms_sq == NULL || dir_sq == NULL) return DDO_INVALID;
    for (j = 0; j < s; ++j) {
        double nm = sqrt(norms_sq[j]);
        rec->delta_m_sq[j] = norms_sq[j];
        radial += w_hat[j] * nm;
        dir_coef[j] = nm > 0.0 ? w_hat[j] / nm : 0.0;
    }
    if (stage == 1) {
        double acc = 0.0;
        for (i = 0; i < n; ++i) {
            double T = (double)Theta[i], u = 0.0;
            for (j = 0; j < s; ++j)
                u += dir_coef[j] * (T - learner_at(learners[rec->idx[j]], learner_is_bf16, i));
            acc += u * u;
        }
        *dir_sq = acc;
        return 0;
    }
    if (stage != 2) return DDO_INVALID;
    scale = *dir_sq > 0.0 ? radial / sqrt(*dir_sq) : 0.0;
    for (i = 0; i < n; ++i) {
        double T = (double)Theta[i], d = 0.0, vn, u, Tn;
        for (j = 0; j < s; ++j)
            d += dir_coef[j] * (T - learner_at(learners[rec->idx[j]], learner_is_bf16, i));
        d *= scale;
        vn = mu_d * (double)v[i] + d;
        u = nesterov ? d + mu_d * vn : vn;
        Tn = T - eta_d * u;
        v[i] = (float)vn;
        Theta[i] = (float)Tn;
        if (out_bf16 != NULL) out_bf16[i] = ddo_bf16_rne((float)Tn);
        rec->delta_sq += d * d;
        rec->theta_sq += (double)Theta[i] * (double)Theta[i];
        rec->mom_sq += (double)v[i] * (double)v[i];
    }
    return 0;
}

/* ---- learner side of an update (Algorithm 1 step 3; appendix "Mixing learner and syncer params") */

/* theta_m <- alpha theta_m + (1 - alpha) Theta, rounded to the learner dtype. */
void ddo_apply_to_learner(void *learner, int learner_is_bf16, const float *Theta, float alpha,
                          size_t n)
{
    const double a = (double)alpha;
    size_t i;
    for (i = 0; i < n; ++i) {
        double x = a * learner_at(learner, learner_is_bf16, i) + (1.0 - a) * (double)Theta[i];
        if (learner_is_bf16) ((uint16_t *)learner)[i] = ddo_bf16_rne((float)x);
        else ((float *)learner)[i] = (float)x;
    }
}

/* ---- int4 compression of outer gradients (appendix "Outer gradients compression") ---- */

/*
 * The paper compresses outer gradients to 4 bits per value before they are merged
 * but gives no quantiser.  PARITY UNPINNED BY THE PAPER; the reading used here:
 * blocks of 128 consecutive elements, D = Theta - theta in float32, one float32
 * scale = max|D| / 7 per block, code = round-half-even(D / scale) clamped to
 * [-7, 7], stored as code + 8 in a nibble (even element in the low nibble).
 * Every decision is taken in float32, the precision the kernel uses.
 * Non-finite differences poison their block, as IEEE arithmetic would poison the
 * uncompressed merge: a NaN difference makes the block's scale NaN (codes 0), an
 * infinite one makes it infinite (a NaN quotient is coded -7), and either way every
 * element of the block decodes to a non-finite value.
 */
#define DDO_INT4_BLOCK 128

void ddo_quantize_int4(const float *Theta, const void *learner, int learner_is_bf16, size_t n,
                       uint8_t *codes, float *scales)
{
    size_t b, i, nblocks = (n + DDO_INT4_BLOCK - 1) / DDO_INT4_BLOCK;
    memset(codes, 0, (n + 1) / 2);
    for (b = 0; b < nblocks; ++b) {
        size_t lo = b * DDO_INT4_BLOCK, hi = lo + DDO_INT4_BLOCK < n ? lo + DDO_INT4_BLOCK : n;
        float amax = 0.0f, scale;
        for (i = lo; i < hi; ++i) {
            float th = learner_is_bf16 ? ddo_bf16_to_f32(((const uint16_t *)learner)[i])
                                       : ((const float *)learner)[i];
            float d = Theta[i] - th;
            float a = fabsf(d);
            if (isnan(a) || a > amax) amax = a;      /* a NaN in the block makes its scale NaN */
        }
        scale = amax / 7.0f;
        scales[b] = scale;
        for (i = lo; i < hi; ++i) {
            float th = learner_is_bf16 ? ddo_bf16_to_f32(((const uint16_t *)learner)[i])
                                       : ((const float *)learner)[i];
            float d = Theta[i] - th;
            float q = scale > 0.0f ? rintf(d / scale) : 0.0f;
            int code;
            if (q > 7.0f) q = 7.0f;
            if (!(q >= -7.0f)) q = -7.0f;            /* also a NaN quotient (infinite D over infinite scale) */
            code = (int)q + 8;
            codes[i / 2] |= (uint8_t)(code << (4 * (i & 1)));
        }
    }
}

/* Outer gradient of element i as the syncer sees it: (code - 8) * scale, in float32. */
static double int4_at(const uint8_t *codes, const float *scales, size_t i)
{
    int code = (codes[i / 2] >> (4 * (i & 1))) & 15;
    float d = (float)(code - 8) * scales[i / DDO_INT4_BLOCK];
    return (double)d;
}

/*
 * The merge of Algorithm 2 with compressed outer gradients: Delta = sum_m w_hat_m D^_m,
 * then the same outer step.  Participation and weights exactly as ddo_merge_fragment.
 */
int ddo_merge_fragment_int4(float *Theta, float *v, const uint8_t *const *codes,
                            const float *const *scales, int M, const uint64_t *tokens,
                            const uint64_t *steps, uint64_t mask, int K, float eta, float mu,
                            int nesterov, size_t n, uint16_t *out_bf16, ddo_record *rec)
{
    double w_hat[DDO_MAX_LEARNERS];
    const double eta_d = (double)eta, mu_d = (double)mu;
    size_t i;
    int j, s, st;
    memset(rec, 0, sizeof *rec);
    st = ddo_participants(mask, tokens, M, K, rec->idx, &rec->n_part);
    if (st == DDO_INVALID) return DDO_INVALID;
    s = rec->n_part;
    if (st != DDO_STATUS_OK) { rec->status = st; return 0; }
    st = ddo_weights(tokens, steps, rec->idx, s, w_hat, &rec->w_total);
    if (st == DDO_INVALID) return DDO_INVALID;
    if (st != DDO_STATUS_OK) { rec->status = st; return 0; }
    for (j = 0; j < s; ++j) {
        rec->w_hat[j] = w_hat[j];
        if (codes[rec->idx[j]] == NULL || scales[rec->idx[j]] == NULL) return DDO_INVALID;
    }
    for (i = 0; i < n; ++i) {
        double d = 0.0, vn, u, Tn;
        for (j = 0; j < s; ++j) d += w_hat[j] * int4_at(codes[rec->idx[j]], scales[rec->idx[j]], i);
        vn = mu_d * (double)v[i] + d;
        u = nesterov ? d + mu_d * vn : vn;
        Tn = (double)Theta[i] - eta_d * u;
        v[i] = (float)vn;
        Theta[i] = (float)Tn;
        if (out_bf16 != NULL) out_bf16[i] = ddo_bf16_rne((float)Tn);
        rec->delta_sq += d * d;
        rec->theta_sq += (double)Theta[i] * (double)Theta[i];
        rec->mom_sq += (double)v[i] * (double)v[i];
    }
    rec->status = DDO_STATUS_OK;
    return 0;
}

/* ---- quorum / grace window ("Adaptive Quorum Window", Section 3.2) --------- */

/*
 * xi_grace <= gamma * xi_slack,  xi_slack = tau xi_step - (xi_quorum + xi_sync).
 * The largest admissible window, clamped at zero when there is no slack.
 */
double ddo_grace_window(double tau, double xi_step, double xi_quorum, double xi_sync,
                        double gamma)
{
    double slack = tau * xi_step - (xi_quorum + xi_sync);
    double g = gamma * slack;
    return g > 0.0 ? g : 0.0;
}

/*
 * Which learners are admitted: the syncer proceeds once K reports have arrived
 * (time t_K of the K-th earliest finite arrival) and then waits xi_grace more;
 * every report that has arrived by t_K + xi_grace takes part.  Fewer than K
 * finite arrivals: quorum not met, nobody is admitted.  K = 0 acts as K = 1.
 */
int ddo_select_quorum(const double *arrival, int M, int K, double grace,
                      uint64_t *mask_out, int32_t *n_admitted)
{
    double sorted[DDO_MAX_LEARNERS];
    int m, a, b, n_fin = 0, Keff = K > 1 ? K : 1;
    uint64_t mask = 0;
    int cnt = 0;
    if (M < 1 || M > DDO_MAX_LEARNERS || K < 0 || K > M || !(grace >= 0.0)) return DDO_INVALID;
    for (m = 0; m < M; ++m) {
        if (isnan(arrival[m])) return DDO_INVALID;
        if (isfinite(arrival[m])) sorted[n_fin++] = arrival[m];
    }
    for (a = 1; a < n_fin; ++a) {                 /* insertion sort, ascending */
        double key = sorted[a];
        for (b = a - 1; b >= 0 && sorted[b] > key; --b) sorted[b + 1] = sorted[b];
        sorted[b + 1] = key;
    }
    if (n_fin >= Keff) {
        double deadline = sorted[Keff - 1] + grace;
        for (m = 0; m < M; ++m)
            if (isfinite(arrival[m]) && arrival[m] <= deadline) { mask |= (uint64_t)1 << m; ++cnt; }
    }
    *mask_out = mask;
    *n_admitted = cnt;
    return n_fin >= Keff ? DDO_STATUS_OK : DDO_STATUS_QUORUM_NOT_MET;
}
