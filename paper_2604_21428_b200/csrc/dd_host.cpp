// Host-only helpers of libddmerge: quorum / grace-window selection (Section 3.2,
// "Adaptive Quorum Window") and status strings.  No CUDA here.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <vector>

#include "dd_merge.h"

extern "C" double dd_grace_window(double tau, double xi_step, double xi_quorum, double xi_sync,
                                  double gamma)
{
    // xi_grace <= gamma * xi_slack with xi_slack = tau * xi_step - (xi_quorum + xi_sync);
    // without slack the syncer proceeds as soon as the quorum is met.
    const double slack = tau * xi_step - (xi_quorum + xi_sync);
    return std::max(0.0, gamma * slack);
}

extern "C" int dd_grace_controller_init(dd_grace_controller *gc, double tau, double gamma, double beta)
{
    if (!gc || !(tau > 0.0) || !(gamma >= 0.0 && gamma < 1.0) || !(beta >= 0.0 && beta < 1.0))
        return DD_ERR_INVALID_ARG;
    gc->tau = tau;
    gc->gamma = gamma;
    gc->beta = beta;
    gc->xi_step = gc->xi_quorum = gc->xi_sync = 0.0;
    gc->n_obs = 0;
    return DD_OK;
}

extern "C" int dd_grace_controller_observe(dd_grace_controller *gc, double step_s, double quorum_s,
                                           double sync_s)
{
    if (!gc || !(step_s >= 0.0) || !(quorum_s >= 0.0) || !(sync_s >= 0.0)) return DD_ERR_INVALID_ARG;
    if (gc->n_obs == 0) {
        gc->xi_step = step_s;
        gc->xi_quorum = quorum_s;
        gc->xi_sync = sync_s;
    } else {
        const double b = gc->beta;
        gc->xi_step = b * gc->xi_step + (1.0 - b) * step_s;
        gc->xi_quorum = b * gc->xi_quorum + (1.0 - b) * quorum_s;
        gc->xi_sync = b * gc->xi_sync + (1.0 - b) * sync_s;
    }
    if (gc->n_obs < INT32_MAX) gc->n_obs += 1;
    return DD_OK;
}

extern "C" double dd_grace_controller_window(const dd_grace_controller *gc)
{
    if (!gc || gc->n_obs == 0) return 0.0;
    return dd_grace_window(gc->tau, gc->xi_step, gc->xi_quorum, gc->xi_sync, gc->gamma);
}

extern "C" int dd_select_quorum(const double *arrival_s, int M, int K, double grace_s,
                                uint64_t *mask_out, int *n_admitted)
{
    if (!arrival_s || !mask_out || !n_admitted) return DD_ERR_INVALID_ARG;
    if (M > DD_MAX_LEARNERS) return DD_ERR_TOO_MANY_LEARNERS;
    if (M < 1 || K < 0 || K > M || !(grace_s >= 0.0)) return DD_ERR_INVALID_ARG;
    *mask_out = 0;
    *n_admitted = 0;
    std::vector<double> seen;
    seen.reserve((size_t)M);
    for (int m = 0; m < M; ++m) {
        if (std::isnan(arrival_s[m])) return DD_ERR_INVALID_ARG;
        if (std::isfinite(arrival_s[m])) seen.push_back(arrival_s[m]);
    }
    const size_t need = (size_t)std::max(K, 1);
    if (seen.size() < need) return DD_OK;                 // quorum never met: nobody admitted
    // t_K: the moment the K-th report is in.  Everything that has arrived by
    // t_K + grace takes part; ties at the deadline are admitted.
    std::nth_element(seen.begin(), seen.begin() + (need - 1), seen.end());
    const double deadline = seen[need - 1] + grace_s;
    uint64_t mask = 0;
    int count = 0;
    for (int m = 0; m < M; ++m)
        if (arrival_s[m] <= deadline) { mask |= 1ull << m; ++count; }
    *mask_out = mask;
    *n_admitted = count;
    return DD_OK;
}

extern "C" int dd_plan_fragments(const uint64_t *size_bits, const int32_t *layer, int Q, int P,
                                 dd_frag_strategy strategy, int32_t *fragment_of,
                                 uint64_t *fragment_bits)
{
    if (Q < 0 || P < 1 || (Q > 0 && (!size_bits || !fragment_of))) return DD_ERR_INVALID_ARG;
    std::vector<uint64_t> total((size_t)P, 0);
    if (strategy == DD_FRAG_BALANCED) {
        // Greedy number partitioning: largest tensor first, always into the lightest fragment.
        std::vector<int> order((size_t)Q);
        for (int q = 0; q < Q; ++q) order[(size_t)q] = q;
        std::stable_sort(order.begin(), order.end(),
                         [&](int a, int b) { return size_bits[a] > size_bits[b]; });
        for (int q : order) {
            int best = 0;
            for (int p = 1; p < P; ++p)
                if (total[(size_t)p] < total[(size_t)best]) best = p;
            fragment_of[q] = best;
            total[(size_t)best] += size_bits[q];
        }
    } else if (strategy == DD_FRAG_LAYER || strategy == DD_FRAG_TENSOR) {
        if (!layer && Q > 0) return DD_ERR_INVALID_ARG;
        int n_layers = 0;
        for (int q = 0; q < Q; ++q) {
            if (layer[q] < -1) return DD_ERR_INVALID_ARG;
            n_layers = std::max(n_layers, layer[q] + 1);
        }
        const int buckets = P - 1;                   // fragment 0 is the non-transformer one
        int next = 0;                                // running index of transformer tensors
        for (int q = 0; q < Q; ++q) {
            if (layer[q] < 0) { fragment_of[q] = 0; total[0] += size_bits[q]; continue; }
            if (buckets < 1) return DD_ERR_INVALID_ARG;
            if (strategy == DD_FRAG_LAYER && buckets > n_layers) return DD_ERR_INVALID_ARG;
            const int key = strategy == DD_FRAG_LAYER ? layer[q] : next++;
            fragment_of[q] = 1 + key % buckets;
            total[(size_t)fragment_of[q]] += size_bits[q];
        }
    } else {
        return DD_ERR_INVALID_ARG;
    }
    if (fragment_bits)
        for (int p = 0; p < P; ++p) fragment_bits[p] = total[(size_t)p];
    return DD_OK;
}

extern "C" const char *dd_status_string(int rc)
{
    switch (rc) {
    case DD_OK: return "ok";
    case DD_ERR_INVALID_ARG: return "invalid argument";
    case DD_ERR_ALIGNMENT: return "device pointer not 16-byte aligned";
    case DD_ERR_ALIAS: return "learner buffer overlaps the global fragment, the momentum or the bf16 output";
    case DD_ERR_TOO_MANY_LEARNERS: return "more than DD_MAX_LEARNERS learners";
    case DD_ERR_CUDA: return "CUDA runtime error (see dd_last_cuda_error)";
    case DD_ERR_TOO_LARGE: return "size exceeds what this entry point supports";
    default: return "unknown status";
    }
}
