// Private context layout of libddmerge (shared by its translation units).
#pragma once

#include <cstdio>

#include <cuda_runtime.h>

#include "dd_internal.h"

namespace ddm {

constexpr int kSlots = 4;   // descriptor staging ring (batched calls in flight)

struct Slot {
    DevFrag *host = nullptr;    // pinned
    DevFrag *dev = nullptr;
    size_t cap = 0;             // fragments
    cudaEvent_t done = nullptr;
    bool used = false;
};

struct HostPipe;   // staging for dd_merge_fragment_host (dd_host_stream.cu)

}  // namespace ddm

struct dd_ctx {
    int device = 0;
    int sm_count = 0;
    int grid[2][2] = {{0, 0}, {0, 0}};        // [bf16][per-learner diag] persistent grid size
    double *partials = nullptr;
    size_t partials_cap = 0;                  // doubles
    unsigned *tickets = nullptr;
    size_t tickets_cap = 0;
    ddm::Slot slots[ddm::kSlots];
    int next_slot = 0;
    float *rda_scratch = nullptr;             // mean direction of radial-directional merges
    size_t rda_scratch_cap = 0;               // floats
    dd_merge_record *rda_records = nullptr;   // hand-over records when the caller passes none
    size_t rda_records_cap = 0;
    double *gram = nullptr;                   // Gram matrices of two-launch radial-directional merges
    size_t gram_cap = 0;                      // fragments
    int gram_grid[2] = {0, 0};                // [bf16] persistent grid of the Gram launch
    ddm::HostPipe *pipe = nullptr;
    char cuda_err[256] = {0};
};

namespace ddm {

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard()
    {
        int cur = -1;
        if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
    }
};

inline int cuda_fail(dd_ctx *ctx, cudaError_t e, const char *where)
{
    if (ctx) snprintf(ctx->cuda_err, sizeof ctx->cuda_err, "%s: %s", where, cudaGetErrorString(e));
    (void)cudaGetLastError();
    return DD_ERR_CUDA;
}

#define DD_CUDA(ctx, call)                                           \
    do {                                                             \
        cudaError_t e_ = (call);                                     \
        if (e_ != cudaSuccess) return cuda_fail((ctx), e_, #call);   \
    } while (0)

void host_pipe_destroy(dd_ctx *ctx);

// Shared by the entry points (defined in dd_merge.cu).
// Validates one fragment's arguments and fills its device descriptor (tile range excluded);
// learner_bytes is the size of one learner buffer, for the overlap checks.
int fill_fragment(DevFrag &d, float *global, float *momentum, void *out_bf16,
                  const void *const *learner_ptrs, const uint64_t *tokens, const uint64_t *steps,
                  uint64_t mask, int K, uint64_t n, int M, size_t learner_bytes);
int check_common(const dd_ctx *ctx, int M, dd_dtype dtype, float lr, float mu, uint32_t flags);
// Grows the diagnostics workspace to P x nq x grid partial sums (and P tickets).
int ensure_workspace(dd_ctx *ctx, size_t P, size_t nq, size_t grid);

}  // namespace ddm
