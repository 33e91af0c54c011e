// dd_merge_fragment_host: the merge for a fragment whose operands live in HOST
// memory (the syncer pulls learner fragments from the learners' host RAM, Section 4
// and the system-overview figure).  The fragment is cut into chunks that flow
// through a ring of device staging sets on three streams:
//     copy-in (H2D)  ->  fused merge kernel  ->  copy-out (D2H)
// so PCIe traffic in both directions overlaps the kernel.  Only the copies of
// participating learners cross the bus.
#include <cstring>
#include <new>
#include <vector>

#include <cuda_runtime.h>

#include "dd_ctx.h"

namespace ddm {

constexpr int kSets = 3;                              // staging sets in flight
constexpr size_t kDefaultChunk = (size_t)1 << 22;     // elements per chunk

struct StageSet {
    float *theta = nullptr;
    float *mom = nullptr;
    uint16_t *out = nullptr;
    char *learners = nullptr;                         // [s_cap][chunk] learner elements
    cudaEvent_t in_done = nullptr, k_done = nullptr, out_done = nullptr;
    bool busy = false;
};

struct HostPipe {
    StageSet set[kSets];
    size_t chunk_cap = 0;                             // elements
    size_t learner_bytes_cap = 0;                     // bytes of `learners` per set
    cudaStream_t s_in = nullptr, s_k = nullptr, s_out = nullptr;
    cudaEvent_t start = nullptr;
    dd_merge_record *dev_records = nullptr;
    dd_merge_record *host_records = nullptr;          // pinned
    size_t records_cap = 0;
};

static void free_sets(HostPipe *hp)
{
    for (StageSet &s : hp->set) {
        if (s.theta) cudaFree(s.theta);
        if (s.mom) cudaFree(s.mom);
        if (s.out) cudaFree(s.out);
        if (s.learners) cudaFree(s.learners);
        s.theta = s.mom = nullptr;
        s.out = nullptr;
        s.learners = nullptr;
    }
    hp->chunk_cap = 0;
    hp->learner_bytes_cap = 0;
}

void host_pipe_destroy(dd_ctx *ctx)
{
    HostPipe *hp = ctx->pipe;
    if (!hp) return;
    free_sets(hp);
    for (StageSet &s : hp->set) {
        if (s.in_done) cudaEventDestroy(s.in_done);
        if (s.k_done) cudaEventDestroy(s.k_done);
        if (s.out_done) cudaEventDestroy(s.out_done);
    }
    if (hp->start) cudaEventDestroy(hp->start);
    if (hp->s_in) cudaStreamDestroy(hp->s_in);
    if (hp->s_k) cudaStreamDestroy(hp->s_k);
    if (hp->s_out) cudaStreamDestroy(hp->s_out);
    if (hp->dev_records) cudaFree(hp->dev_records);
    if (hp->host_records) cudaFreeHost(hp->host_records);
    delete hp;
    ctx->pipe = nullptr;
}

static int pipe_prepare(dd_ctx *ctx, size_t chunk, size_t learner_bytes, size_t nchunks)
{
    if (!ctx->pipe) {
        HostPipe *hp = new (std::nothrow) HostPipe();
        if (!hp) return DD_ERR_INVALID_ARG;
        ctx->pipe = hp;
        DD_CUDA(ctx, cudaStreamCreateWithFlags(&hp->s_in, cudaStreamNonBlocking));
        DD_CUDA(ctx, cudaStreamCreateWithFlags(&hp->s_k, cudaStreamNonBlocking));
        DD_CUDA(ctx, cudaStreamCreateWithFlags(&hp->s_out, cudaStreamNonBlocking));
        DD_CUDA(ctx, cudaEventCreateWithFlags(&hp->start, cudaEventDisableTiming));
        for (StageSet &s : hp->set) {
            DD_CUDA(ctx, cudaEventCreateWithFlags(&s.in_done, cudaEventDisableTiming));
            DD_CUDA(ctx, cudaEventCreateWithFlags(&s.k_done, cudaEventDisableTiming));
            DD_CUDA(ctx, cudaEventCreateWithFlags(&s.out_done, cudaEventDisableTiming));
        }
    }
    HostPipe *hp = ctx->pipe;
    if (chunk > hp->chunk_cap || learner_bytes > hp->learner_bytes_cap) {
        DD_CUDA(ctx, cudaDeviceSynchronize());
        free_sets(hp);
        for (StageSet &s : hp->set) {
            DD_CUDA(ctx, cudaMalloc(&s.theta, chunk * sizeof(float)));
            DD_CUDA(ctx, cudaMalloc(&s.mom, chunk * sizeof(float)));
            DD_CUDA(ctx, cudaMalloc(&s.out, chunk * sizeof(uint16_t)));
            DD_CUDA(ctx, cudaMalloc(&s.learners, learner_bytes ? learner_bytes : 16));
            s.busy = false;
        }
        hp->chunk_cap = chunk;
        hp->learner_bytes_cap = learner_bytes;
    }
    if (nchunks > hp->records_cap) {
        DD_CUDA(ctx, cudaDeviceSynchronize());
        if (hp->dev_records) cudaFree(hp->dev_records);
        if (hp->host_records) cudaFreeHost(hp->host_records);
        hp->dev_records = nullptr;
        hp->host_records = nullptr;
        hp->records_cap = 0;
        DD_CUDA(ctx, cudaMalloc(&hp->dev_records, nchunks * sizeof(dd_merge_record)));
        DD_CUDA(ctx, cudaMallocHost(&hp->host_records, nchunks * sizeof(dd_merge_record)));
        hp->records_cap = nchunks;
    }
    return DD_OK;
}

}  // namespace ddm

using namespace ddm;

extern "C" int dd_merge_fragment_host(dd_ctx *ctx, float *global, float *momentum,
                                      const void *const *learner_ptrs, int M,
                                      dd_dtype learner_dtype, const uint64_t *tokens,
                                      const uint64_t *steps, uint64_t quorum_mask, int K,
                                      float outer_lr, float outer_mu, uint32_t flags, size_t n,
                                      void *out_bf16, dd_merge_record *record,
                                      size_t chunk_elems, void *cuda_stream)
{
    if (!ctx) return DD_ERR_INVALID_ARG;
    if (M > DD_MAX_LEARNERS) return DD_ERR_TOO_MANY_LEARNERS;
    if (M < 1 || !learner_ptrs || !tokens || K < 0 || K > M) return DD_ERR_INVALID_ARG;
    if (learner_dtype != DD_F32 && learner_dtype != DD_BF16) return DD_ERR_INVALID_ARG;
    if (n > 0 && (!global || !momentum)) return DD_ERR_INVALID_ARG;
    if (chunk_elems == 0) chunk_elems = kDefaultChunk;
    if (chunk_elems % 8 != 0) return DD_ERR_INVALID_ARG;
    const size_t esz = learner_dtype == DD_BF16 ? 2 : 4;

    // Which copies have to cross the bus: the same predicate the kernel applies.
    // The kernel still derives participation, ranks and weights itself from the
    // raw mask and counters; learners that do not take part get no staging slot.
    const uint64_t mask = M >= 64 ? quorum_mask : (quorum_mask & ((1ull << M) - 1ull));
    int slot_of[DD_MAX_LEARNERS];
    int s = 0;
    for (int m = 0; m < M; ++m) {
        const bool takes_part = ((mask >> m) & 1ull) && tokens[m] > 0;
        slot_of[m] = takes_part ? s++ : -1;
        if (takes_part && n > 0 && !learner_ptrs[m]) return DD_ERR_INVALID_ARG;
    }
    const bool quorum = s >= (K > 1 ? K : 1);
    const size_t chunk = n < chunk_elems ? (n ? ((n + 7) / 8) * 8 : 8) : chunk_elems;
    const size_t nchunks = (quorum && n > 0) ? (n + chunk - 1) / chunk : 1;

    DeviceGuard guard(ctx->device);
    if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice, "cudaSetDevice");
    int rc = pipe_prepare(ctx, chunk, (size_t)s * chunk * esz, nchunks);
    if (rc != DD_OK) return rc;
    HostPipe *hp = ctx->pipe;

    // Order this call after whatever the caller queued on its stream.
    DD_CUDA(ctx, cudaEventRecord(hp->start, (cudaStream_t)cuda_stream));
    DD_CUDA(ctx, cudaStreamWaitEvent(hp->s_in, hp->start, 0));
    DD_CUDA(ctx, cudaStreamWaitEvent(hp->s_k, hp->start, 0));
    DD_CUDA(ctx, cudaStreamWaitEvent(hp->s_out, hp->start, 0));
    for (StageSet &st : hp->set) st.busy = false;

    const void *dev_ptrs[DD_MAX_LEARNERS];
    for (size_t c = 0; c < nchunks; ++c) {
        StageSet &st = hp->set[c % kSets];
        const size_t lo = c * chunk;
        const size_t len = (quorum && n > 0) ? (n - lo < chunk ? n - lo : chunk) : 0;
        if (st.busy) DD_CUDA(ctx, cudaStreamWaitEvent(hp->s_in, st.out_done, 0));
        if (len) {
            DD_CUDA(ctx, cudaMemcpyAsync(st.theta, global + lo, len * sizeof(float),
                                         cudaMemcpyHostToDevice, hp->s_in));
            DD_CUDA(ctx, cudaMemcpyAsync(st.mom, momentum + lo, len * sizeof(float),
                                         cudaMemcpyHostToDevice, hp->s_in));
        }
        for (int m = 0; m < M; ++m) {
            dev_ptrs[m] = nullptr;
            if (slot_of[m] < 0) continue;
            char *dst = st.learners + (size_t)slot_of[m] * chunk * esz;
            dev_ptrs[m] = dst;
            if (len)
                DD_CUDA(ctx, cudaMemcpyAsync(dst, (const char *)learner_ptrs[m] + lo * esz, len * esz,
                                             cudaMemcpyHostToDevice, hp->s_in));
        }
        DD_CUDA(ctx, cudaEventRecord(st.in_done, hp->s_in));
        DD_CUDA(ctx, cudaStreamWaitEvent(hp->s_k, st.in_done, 0));
        rc = dd_merge_fragment(ctx, st.theta, st.mom, dev_ptrs, M, learner_dtype, tokens, steps,
                               quorum_mask, K, outer_lr, outer_mu, flags, len,
                               out_bf16 ? st.out : nullptr, hp->dev_records + c, hp->s_k);
        if (rc != DD_OK) {
            cudaDeviceSynchronize();
            return rc;
        }
        DD_CUDA(ctx, cudaEventRecord(st.k_done, hp->s_k));
        DD_CUDA(ctx, cudaStreamWaitEvent(hp->s_out, st.k_done, 0));
        if (len) {
            DD_CUDA(ctx, cudaMemcpyAsync(global + lo, st.theta, len * sizeof(float),
                                         cudaMemcpyDeviceToHost, hp->s_out));
            DD_CUDA(ctx, cudaMemcpyAsync(momentum + lo, st.mom, len * sizeof(float),
                                         cudaMemcpyDeviceToHost, hp->s_out));
            if (out_bf16)
                DD_CUDA(ctx, cudaMemcpyAsync((uint16_t *)out_bf16 + lo, st.out, len * sizeof(uint16_t),
                                             cudaMemcpyDeviceToHost, hp->s_out));
        }
        DD_CUDA(ctx, cudaEventRecord(st.out_done, hp->s_out));
        st.busy = true;
    }
    DD_CUDA(ctx, cudaStreamWaitEvent(hp->s_out, hp->set[(nchunks - 1) % kSets].k_done, 0));
    DD_CUDA(ctx, cudaMemcpyAsync(hp->host_records, hp->dev_records, nchunks * sizeof(dd_merge_record),
                                 cudaMemcpyDeviceToHost, hp->s_out));
    DD_CUDA(ctx, cudaStreamSynchronize(hp->s_out));
    DD_CUDA(ctx, cudaStreamSynchronize(hp->s_k));

    if (record) {
        // Participation and weights are the same in every chunk; squared norms add up.
        *record = hp->host_records[0];
        for (size_t c = 1; c < nchunks; ++c) {
            const dd_merge_record &r = hp->host_records[c];
            if (r.status != DD_STATUS_OK) record->status = r.status;
            record->delta_sq += r.delta_sq;
            record->theta_sq += r.theta_sq;
            record->mom_sq += r.mom_sq;
            for (int j = 0; j < DD_MAX_LEARNERS; ++j) record->delta_m_sq[j] += r.delta_m_sq[j];
        }
    }
    return DD_OK;
}
