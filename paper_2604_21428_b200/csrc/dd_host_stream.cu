// dd_merge_fragment_host and its batched and int4 variants: the merge for fragments
// whose operands live in HOST memory (the syncer pulls learner fragments from the
// learners' host RAM, Section 4 and the system-overview figure).  The fragments are
// cut into chunks that flow through a ring of device staging sets on three streams:
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
// Default chunk: an eighth of the fragment in whole 2^20 elements, between 2^20 and 2^24.  Copies
// of 16 MB and more run PCIe at its best rate (2^24 elements: +2.7 % end to end over 2^22 on a
// 125 M-element fragment); a fragment that is cut into fewer than about 8 chunks loses more to the
// first copy-in and the last copy-out, which overlap nothing.  Smaller units do not pay: a chunk
// costs about 45 us of host work (its copies, events and launch), so 2^18-element chunks made a
// 21 M-element fragment 40 % slower and a 1 M-element one no faster than a single chunk.
constexpr size_t kChunkUnit = (size_t)1 << 20, kMaxDefaultChunk = (size_t)1 << 24;
static size_t default_chunk(size_t n)
{
    size_t c = (n / 8 + kChunkUnit - 1) / kChunkUnit * kChunkUnit;
    if (c < kChunkUnit) c = kChunkUnit;
    return c > kMaxDefaultChunk ? kMaxDefaultChunk : c;
}

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
        // grow both capacities monotonically, so alternating callers do not reallocate every time
        if (chunk < hp->chunk_cap) chunk = hp->chunk_cap;
        if (learner_bytes < hp->learner_bytes_cap) learner_bytes = hp->learner_bytes_cap;
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

// What the learners' payload is: their copies, or int4 codes with one float32 scale per block.
enum PayloadKind { kPayloadF32 = 0, kPayloadBF16 = 1, kPayloadInt4 = 2 };

// One fragment whose operands live in host memory.
struct HostFrag {
    float *global;
    float *momentum;
    void *out_bf16;
    const void *const *payload;        // M host pointers: learner copies, or int4 codes
    const float *const *scales;        // int4 only: M host pointers
    const uint64_t *tokens;
    const uint64_t *steps;
    uint64_t mask;
    int K;
    size_t n;
    dd_merge_record *record;           // host, nullable
};

static size_t round16(size_t b) { return (b + 15) / 16 * 16; }

// Bytes one participant's payload of `len` elements occupies in a staging set: the copy itself,
// or the codes followed (16-byte aligned) by the scales.
static size_t payload_bytes(int kind, size_t len)
{
    if (kind == kPayloadInt4) return round16((len + 1) / 2) + round16((len + DD_INT4_BLOCK - 1) / DD_INT4_BLOCK * sizeof(float));
    return round16(len * (kind == kPayloadBF16 ? 2 : 4));
}

// The pipeline shared by the host-buffer entry points: the fragments are cut into chunks that flow,
// without a pause at fragment boundaries, through kSets staging sets on three streams
//     copy-in (H2D)  ->  fused merge kernel  ->  copy-out (D2H).
// Blocks until every result is in host memory.
static int run_host_pipeline(dd_ctx *ctx, const HostFrag *frags, int P, int M, int kind, float outer_lr,
                             float outer_mu, uint32_t flags, size_t chunk_elems, void *cuda_stream)
{
    if (!ctx) return DD_ERR_INVALID_ARG;
    if (M > DD_MAX_LEARNERS) return DD_ERR_TOO_MANY_LEARNERS;
    if (M < 1 || P < 0 || (P > 0 && !frags)) return DD_ERR_INVALID_ARG;
    // a chunk boundary must not split an 8-element step, nor (int4) a quantisation block
    if (chunk_elems != 0 && chunk_elems % (kind == kPayloadInt4 ? DD_INT4_BLOCK : 8) != 0) return DD_ERR_INVALID_ARG;
    if (P == 0) return DD_OK;

    struct Plan {
        int slot_of[DD_MAX_LEARNERS];
        int s;
        bool quorum;
        size_t first_chunk, nchunks, chunk;
    };
    std::vector<Plan> plan((size_t)P);
    size_t total_chunks = 0, max_chunk = 8, max_payload = 16;
    for (int p = 0; p < P; ++p) {
        const HostFrag &f = frags[p];
        Plan &pl = plan[(size_t)p];
        if (!f.payload || !f.tokens || f.K < 0 || f.K > M) return DD_ERR_INVALID_ARG;
        if (kind == kPayloadInt4 && !f.scales) return DD_ERR_INVALID_ARG;
        if (f.n > 0 && (!f.global || !f.momentum)) return DD_ERR_INVALID_ARG;
        // Which payloads have to cross the bus: the same predicate the kernel applies.  The kernel
        // still derives participation, ranks and weights itself from the raw mask and counters;
        // learners that do not take part get no staging slot.
        const uint64_t mask = M >= 64 ? f.mask : (f.mask & ((1ull << M) - 1ull));
        pl.s = 0;
        for (int m = 0; m < M; ++m) {
            const bool takes_part = ((mask >> m) & 1ull) && f.tokens[m] > 0;
            pl.slot_of[m] = takes_part ? pl.s++ : -1;
            if (takes_part && f.n > 0 && (!f.payload[m] || (kind == kPayloadInt4 && !f.scales[m]))) return DD_ERR_INVALID_ARG;
        }
        pl.quorum = pl.s >= (f.K > 1 ? f.K : 1);
        const size_t want = chunk_elems ? chunk_elems : default_chunk(f.n);
        pl.chunk = f.n < want ? (f.n ? ((f.n + 7) / 8) * 8 : 8) : want;
        pl.nchunks = (pl.quorum && f.n > 0) ? (f.n + pl.chunk - 1) / pl.chunk : 1;
        pl.first_chunk = total_chunks;
        total_chunks += pl.nchunks;
        if (pl.chunk > max_chunk) max_chunk = pl.chunk;
        const size_t pb = (size_t)pl.s * payload_bytes(kind, pl.chunk);
        if (pb > max_payload) max_payload = pb;
    }

    DeviceGuard guard(ctx->device);
    if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice, "cudaSetDevice");
    int rc = pipe_prepare(ctx, max_chunk, max_payload, total_chunks);
    if (rc != DD_OK) return rc;
    HostPipe *hp = ctx->pipe;

    // Order this call after whatever the caller queued on its stream.
    DD_CUDA(ctx, cudaEventRecord(hp->start, (cudaStream_t)cuda_stream));
    DD_CUDA(ctx, cudaStreamWaitEvent(hp->s_in, hp->start, 0));
    DD_CUDA(ctx, cudaStreamWaitEvent(hp->s_k, hp->start, 0));
    DD_CUDA(ctx, cudaStreamWaitEvent(hp->s_out, hp->start, 0));
    for (StageSet &st : hp->set) st.busy = false;

    const void *dev_ptrs[DD_MAX_LEARNERS];
    const float *dev_scales[DD_MAX_LEARNERS];
    size_t c = 0;                                     // running chunk index over all fragments
    for (int p = 0; p < P; ++p) {
        const HostFrag &f = frags[p];
        const Plan &pl = plan[(size_t)p];
        const size_t per = payload_bytes(kind, pl.chunk);
        for (size_t k = 0; k < pl.nchunks; ++k, ++c) {
            StageSet &st = hp->set[c % kSets];
            const size_t lo = k * pl.chunk;
            const size_t len = (pl.quorum && f.n > 0) ? (f.n - lo < pl.chunk ? f.n - lo : pl.chunk) : 0;
            if (st.busy) DD_CUDA(ctx, cudaStreamWaitEvent(hp->s_in, st.out_done, 0));
            if (len) {
                DD_CUDA(ctx, cudaMemcpyAsync(st.theta, f.global + lo, len * sizeof(float),
                                             cudaMemcpyHostToDevice, hp->s_in));
                DD_CUDA(ctx, cudaMemcpyAsync(st.mom, f.momentum + lo, len * sizeof(float),
                                             cudaMemcpyHostToDevice, hp->s_in));
            }
            for (int m = 0; m < M; ++m) {
                dev_ptrs[m] = nullptr;
                dev_scales[m] = nullptr;
                if (pl.slot_of[m] < 0) continue;
                char *dst = st.learners + (size_t)pl.slot_of[m] * per;
                dev_ptrs[m] = dst;
                if (kind == kPayloadInt4) {
                    const size_t code_bytes = (len + 1) / 2, nblk = (len + DD_INT4_BLOCK - 1) / DD_INT4_BLOCK;
                    char *sdst = dst + round16((pl.chunk + 1) / 2);
                    dev_scales[m] = reinterpret_cast<const float *>(sdst);
                    if (len) {
                        DD_CUDA(ctx, cudaMemcpyAsync(dst, (const char *)f.payload[m] + lo / 2, code_bytes,
                                                     cudaMemcpyHostToDevice, hp->s_in));
                        DD_CUDA(ctx, cudaMemcpyAsync(sdst, f.scales[m] + lo / DD_INT4_BLOCK, nblk * sizeof(float),
                                                     cudaMemcpyHostToDevice, hp->s_in));
                    }
                } else if (len) {
                    const size_t esz = kind == kPayloadBF16 ? 2 : 4;
                    DD_CUDA(ctx, cudaMemcpyAsync(dst, (const char *)f.payload[m] + lo * esz, len * esz,
                                                 cudaMemcpyHostToDevice, hp->s_in));
                }
            }
            DD_CUDA(ctx, cudaEventRecord(st.in_done, hp->s_in));
            DD_CUDA(ctx, cudaStreamWaitEvent(hp->s_k, st.in_done, 0));
            if (kind == kPayloadInt4)
                rc = dd_merge_fragment_int4(ctx, st.theta, st.mom, reinterpret_cast<const uint8_t *const *>(dev_ptrs),
                                            dev_scales, M, f.tokens, f.steps, f.mask, f.K, outer_lr, outer_mu, flags,
                                            len, f.out_bf16 ? st.out : nullptr, hp->dev_records + c, hp->s_k);
            else
                rc = dd_merge_fragment(ctx, st.theta, st.mom, dev_ptrs, M, kind == kPayloadBF16 ? DD_BF16 : DD_F32,
                                       f.tokens, f.steps, f.mask, f.K, outer_lr, outer_mu, flags, len,
                                       f.out_bf16 ? st.out : nullptr, hp->dev_records + c, hp->s_k);
            if (rc != DD_OK) {
                cudaDeviceSynchronize();
                return rc;
            }
            DD_CUDA(ctx, cudaEventRecord(st.k_done, hp->s_k));
            DD_CUDA(ctx, cudaStreamWaitEvent(hp->s_out, st.k_done, 0));
            if (len) {
                DD_CUDA(ctx, cudaMemcpyAsync(f.global + lo, st.theta, len * sizeof(float),
                                             cudaMemcpyDeviceToHost, hp->s_out));
                DD_CUDA(ctx, cudaMemcpyAsync(f.momentum + lo, st.mom, len * sizeof(float),
                                             cudaMemcpyDeviceToHost, hp->s_out));
                if (f.out_bf16)
                    DD_CUDA(ctx, cudaMemcpyAsync((uint16_t *)f.out_bf16 + lo, st.out, len * sizeof(uint16_t),
                                                 cudaMemcpyDeviceToHost, hp->s_out));
            }
            DD_CUDA(ctx, cudaEventRecord(st.out_done, hp->s_out));
            st.busy = true;
        }
    }
    DD_CUDA(ctx, cudaStreamWaitEvent(hp->s_out, hp->set[(total_chunks - 1) % kSets].k_done, 0));
    DD_CUDA(ctx, cudaMemcpyAsync(hp->host_records, hp->dev_records, total_chunks * sizeof(dd_merge_record),
                                 cudaMemcpyDeviceToHost, hp->s_out));
    DD_CUDA(ctx, cudaStreamSynchronize(hp->s_out));
    DD_CUDA(ctx, cudaStreamSynchronize(hp->s_k));

    for (int p = 0; p < P; ++p) {
        dd_merge_record *record = frags[p].record;
        if (!record) continue;
        // Participation and weights are the same in every chunk; squared norms add up, in chunk order.
        const Plan &pl = plan[(size_t)p];
        *record = hp->host_records[pl.first_chunk];
        for (size_t k = 1; k < pl.nchunks; ++k) {
            const dd_merge_record &r = hp->host_records[pl.first_chunk + k];
            if (r.status != DD_STATUS_OK) record->status = r.status;
            record->delta_sq += r.delta_sq;
            record->theta_sq += r.theta_sq;
            record->mom_sq += r.mom_sq;
            for (int j = 0; j < DD_MAX_LEARNERS; ++j) record->delta_m_sq[j] += r.delta_m_sq[j];
        }
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
    if (learner_dtype != DD_F32 && learner_dtype != DD_BF16) return DD_ERR_INVALID_ARG;
    const HostFrag f = {global, momentum, out_bf16, learner_ptrs, nullptr, tokens, steps, quorum_mask, K, n, record};
    return run_host_pipeline(ctx, &f, 1, M, learner_dtype == DD_BF16 ? kPayloadBF16 : kPayloadF32, outer_lr, outer_mu,
                             flags, chunk_elems, cuda_stream);
}

extern "C" int dd_merge_fragments_batched_host(dd_ctx *ctx, const dd_fragment_desc *descs, int P, int M,
                                               dd_dtype learner_dtype, float outer_lr, float outer_mu,
                                               uint32_t flags, dd_merge_record *records, size_t chunk_elems,
                                               void *cuda_stream)
{
    if (learner_dtype != DD_F32 && learner_dtype != DD_BF16) return DD_ERR_INVALID_ARG;
    if (P < 0 || (P > 0 && !descs)) return DD_ERR_INVALID_ARG;
    std::vector<HostFrag> frags((size_t)(P > 0 ? P : 0));
    for (int p = 0; p < P; ++p) {
        const dd_fragment_desc &d = descs[p];
        frags[(size_t)p] = {d.global, d.momentum, d.out_bf16, d.learner_ptrs, nullptr, d.tokens, d.steps,
                            d.quorum_mask, d.K, (size_t)d.n, records ? records + p : nullptr};
    }
    return run_host_pipeline(ctx, frags.data(), P, M, learner_dtype == DD_BF16 ? kPayloadBF16 : kPayloadF32, outer_lr,
                             outer_mu, flags, chunk_elems, cuda_stream);
}

extern "C" int dd_merge_fragment_int4_host(dd_ctx *ctx, float *global, float *momentum,
                                           const uint8_t *const *code_ptrs, const float *const *scale_ptrs, int M,
                                           const uint64_t *tokens, const uint64_t *steps, uint64_t quorum_mask,
                                           int K, float outer_lr, float outer_mu, uint32_t flags, size_t n,
                                           void *out_bf16, dd_merge_record *record, size_t chunk_elems,
                                           void *cuda_stream)
{
    const HostFrag f = {global, momentum, out_bf16, reinterpret_cast<const void *const *>(code_ptrs), scale_ptrs,
                        tokens, steps, quorum_mask, K, n, record};
    return run_host_pipeline(ctx, &f, 1, M, kPayloadInt4, outer_lr, outer_mu, flags, chunk_elems, cuda_stream);
}
