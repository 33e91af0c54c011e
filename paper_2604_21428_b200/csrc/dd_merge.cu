// libddmerge: context, argument validation and launch of the fused merge kernel.
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include <cuda_runtime.h>

#include "dd_merge_tma.cuh"
#include "dd_rda_gram.cuh"

namespace ddm {

// Every kernel runs 2 CTAs of 256 threads per SM (up to 128 registers per thread),
// each CTA with kTmaRingBytes of dynamic shared memory for its warps' rings.

// Direct averaging, one fragment passed by value in the kernel parameters.
template <bool BF16, bool PL>
__global__ void __launch_bounds__(kThreads, 2)
merge_single_tma_kernel(const __grid_constant__ DevFrag frag, const __grid_constant__ Common c)
{
    merge_body_tma<BF16, kModeMerge, PL>(&frag, c);
}

// Direct averaging, many fragments from a descriptor table in global memory.
template <bool BF16, bool PL>
__global__ void __launch_bounds__(kThreads, 2)
merge_batched_tma_kernel(const DevFrag *__restrict__ frags, const __grid_constant__ Common c)
{
    merge_body_tma<BF16, kModeMerge, PL>(frags, c);
}

// One pass of a radial-directional merge over a batch of fragments.
template <bool BF16, int MODE>
__global__ void __launch_bounds__(kThreads, 2)
rda_pass_kernel(const DevFrag *__restrict__ frags, const __grid_constant__ Common c)
{
    merge_body_tma<BF16, MODE, MODE == kModeNorms>(frags, c);
}

// Second launch of the two-launch radial-directional merge: the ordinary merge with the
// weights the header derives from the Gram matrix (direct averaging for DD_MERGE_AVG fragments).
template <bool BF16>
__global__ void __launch_bounds__(kThreads, 2)
rda_gram_merge_kernel(const DevFrag *__restrict__ frags, const __grid_constant__ Common c)
{
    merge_body_tma<BF16, kModeMergeGram, false>(frags, c);
}

}  // namespace ddm

#include "dd_ctx.h"

namespace ddm {

// Shared memory of the per-lane norm sums: 32 floats per warp and participant.
static size_t pl_area_bytes(int participants) { return (size_t)participants * kWarps * 32 * sizeof(float); }

// Participants the per-lane norm area must hold for a batch (0: some fragment has too many and
// every piece is reduced at once instead).
static int pl_capacity(const DevFrag *frags, int P, bool rda_only)
{
    int cap = 0;
    for (int p = 0; p < P; ++p)
        if (!rda_only || frags[p].kind == DD_MERGE_RDA) cap = frags[p].n_part_host > cap ? frags[p].n_part_host : cap;
    return cap <= kPlMaxParticipants ? cap : 0;
}

// Opts a kernel in to its dynamic shared memory and reports how many CTAs fit on an SM.
template <typename K>
static cudaError_t prepare_kernel(K kernel, int *blocks)
{
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)(kTmaRingBytes + pl_area_bytes(kPlMaxParticipants)));
    int b = 0;
    if (e == cudaSuccess)
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b, kernel, kThreads, kTmaRingBytes);
    if (e == cudaSuccess && b < *blocks) *blocks = b;
    return e;
}

template <bool BF16, bool PL>
static cudaError_t occupancy(int *blocks)
{
    *blocks = 2;      // 16 warps x 2 pieces in flight per SM is the measured sweet spot
    cudaError_t e = prepare_kernel(merge_single_tma_kernel<BF16, PL>, blocks);
    if (e == cudaSuccess) e = prepare_kernel(merge_batched_tma_kernel<BF16, PL>, blocks);
    if (PL) {         // the RDA passes share the grid of the per-learner-norm variants
        if (e == cudaSuccess) e = prepare_kernel(rda_pass_kernel<BF16, kModeNorms>, blocks);
        if (e == cudaSuccess) e = prepare_kernel(rda_pass_kernel<BF16, kModeDir>, blocks);
        if (e == cudaSuccess) e = prepare_kernel(rda_pass_kernel<BF16, kModeApply>, blocks);
        if (e == cudaSuccess) e = prepare_kernel(rda_gram_merge_kernel<BF16>, blocks);
    }
    return e;
}

// The Gram launch has its own shape (nine warps, CTA-wide stages): resident CTAs per SM, at most 2.
template <bool BF16>
static cudaError_t gram_occupancy(int *blocks)
{
    // both instances (with and without the packed consumer) get the shared-memory attribute; the
    // grid is sized for the one that fits fewer CTAs
    int b = 2;
    cudaError_t e = cudaSuccess;
    auto one = [&](auto kernel) {
        if (e != cudaSuccess) return;
        e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kGramRingBytes);
        int x = 0;
        if (e == cudaSuccess) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&x, kernel, kGramThreads, kGramRingBytes);
        if (x < b) b = x;
    };
    one(rda_gram_kernel<BF16, true>);
    one(rda_gram_kernel<BF16, false>);
    *blocks = b;
    return e;
}

static bool overlaps(const void *a, size_t abytes, const void *b, size_t bbytes)
{
    if (!a || !b || abytes == 0 || bbytes == 0) return false;
    const uintptr_t a0 = (uintptr_t)a, b0 = (uintptr_t)b;
    return a0 < b0 + bbytes && b0 < a0 + abytes;
}

static bool misaligned(const void *p) { return ((uintptr_t)p & 15u) != 0; }

// Validates one fragment and fills its device descriptor (tile range excluded).
int fill_fragment(DevFrag &d, float *global, float *momentum, void *out_bf16,
                  const void *const *learner_ptrs, const uint64_t *tokens, const uint64_t *steps,
                  uint64_t mask, int K, uint64_t n, int M, size_t learner_bytes)
{
    if (!learner_ptrs || !tokens) return DD_ERR_INVALID_ARG;
    if (K < 0 || K > M) return DD_ERR_INVALID_ARG;
    if (n > 0 && (!global || !momentum)) return DD_ERR_INVALID_ARG;
    if (n > kMaxFragmentElems) return DD_ERR_TOO_LARGE;
    if (misaligned(global) || misaligned(momentum) || misaligned(out_bf16)) return DD_ERR_ALIGNMENT;
    const size_t lb = learner_bytes;
    if (overlaps(global, 4 * n, momentum, 4 * n) || overlaps(global, 4 * n, out_bf16, 2 * n) ||
        overlaps(momentum, 4 * n, out_bf16, 2 * n))
        return DD_ERR_ALIAS;
    std::memset(&d, 0, sizeof d);
    d.theta = global;
    d.mom = momentum;
    d.out_bf16 = static_cast<uint16_t *>(out_bf16);
    d.n = n;
    d.mask = M >= 64 ? mask : (mask & ((1ull << M) - 1ull));
    d.K = K;
    d.has_steps = steps != nullptr;
    uint64_t token_sum = 0;
    for (int m = 0; m < M; ++m) {
        d.tokens[m] = tokens[m];
        d.steps[m] = steps ? steps[m] : 0;
        d.ptrs[m] = learner_ptrs[m];
        if (steps && tokens[m] > 0 && steps[m] == 0) return DD_ERR_INVALID_ARG;
        const bool takes_part = ((d.mask >> m) & 1ull) && tokens[m] > 0;
        // the kernel sums the participants' token counts exactly, in 64 bits
        if (takes_part && __builtin_add_overflow(token_sum, tokens[m], &token_sum)) return DD_ERR_INVALID_ARG;
        if (takes_part) ++d.n_part_host;
        if (takes_part && n > 0) {
            const void *p = learner_ptrs[m];
            if (!p) return DD_ERR_INVALID_ARG;
            if (misaligned(p)) return DD_ERR_ALIGNMENT;
            if (overlaps(p, lb, global, 4 * n) || overlaps(p, lb, momentum, 4 * n) ||
                overlaps(p, lb, out_bf16, 2 * n))
                return DD_ERR_ALIAS;
        }
    }
    return DD_OK;
}

static size_t learner_bytes_of(dd_dtype dtype, uint64_t n)
{
    return (dtype == DD_BF16 ? 2u : 4u) * (size_t)n;
}

// Fused push: marks the learners whose copy the merge overwrites with Theta'.  Their
// pointers are written through, so each must be a valid, aligned buffer of its own.
static int set_push(DevFrag &d, const void *const *learner_ptrs, uint64_t push_mask, int M, uint64_t n,
                    size_t lb)
{
    const uint64_t pm = M >= 64 ? push_mask : (push_mask & ((1ull << M) - 1ull));
    for (int m = 0; m < M && n > 0; ++m) {
        if (!((pm >> m) & 1ull)) continue;
        const void *p = learner_ptrs[m];
        if (!p) return DD_ERR_INVALID_ARG;
        if (misaligned(p)) return DD_ERR_ALIGNMENT;
        if (overlaps(p, lb, d.theta, 4 * n) || overlaps(p, lb, d.mom, 4 * n) || overlaps(p, lb, d.out_bf16, 2 * n))
            return DD_ERR_ALIAS;
        for (int k = 0; k < M; ++k)        // a pushed copy sharing memory with another pushed or read copy would race
            if (k != m && learner_ptrs[k] &&
                (((pm >> k) & 1ull) || (((d.mask >> k) & 1ull) && d.tokens[k] > 0)) &&
                overlaps(p, lb, learner_ptrs[k], lb))
                return DD_ERR_ALIAS;
    }
    d.push_mask = pm;
    return DD_OK;
}

static unsigned long long tiles_of(uint64_t n)
{
    const unsigned long long t = (n + kTileElems - 1) / kTileElems;
    return t ? t : 1;       // an empty fragment still owns one (empty) tile so its record is written
}

int check_common(const dd_ctx *ctx, int M, dd_dtype dtype, float lr, float mu, uint32_t flags)
{
    if (!ctx) return DD_ERR_INVALID_ARG;
    if (M > DD_MAX_LEARNERS) return DD_ERR_TOO_MANY_LEARNERS;
    if (M < 1) return DD_ERR_INVALID_ARG;
    if (dtype != DD_F32 && dtype != DD_BF16) return DD_ERR_INVALID_ARG;
    if (!std::isfinite(lr) || !std::isfinite(mu)) return DD_ERR_INVALID_ARG;
    if (flags & ~(uint32_t)(DD_HEAVY_BALL | DD_DIAG_PER_LEARNER | DD_DIAG_STATE | DD_RDA_THREE_PASS |
                            DD_DEBUG_EXPIRE_WAIT))
        return DD_ERR_INVALID_ARG;
    return DD_OK;
}

// Grows the diagnostics workspace; growth waits for the device to drain because
// kernels in flight may still use the old one.  The first allocation already covers
// every single-fragment call (any M, any flags, any of the library's grids), so only
// a batch of many fragments can make it grow again.
int ensure_workspace(dd_ctx *ctx, size_t P, size_t nq, size_t grid)
{
    size_t need = P * nq * grid;
    const size_t single_max = (size_t)(kNumScalarDiag + DD_MAX_LEARNERS) * (size_t)ctx->sm_count * 4;
    if (need < single_max) need = single_max;
    if (need > ctx->partials_cap) {
        DD_CUDA(ctx, cudaDeviceSynchronize());
        if (ctx->partials) cudaFree(ctx->partials);
        ctx->partials = nullptr;
        ctx->partials_cap = 0;
        DD_CUDA(ctx, cudaMalloc(&ctx->partials, need * sizeof(double)));
        ctx->partials_cap = need;
    }
    if (P > ctx->tickets_cap) {
        DD_CUDA(ctx, cudaDeviceSynchronize());
        if (ctx->tickets) cudaFree(ctx->tickets);
        ctx->tickets = nullptr;
        ctx->tickets_cap = 0;
        const size_t cap = P < 64 ? 64 : P;
        DD_CUDA(ctx, cudaMalloc(&ctx->tickets, cap * sizeof(unsigned)));
        DD_CUDA(ctx, cudaMemset(ctx->tickets, 0, cap * sizeof(unsigned)));
        ctx->tickets_cap = cap;
    }
    return DD_OK;
}

// Takes the next descriptor staging slot (pinned host + device array of at least P
// fragments); waits only if a call from kSlots calls ago still owns it.
static int acquire_slot(dd_ctx *ctx, int P)
{
    Slot &slot = ctx->slots[ctx->next_slot];
    if (slot.used) DD_CUDA(ctx, cudaEventSynchronize(slot.done));
    if (!slot.done) DD_CUDA(ctx, cudaEventCreateWithFlags(&slot.done, cudaEventDisableTiming));
    if ((size_t)P > slot.cap) {
        if (slot.host) cudaFreeHost(slot.host);
        if (slot.dev) cudaFree(slot.dev);
        slot.host = nullptr;
        slot.dev = nullptr;
        slot.cap = 0;
        const size_t cap = P < 32 ? 32 : (size_t)P;
        DD_CUDA(ctx, cudaMallocHost(&slot.host, cap * sizeof(DevFrag)));
        DD_CUDA(ctx, cudaMalloc(&slot.dev, cap * sizeof(DevFrag)));
        slot.cap = cap;
    }
    return DD_OK;
}

template <bool BF16, bool PL>
static cudaError_t launch(bool single, const DevFrag *one, const DevFrag *dev_frags,
                          const Common &c, unsigned grid, cudaStream_t stream)
{
    const size_t smem = kTmaRingBytes + pl_area_bytes(c.pl_cap);
    if (single)
        merge_single_tma_kernel<BF16, PL><<<grid, kThreads, smem, stream>>>(*one, c);
    else
        merge_batched_tma_kernel<BF16, PL><<<grid, kThreads, smem, stream>>>(dev_frags, c);
    return cudaGetLastError();
}

static cudaError_t dispatch(bool bf16, bool pl, bool single, const DevFrag *one,
                            const DevFrag *dev_frags, const Common &c, unsigned grid,
                            cudaStream_t stream)
{
    if (bf16) return pl ? launch<true, true>(single, one, dev_frags, c, grid, stream)
                        : launch<true, false>(single, one, dev_frags, c, grid, stream);
    return pl ? launch<false, true>(single, one, dev_frags, c, grid, stream)
              : launch<false, false>(single, one, dev_frags, c, grid, stream);
}

}  // namespace ddm

using namespace ddm;

extern "C" int dd_create(dd_ctx **out, int device)
{
    if (!out) return DD_ERR_INVALID_ARG;
    *out = nullptr;
    if (device < 0 && cudaGetDevice(&device) != cudaSuccess) { (void)cudaGetLastError(); return DD_ERR_CUDA; }
    dd_ctx *ctx = new (std::nothrow) dd_ctx();
    if (!ctx) return DD_ERR_INVALID_ARG;
    ctx->device = device;
    DeviceGuard guard(device);
    int rc = DD_OK;
    cudaError_t e = guard.ok ? cudaSuccess : cudaErrorInvalidDevice;
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, device);
    int occ[2][2] = {{0, 0}, {0, 0}};
    if (e == cudaSuccess) e = occupancy<false, false>(&occ[0][0]);
    if (e == cudaSuccess) e = occupancy<false, true>(&occ[0][1]);
    if (e == cudaSuccess) e = occupancy<true, false>(&occ[1][0]);
    if (e == cudaSuccess) e = occupancy<true, true>(&occ[1][1]);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        delete ctx;
        return DD_ERR_CUDA;
    }
    for (int a = 0; a < 2; ++a)
        for (int b = 0; b < 2; ++b) ctx->grid[a][b] = ctx->sm_count * (occ[a][b] > 0 ? occ[a][b] : 1);
    int gocc[2] = {0, 0};
    if (gram_occupancy<false>(&gocc[0]) != cudaSuccess || gram_occupancy<true>(&gocc[1]) != cudaSuccess) {
        (void)cudaGetLastError();
        delete ctx;
        return DD_ERR_CUDA;
    }
    for (int a = 0; a < 2; ++a) ctx->gram_grid[a] = ctx->sm_count * (gocc[a] > 0 ? gocc[a] : 1);
    *out = ctx;
    return rc;
}

extern "C" int dd_destroy(dd_ctx *ctx)
{
    if (!ctx) return DD_OK;
    DeviceGuard guard(ctx->device);
    cudaDeviceSynchronize();
    if (ctx->partials) cudaFree(ctx->partials);
    if (ctx->tickets) cudaFree(ctx->tickets);
    if (ctx->rda_scratch) cudaFree(ctx->rda_scratch);
    if (ctx->rda_records) cudaFree(ctx->rda_records);
    if (ctx->gram) cudaFree(ctx->gram);
    host_pipe_destroy(ctx);
    for (Slot &s : ctx->slots) {
        if (s.host) cudaFreeHost(s.host);
        if (s.dev) cudaFree(s.dev);
        if (s.done) cudaEventDestroy(s.done);
    }
    (void)cudaGetLastError();
    delete ctx;
    return DD_OK;
}

// Launch shape of a merge with a fused push.  Measured on B200 (bf16 copies, 4 to 24
// participants, 1 to 24 pushed copies): when writes are 45 % or more of the bytes moved, one CTA
// per SM with the full ring is 5-7 % faster than two (fewer warps storing at once); below that,
// two CTAs per SM with one copy in flight per warp are 6-14 % faster than with two in flight.
// `read_bytes` / `write_bytes`: per-launch totals over the fragments that will be merged.
struct PushShape {
    bool one_cta_per_sm;
    int ring_depth;
};
static PushShape push_shape(double read_bytes, double write_bytes)
{
    const bool heavy = write_bytes >= kPushHeavyWriteShare * (read_bytes + write_bytes);
    return PushShape{heavy, heavy ? kTmaStages : 2};
}
static void add_fragment_bytes(const DevFrag &f, size_t esz, double &rd, double &wr)
{
    if (f.n_part_host == 0 || f.n_part_host < f.K) return;   // below quorum: nothing moves
    const double n = (double)f.n;
    rd += n * (8.0 + (double)esz * f.n_part_host);
    wr += n * (8.0 + (f.out_bf16 ? 2.0 : 0.0) + (double)esz * __builtin_popcountll(f.push_mask));
}

static int merge_fragment_impl(dd_ctx *ctx, float *global, float *momentum,
                               const void *const *learner_ptrs, int M, dd_dtype learner_dtype,
                               const uint64_t *tokens, const uint64_t *steps,
                               uint64_t quorum_mask, int K, float outer_lr, float outer_mu,
                               uint32_t flags, size_t n, uint64_t push_mask, void *out_bf16,
                               dd_merge_record *record, void *cuda_stream)
{
    int rc = check_common(ctx, M, learner_dtype, outer_lr, outer_mu, flags);
    if (rc != DD_OK) return rc;
    DevFrag frag;
    rc = fill_fragment(frag, global, momentum, out_bf16, learner_ptrs, tokens, steps, quorum_mask, K,
                       n, M, learner_bytes_of(learner_dtype, n));
    if (rc != DD_OK) return rc;
    if (push_mask) {
        rc = set_push(frag, learner_ptrs, push_mask, M, n, learner_bytes_of(learner_dtype, n));
        if (rc != DD_OK) return rc;
    }
    if (n == 0 && record == nullptr) return DD_OK;
    frag.tile_begin = 0;
    frag.tile_end = tiles_of(n);

    DeviceGuard guard(ctx->device);
    if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice, "cudaSetDevice");
    const bool bf16 = learner_dtype == DD_BF16, pl = (flags & DD_DIAG_PER_LEARNER) != 0;
    unsigned long long g = (unsigned long long)ctx->grid[bf16][pl];
    Common c;
    if (push_mask) {
        double rd = 0.0, wr = 0.0;
        add_fragment_bytes(frag, bf16 ? 2 : 4, rd, wr);
        const PushShape shape = push_shape(rd, wr);
        if (shape.one_cta_per_sm) g = (unsigned long long)ctx->sm_count;
        c.push_depth = shape.ring_depth;
    }
    if (g > frag.tile_end) g = frag.tile_end;
    c.eta = outer_lr;
    c.mu = outer_mu;
    c.flags = flags;
    c.M = M;
    c.P = 1;
    c.total_tiles = frag.tile_end;
    c.records = record;
    c.nq = kNumScalarDiag + (pl ? M : 0);
    if (pl && frag.n_part_host <= kPlMaxParticipants) c.pl_cap = frag.n_part_host;
    if (record) {
        rc = ensure_workspace(ctx, 1, (size_t)c.nq, (size_t)ctx->grid[bf16][pl]);
        if (rc != DD_OK) return rc;
    }
    c.partials = ctx->partials;
    c.tickets = ctx->tickets;
    cudaError_t e = dispatch(bf16, pl, true, &frag, nullptr, c, (unsigned)g, (cudaStream_t)cuda_stream);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "merge_single_kernel launch");
    return DD_OK;
}

extern "C" int dd_merge_fragment(dd_ctx *ctx, float *global, float *momentum,
                                 const void *const *learner_ptrs, int M, dd_dtype learner_dtype,
                                 const uint64_t *tokens, const uint64_t *steps,
                                 uint64_t quorum_mask, int K, float outer_lr, float outer_mu,
                                 uint32_t flags, size_t n, void *out_bf16,
                                 dd_merge_record *record, void *cuda_stream)
{
    return merge_fragment_impl(ctx, global, momentum, learner_ptrs, M, learner_dtype, tokens, steps,
                               quorum_mask, K, outer_lr, outer_mu, flags, n, 0, out_bf16, record,
                               cuda_stream);
}

extern "C" int dd_merge_fragment_push(dd_ctx *ctx, float *global, float *momentum,
                                      void *const *learner_ptrs, int M, dd_dtype learner_dtype,
                                      const uint64_t *tokens, const uint64_t *steps,
                                      uint64_t quorum_mask, int K, float outer_lr, float outer_mu,
                                      uint32_t flags, size_t n, uint64_t push_mask, void *out_bf16,
                                      dd_merge_record *record, void *cuda_stream)
{
    return merge_fragment_impl(ctx, global, momentum, learner_ptrs, M, learner_dtype, tokens, steps,
                               quorum_mask, K, outer_lr, outer_mu, flags, n, push_mask, out_bf16, record,
                               cuda_stream);
}

static int merge_batched_impl(dd_ctx *ctx, const dd_fragment_desc *descs, const uint64_t *push_masks,
                              int P, int M, dd_dtype learner_dtype, float outer_lr, float outer_mu,
                              uint32_t flags, dd_merge_record *records, void *cuda_stream)
{
    int rc = check_common(ctx, M, learner_dtype, outer_lr, outer_mu, flags);
    if (rc != DD_OK) return rc;
    if (P < 0 || (P > 0 && !descs)) return DD_ERR_INVALID_ARG;
    if (P > (1 << 20)) return DD_ERR_TOO_LARGE;
    if (P == 0) return DD_OK;
    cudaStream_t stream = (cudaStream_t)cuda_stream;

    if (P == 1) {
        // one fragment travels in the kernel parameters: no staging slot, no descriptor copy
        const dd_fragment_desc &d = descs[0];
        return merge_fragment_impl(ctx, d.global, d.momentum, d.learner_ptrs, M, learner_dtype, d.tokens, d.steps,
                                   d.quorum_mask, d.K, outer_lr, outer_mu, flags, (size_t)d.n,
                                   push_masks ? push_masks[0] : 0, d.out_bf16, records, cuda_stream);
    }

    DeviceGuard guard(ctx->device);
    if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice, "cudaSetDevice");

    rc = acquire_slot(ctx, P);
    if (rc != DD_OK) return rc;
    Slot &slot = ctx->slots[ctx->next_slot];

    unsigned long long tile = 0;
    for (int p = 0; p < P; ++p) {
        const dd_fragment_desc &d = descs[p];
        rc = fill_fragment(slot.host[p], d.global, d.momentum, d.out_bf16, d.learner_ptrs, d.tokens,
                           d.steps, d.quorum_mask, d.K, d.n, M, learner_bytes_of(learner_dtype, d.n));
        if (rc != DD_OK) return rc;
        if (push_masks && push_masks[p]) {
            rc = set_push(slot.host[p], d.learner_ptrs, push_masks[p], M, d.n,
                          learner_bytes_of(learner_dtype, d.n));
            if (rc != DD_OK) return rc;
        }
        slot.host[p].tile_begin = tile;
        tile += tiles_of(d.n);
        slot.host[p].tile_end = tile;
    }

    const bool bf16 = learner_dtype == DD_BF16, pl = (flags & DD_DIAG_PER_LEARNER) != 0;
    unsigned long long g = (unsigned long long)ctx->grid[bf16][pl];
    Common c;
    if (push_masks) {
        double rd = 0.0, wr = 0.0;
        bool any = false;
        for (int p = 0; p < P; ++p) {
            add_fragment_bytes(slot.host[p], bf16 ? 2 : 4, rd, wr);
            any = any || slot.host[p].push_mask != 0;
        }
        if (any) {
            const PushShape shape = push_shape(rd, wr);
            if (shape.one_cta_per_sm) g = (unsigned long long)ctx->sm_count;
            c.push_depth = shape.ring_depth;
        }
    }
    if (g > tile) g = tile;
    c.eta = outer_lr;
    c.mu = outer_mu;
    c.flags = flags;
    c.M = M;
    c.P = P;
    c.total_tiles = tile;
    c.records = records;
    c.nq = kNumScalarDiag + (pl ? M : 0);
    if (pl) c.pl_cap = pl_capacity(slot.host, P, false);
    if (records) {
        rc = ensure_workspace(ctx, (size_t)P, (size_t)c.nq, (size_t)ctx->grid[bf16][pl]);
        if (rc != DD_OK) return rc;
    }
    c.partials = ctx->partials;
    c.tickets = ctx->tickets;

    DD_CUDA(ctx, cudaMemcpyAsync(slot.dev, slot.host, (size_t)P * sizeof(DevFrag),
                                 cudaMemcpyHostToDevice, stream));
    cudaError_t e = dispatch(bf16, pl, false, nullptr, slot.dev, c, (unsigned)g, stream);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "merge_batched_kernel launch");
    DD_CUDA(ctx, cudaEventRecord(slot.done, stream));
    slot.used = true;
    ctx->next_slot = (ctx->next_slot + 1) % kSlots;
    return DD_OK;
}

extern "C" int dd_merge_fragments_batched(dd_ctx *ctx, const dd_fragment_desc *descs, int P, int M,
                                          dd_dtype learner_dtype, float outer_lr, float outer_mu,
                                          uint32_t flags, dd_merge_record *records,
                                          void *cuda_stream)
{
    return merge_batched_impl(ctx, descs, nullptr, P, M, learner_dtype, outer_lr, outer_mu, flags, records,
                              cuda_stream);
}

extern "C" int dd_merge_fragments_batched_push(dd_ctx *ctx, const dd_fragment_desc *descs,
                                               const uint64_t *push_masks, int P, int M,
                                               dd_dtype learner_dtype, float outer_lr, float outer_mu,
                                               uint32_t flags, dd_merge_record *records,
                                               void *cuda_stream)
{
    if (P > 0 && !push_masks) return DD_ERR_INVALID_ARG;
    return merge_batched_impl(ctx, descs, push_masks, P, M, learner_dtype, outer_lr, outer_mu, flags,
                              records, cuda_stream);
}

namespace ddm {

template <bool BF16>
static cudaError_t launch_rda_passes(const DevFrag *dev_frags, const Common &c, unsigned grid,
                                     unsigned apply_grid, cudaStream_t stream, int only_pass)
{
    if (only_pass < 0 || only_pass == DD_RDA_PASS_NORMS)
        rda_pass_kernel<BF16, kModeNorms><<<grid, kThreads, kTmaRingBytes + pl_area_bytes(c.pl_cap), stream>>>(dev_frags, c);
    if (only_pass < 0 || only_pass == DD_RDA_PASS_DIRECTION)
        rda_pass_kernel<BF16, kModeDir><<<grid, kThreads, kTmaRingBytes, stream>>>(dev_frags, c);
    if (only_pass < 0 || only_pass == DD_RDA_PASS_APPLY) {
        // The apply pass reads 12 bytes per element and writes 8: with so large a share of writes
        // one CTA per SM with the full ring is the faster shape (as for a write-heavy fused push).
        Common ca = c;
        if (apply_grid != grid) ca.apply_depth = kTmaStages;
        rda_pass_kernel<BF16, kModeApply><<<apply_grid, kThreads, kTmaRingBytes, stream>>>(dev_frags, ca);
    }
    return cudaGetLastError();
}

static size_t round_up8(size_t n) { return (n + 7) / 8 * 8; }

}  // namespace ddm

static int rda_batched_impl(dd_ctx *ctx, const dd_fragment_desc *descs, const uint64_t *push_masks,
                            int P, int M, dd_dtype learner_dtype, float outer_lr, float outer_mu,
                            uint32_t flags, const uint8_t *merge_kinds, dd_merge_record *records,
                            float *scratch, size_t scratch_elems, void *cuda_stream, int only_pass = -1)
{
    int rc = check_common(ctx, M, learner_dtype, outer_lr, outer_mu, flags);
    if (rc != DD_OK) return rc;
    if (flags & DD_DIAG_PER_LEARNER) flags &= ~(uint32_t)DD_DIAG_PER_LEARNER;   // always on for RDA fragments
    if (P < 0 || (P > 0 && !descs)) return DD_ERR_INVALID_ARG;
    if (P > (1 << 20)) return DD_ERR_TOO_LARGE;
    if (P == 0) return DD_OK;
    if (misaligned(scratch)) return DD_ERR_ALIGNMENT;
    cudaStream_t stream = (cudaStream_t)cuda_stream;

    DeviceGuard guard(ctx->device);
    if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice, "cudaSetDevice");

    for (int p = 0; p < P; ++p)
        if (merge_kinds && merge_kinds[p] != DD_MERGE_RDA && merge_kinds[p] != DD_MERGE_AVG) return DD_ERR_INVALID_ARG;
    // The passes hand norms to one another through the records: use the context's
    // own when the caller wants none.
    if (!records) {
        if ((size_t)P > ctx->rda_records_cap) {
            DD_CUDA(ctx, cudaDeviceSynchronize());
            if (ctx->rda_records) cudaFree(ctx->rda_records);
            ctx->rda_records = nullptr;
            ctx->rda_records_cap = 0;
            DD_CUDA(ctx, cudaMalloc(&ctx->rda_records, (size_t)P * sizeof(dd_merge_record)));
            ctx->rda_records_cap = (size_t)P;
        }
        records = ctx->rda_records;
    }

    rc = acquire_slot(ctx, P);
    if (rc != DD_OK) return rc;
    Slot &slot = ctx->slots[ctx->next_slot];
    unsigned long long tile = 0;
    // With few participants everywhere the merge takes two launches (Gram matrix, then the ordinary
    // merge with weights derived from it) and needs no scratch for the mean direction.
    bool use_gram = only_pass < 0 && !(flags & DD_RDA_THREE_PASS);
    bool any_rda = false;
    for (int p = 0; p < P; ++p) {
        const dd_fragment_desc &d = descs[p];
        DevFrag &f = slot.host[p];
        rc = fill_fragment(f, d.global, d.momentum, d.out_bf16, d.learner_ptrs, d.tokens, d.steps,
                           d.quorum_mask, d.K, d.n, M, learner_bytes_of(learner_dtype, d.n));
        if (rc != DD_OK) return rc;
        if (push_masks && push_masks[p]) {      // written by the last launch, after every launch that reads
            rc = set_push(f, d.learner_ptrs, push_masks[p], M, d.n, learner_bytes_of(learner_dtype, d.n));
            if (rc != DD_OK) return rc;
        }
        f.kind = (!merge_kinds || merge_kinds[p] == DD_MERGE_RDA) ? DD_MERGE_RDA : DD_MERGE_AVG;
        if (f.kind == DD_MERGE_RDA) {
            any_rda = true;
            if (f.n_part_host > kGramMaxPart) use_gram = false;
        }
        f.tile_begin = tile;
        tile += tiles_of(d.n);
        f.tile_end = tile;
    }
    use_gram = use_gram && any_rda;

    if (!use_gram) {
        // Scratch for the mean direction: n floats per radial-directional fragment.
        size_t need = 0;
        for (int p = 0; p < P; ++p)
            if (slot.host[p].kind == DD_MERGE_RDA) need += round_up8((size_t)descs[p].n);
        if (scratch) {
            if (scratch_elems < need) return DD_ERR_INVALID_ARG;
        } else if (need > ctx->rda_scratch_cap) {
            DD_CUDA(ctx, cudaDeviceSynchronize());
            if (ctx->rda_scratch) cudaFree(ctx->rda_scratch);
            ctx->rda_scratch = nullptr;
            ctx->rda_scratch_cap = 0;
            DD_CUDA(ctx, cudaMalloc(&ctx->rda_scratch, need * sizeof(float)));
            ctx->rda_scratch_cap = need;
        }
        float *next_scratch = scratch ? scratch : ctx->rda_scratch;
        for (int p = 0; p < P; ++p) {
            const dd_fragment_desc &d = descs[p];
            DevFrag &f = slot.host[p];
            if (f.kind != DD_MERGE_RDA) continue;
            f.scratch = next_scratch;
            next_scratch += round_up8((size_t)d.n);
            const size_t n = (size_t)d.n;
            if (overlaps(f.scratch, 4 * n, d.global, 4 * n) || overlaps(f.scratch, 4 * n, d.momentum, 4 * n) ||
                overlaps(f.scratch, 4 * n, d.out_bf16, 2 * n))
                return DD_ERR_ALIAS;
        }
    } else if ((size_t)P > ctx->gram_cap) {
        DD_CUDA(ctx, cudaDeviceSynchronize());
        if (ctx->gram) cudaFree(ctx->gram);
        ctx->gram = nullptr;
        ctx->gram_cap = 0;
        const size_t cap = P < 64 ? 64 : (size_t)P;
        DD_CUDA(ctx, cudaMalloc(&ctx->gram, cap * kGramPairs * sizeof(double)));
        ctx->gram_cap = cap;
    }

    const bool bf16 = learner_dtype == DD_BF16;
    unsigned long long g = (unsigned long long)ctx->grid[bf16][1];
    if (g > tile) g = tile;
    unsigned long long gg = (unsigned long long)ctx->gram_grid[bf16];
    if (gg > tile) gg = tile;
    Common c;
    c.eta = outer_lr;
    c.mu = outer_mu;
    c.flags = flags & ~(uint32_t)DD_RDA_THREE_PASS;
    c.M = M;
    c.P = P;
    c.total_tiles = tile;
    c.records = records;
    c.nq = kNumScalarDiag + M;
    if (use_gram && c.nq < kGramPairs) c.nq = kGramPairs;
    c.pl_cap = use_gram ? 0 : pl_capacity(slot.host, P, true);
    const size_t widest = ctx->grid[bf16][1] > ctx->gram_grid[bf16] ? ctx->grid[bf16][1] : ctx->gram_grid[bf16];
    rc = ensure_workspace(ctx, (size_t)P, (size_t)c.nq, widest);
    if (rc != DD_OK) return rc;
    c.partials = ctx->partials;
    c.tickets = ctx->tickets;
    c.gram = ctx->gram;

    DD_CUDA(ctx, cudaMemcpyAsync(slot.dev, slot.host, (size_t)P * sizeof(DevFrag),
                                 cudaMemcpyHostToDevice, stream));
    cudaError_t e;
    if (use_gram) {
        int most = 0;                         // participants of the largest radial-directional fragment
        for (int p = 0; p < P; ++p)
            if (slot.host[p].kind == DD_MERGE_RDA && slot.host[p].n_part_host > most) most = slot.host[p].n_part_host;
        const bool packed = most <= kGramPackedMaxPart;
        if (bf16) {
            if (packed) rda_gram_kernel<true, true><<<(unsigned)gg, kGramThreads, kGramRingBytes, stream>>>(slot.dev, c);
            else rda_gram_kernel<true, false><<<(unsigned)gg, kGramThreads, kGramRingBytes, stream>>>(slot.dev, c);
            rda_gram_merge_kernel<true><<<(unsigned)g, kThreads, kTmaRingBytes, stream>>>(slot.dev, c);
        } else {
            if (packed) rda_gram_kernel<false, true><<<(unsigned)gg, kGramThreads, kGramRingBytes, stream>>>(slot.dev, c);
            else rda_gram_kernel<false, false><<<(unsigned)gg, kGramThreads, kGramRingBytes, stream>>>(slot.dev, c);
            rda_gram_merge_kernel<false><<<(unsigned)g, kThreads, kTmaRingBytes, stream>>>(slot.dev, c);
        }
        e = cudaGetLastError();
    } else {
        // Fragments of kind DD_MERGE_AVG get the ordinary merge in the last launch, which wants the
        // ordinary grid: the narrower one is taken only when every fragment is radial-directional.
        bool all_rda = true;
        for (int p = 0; p < P; ++p) all_rda = all_rda && slot.host[p].kind == DD_MERGE_RDA;
        unsigned long long ga = g;
        if (all_rda && (unsigned long long)ctx->sm_count < ga) ga = (unsigned long long)ctx->sm_count;
        e = bf16 ? launch_rda_passes<true>(slot.dev, c, (unsigned)g, (unsigned)ga, stream, only_pass)
                 : launch_rda_passes<false>(slot.dev, c, (unsigned)g, (unsigned)ga, stream, only_pass);
    }
    if (e != cudaSuccess) return cuda_fail(ctx, e, "radial-directional merge launch");
    DD_CUDA(ctx, cudaEventRecord(slot.done, stream));
    slot.used = true;
    ctx->next_slot = (ctx->next_slot + 1) % kSlots;
    return DD_OK;
}

extern "C" int dd_merge_fragments_batched_rda(dd_ctx *ctx, const dd_fragment_desc *descs, int P,
                                              int M, dd_dtype learner_dtype, float outer_lr,
                                              float outer_mu, uint32_t flags,
                                              const uint8_t *merge_kinds, dd_merge_record *records,
                                              float *scratch, size_t scratch_elems,
                                              void *cuda_stream)
{
    return rda_batched_impl(ctx, descs, nullptr, P, M, learner_dtype, outer_lr, outer_mu, flags, merge_kinds,
                            records, scratch, scratch_elems, cuda_stream);
}

extern "C" int dd_merge_fragments_batched_rda_push(dd_ctx *ctx, const dd_fragment_desc *descs,
                                                   const uint64_t *push_masks, int P, int M,
                                                   dd_dtype learner_dtype, float outer_lr,
                                                   float outer_mu, uint32_t flags,
                                                   const uint8_t *merge_kinds, dd_merge_record *records,
                                                   float *scratch, size_t scratch_elems,
                                                   void *cuda_stream)
{
    if (P > 0 && !push_masks) return DD_ERR_INVALID_ARG;
    return rda_batched_impl(ctx, descs, push_masks, P, M, learner_dtype, outer_lr, outer_mu, flags,
                            merge_kinds, records, scratch, scratch_elems, cuda_stream);
}

extern "C" int dd_merge_fragments_batched_rda_pass(dd_ctx *ctx, const dd_fragment_desc *descs,
                                                   const uint64_t *push_masks, int P, int M,
                                                   dd_dtype learner_dtype, float outer_lr,
                                                   float outer_mu, uint32_t flags,
                                                   const uint8_t *merge_kinds, dd_merge_record *records,
                                                   float *scratch, size_t scratch_elems, int pass,
                                                   void *cuda_stream)
{
    if (pass != DD_RDA_PASS_NORMS && pass != DD_RDA_PASS_DIRECTION && pass != DD_RDA_PASS_APPLY)
        return DD_ERR_INVALID_ARG;
    // the passes hand their results over in memory the caller keeps between the calls
    if (P > 0 && (!records || !scratch)) return DD_ERR_INVALID_ARG;
    return rda_batched_impl(ctx, descs, push_masks, P, M, learner_dtype, outer_lr, outer_mu, flags,
                            merge_kinds, records, scratch, scratch_elems, cuda_stream, pass);
}

extern "C" int dd_merge_fragment_rda(dd_ctx *ctx, float *global, float *momentum,
                                     const void *const *learner_ptrs, int M, dd_dtype learner_dtype,
                                     const uint64_t *tokens, const uint64_t *steps,
                                     uint64_t quorum_mask, int K, float outer_lr, float outer_mu,
                                     uint32_t flags, size_t n, void *out_bf16,
                                     dd_merge_record *record, float *scratch, void *cuda_stream)
{
    dd_fragment_desc d;
    d.global = global;
    d.momentum = momentum;
    d.out_bf16 = out_bf16;
    d.learner_ptrs = learner_ptrs;
    d.tokens = tokens;
    d.steps = steps;
    d.quorum_mask = quorum_mask;
    d.K = K;
    d.n = n;
    return dd_merge_fragments_batched_rda(ctx, &d, 1, M, learner_dtype, outer_lr, outer_mu, flags,
                                          nullptr, record, scratch, scratch ? round_up8(n) : 0,
                                          cuda_stream);
}

extern "C" const char *dd_last_cuda_error(const dd_ctx *ctx)
{
    return ctx ? ctx->cuda_err : "";
}

extern "C" int dd_launch_shape(dd_dtype learner_dtype, int participants, int pushed, int with_out_bf16,
                               int *ctas_per_sm, int *ring_slots)
{
    if ((learner_dtype != DD_F32 && learner_dtype != DD_BF16) || participants < 1 ||
        participants > DD_MAX_LEARNERS || pushed < 0 || pushed > DD_MAX_LEARNERS)
        return DD_ERR_INVALID_ARG;
    const bool bf16 = learner_dtype == DD_BF16;
    int ctas = 2, slots = merge_ring_slots(bf16, participants);
    if (pushed > 0) {
        const double esz = bf16 ? 2.0 : 4.0;
        const PushShape shape = push_shape(8.0 + esz * participants, 8.0 + (with_out_bf16 ? 2.0 : 0.0) + esz * pushed);
        ctas = shape.one_cta_per_sm ? 1 : 2;
        slots = shape.ring_depth;
    }
    if (ctas_per_sm) *ctas_per_sm = ctas;
    if (ring_slots) *ring_slots = slots;
    return DD_OK;
}

extern "C" int dd_launch_geometry(const dd_ctx *ctx, dd_dtype learner_dtype, int *grid, int *block,
                                  int *tile)
{
    if (!ctx || (learner_dtype != DD_F32 && learner_dtype != DD_BF16)) return DD_ERR_INVALID_ARG;
    if (grid) *grid = ctx->grid[learner_dtype == DD_BF16][0];
    if (block) *block = kThreads;
    if (tile) *tile = kTileElems;
    return DD_OK;
}
