// dd_merge_fragments_batched_noalloc: the batched merge for callers that must
// not allocate.  It needs no dd_ctx and calls no cudaMalloc / cudaFree (nor any
// routine that allocates): the kernel's scratch -- the device copy of the
// fragment descriptors, the per-CTA partial sums of the norm diagnostics and the
// completion tickets -- lives in one fixed array in this library's device image.
//
// Who needs this: a syncer that runs inside a process whose framework allocator
// already owns almost all device memory (a raw cudaMalloc may simply fail there),
// a loop that cannot afford the device-wide synchronisation cudaMalloc and
// cudaFree imply, or a deployment whose policy is "no allocation after start-up".
#include <cmath>
#include <cstring>
#include <mutex>

#include <cuda_runtime.h>

#include "dd_merge_tma.cuh"
#include "dd_ctx.h"

namespace ddm {
namespace noalloc {

constexpr int kMaxFragments = DD_NOALLOC_MAX_FRAGMENTS;
constexpr int kMaxCtas = 592;                         // 4 CTAs on each of 148 SMs
constexpr int kNq = kNumScalarDiag;                   // no per-learner norms here
constexpr int kMaxDevices = 64;

constexpr size_t kFragBytes = sizeof(DevFrag) * kMaxFragments;
constexpr size_t kPartialsOffset = (kFragBytes + 255) / 256 * 256;
constexpr size_t kPartialsBytes = sizeof(double) * kMaxFragments * kNq * kMaxCtas;
constexpr size_t kTicketsOffset = (kPartialsOffset + kPartialsBytes + 255) / 256 * 256;
constexpr size_t kTicketsBytes = sizeof(unsigned) * kMaxFragments;
constexpr size_t kScratchBytes = kTicketsOffset + kTicketsBytes;
static_assert(kScratchBytes <= DD_NOALLOC_SCRATCH_BYTES, "header understates the scratch size");

// The scratch itself.  Every GPU on which this library runs a kernel holds one
// copy until the process exits.  In HOST code this name is only a stand-in for
// the symbol, not a device address: the address comes from cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_scratch[DD_NOALLOC_SCRATCH_BYTES];

__global__ void __launch_bounds__(kThreads, 2)
merge_batched_noalloc_kernel(const DevFrag *__restrict__ frags, const __grid_constant__ Common c)
{
    merge_body_tma<true, kModeMerge, false>(frags, c);
}

__global__ void __launch_bounds__(kThreads, 2)
merge_batched_noalloc_kernel_f32(const DevFrag *__restrict__ frags, const __grid_constant__ Common c)
{
    merge_body_tma<false, kModeMerge, false>(frags, c);
}

struct DeviceState {
    bool ready = false;
    unsigned char *scratch = nullptr;     // device address of g_scratch on this device
    int grid[2] = {0, 0};                 // [bf16] persistent grid size
};

static DeviceState g_state[kMaxDevices];
static std::mutex g_mutex;

// One-time set-up for the CURRENT device: resolve the scratch address and size the
// persistent grid.  Nothing here allocates.
static int setup_current_device(DeviceState **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        (void)cudaGetLastError();
        return DD_ERR_CUDA;
    }
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceState &st = g_state[dev];
    if (!st.ready) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_scratch) != cudaSuccess || ptr == nullptr) {
            (void)cudaGetLastError();
            return DD_ERR_CUDA;
        }
        int sms = 0, occ_bf16 = 0, occ_f32 = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
            // the warps' staging rings live in dynamic shared memory: opt in (this sets a
            // function attribute; it allocates nothing)
            cudaFuncSetAttribute(merge_batched_noalloc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)kTmaRingBytes) != cudaSuccess ||
            cudaFuncSetAttribute(merge_batched_noalloc_kernel_f32, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)kTmaRingBytes) != cudaSuccess ||
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ_bf16, merge_batched_noalloc_kernel,
                                                          kThreads, kTmaRingBytes) != cudaSuccess ||
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ_f32, merge_batched_noalloc_kernel_f32,
                                                          kThreads, kTmaRingBytes) != cudaSuccess) {
            (void)cudaGetLastError();
            return DD_ERR_CUDA;
        }
        if (occ_bf16 > 2) occ_bf16 = 2;              // same launch shape as the ordinary entry points
        if (occ_f32 > 2) occ_f32 = 2;
        const int g1 = sms * (occ_bf16 > 0 ? occ_bf16 : 1), g0 = sms * (occ_f32 > 0 ? occ_f32 : 1);
        st.grid[1] = g1 < kMaxCtas ? g1 : kMaxCtas;
        st.grid[0] = g0 < kMaxCtas ? g0 : kMaxCtas;
        st.scratch = static_cast<unsigned char *>(ptr);
        st.ready = true;
    }
    *out = &st;
    return DD_OK;
}

}  // namespace noalloc
}  // namespace ddm

using namespace ddm;
using namespace ddm::noalloc;

extern "C" int dd_merge_fragments_batched_noalloc(const dd_fragment_desc *descs, int P, int M,
                                                  dd_dtype learner_dtype, float outer_lr,
                                                  float outer_mu, uint32_t flags,
                                                  dd_merge_record *records, void *cuda_stream)
{
    if (M > DD_MAX_LEARNERS) return DD_ERR_TOO_MANY_LEARNERS;
    if (M < 1 || P < 0 || (P > 0 && !descs)) return DD_ERR_INVALID_ARG;
    if (P > kMaxFragments) return DD_ERR_TOO_LARGE;          // the fixed scratch holds no more
    if (learner_dtype != DD_F32 && learner_dtype != DD_BF16) return DD_ERR_INVALID_ARG;
    if (!std::isfinite(outer_lr) || !std::isfinite(outer_mu)) return DD_ERR_INVALID_ARG;
    if (flags & ~(uint32_t)(DD_HEAVY_BALL | DD_DIAG_STATE)) return DD_ERR_INVALID_ARG;
    if (P == 0) return DD_OK;

    DeviceState *st = nullptr;
    int rc = setup_current_device(&st);
    if (rc != DD_OK) return rc;

    // Descriptors are assembled in a buffer of this thread and copied into the
    // scratch; the copy from ordinary host memory is staged by the driver before
    // cudaMemcpyAsync returns, so the buffer may be reused at once.
    static thread_local DevFrag host_frags[kMaxFragments];
    unsigned long long tile = 0;
    for (int p = 0; p < P; ++p) {
        const dd_fragment_desc &d = descs[p];
        rc = fill_fragment(host_frags[p], d.global, d.momentum, d.out_bf16, d.learner_ptrs, d.tokens, d.steps,
                           d.quorum_mask, d.K, d.n, M, (learner_dtype == DD_BF16 ? 2u : 4u) * (size_t)d.n);
        if (rc != DD_OK) return rc;
        host_frags[p].tile_begin = tile;
        const unsigned long long t = (descs[p].n + kTileElems - 1) / kTileElems;
        tile += t ? t : 1;
        host_frags[p].tile_end = tile;
    }

    const bool bf16 = learner_dtype == DD_BF16;
    unsigned long long g = (unsigned long long)st->grid[bf16];
    if (g > tile) g = tile;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    DevFrag *dev_frags = reinterpret_cast<DevFrag *>(st->scratch);
    Common c;
    c.eta = outer_lr;
    c.mu = outer_mu;
    c.flags = flags;
    c.M = M;
    c.P = P;
    c.total_tiles = tile;
    c.records = records;
    c.partials = reinterpret_cast<double *>(st->scratch + kPartialsOffset);
    c.tickets = reinterpret_cast<unsigned *>(st->scratch + kTicketsOffset);
    c.nq = kNq;

    // The array keeps whatever the previous call left: the tickets must start at
    // zero (the partial sums need not: every slot that is read is written first).
    if (cudaMemsetAsync(c.tickets, 0, kTicketsBytes, stream) != cudaSuccess ||
        cudaMemcpyAsync(dev_frags, host_frags, sizeof(DevFrag) * (size_t)P, cudaMemcpyHostToDevice,
                        stream) != cudaSuccess) {
        (void)cudaGetLastError();
        return DD_ERR_CUDA;
    }
    if (bf16)
        merge_batched_noalloc_kernel<<<(unsigned)g, kThreads, kTmaRingBytes, stream>>>(dev_frags, c);
    else
        merge_batched_noalloc_kernel_f32<<<(unsigned)g, kThreads, kTmaRingBytes, stream>>>(dev_frags, c);
    if (cudaGetLastError() != cudaSuccess) return DD_ERR_CUDA;
    return DD_OK;
}
