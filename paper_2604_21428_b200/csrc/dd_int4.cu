// int4 compression of outer gradients (appendix "Outer gradients compression") and the
// merge that consumes them.  The paper states that outer gradients are compressed from
// 16 to 4 bits before they are merged but prints no quantiser; this library's reading:
// blocks of 128 consecutive elements, D = Theta - theta in float32, one float32 scale
// max|D| / 7 per block, code = round-half-even(D / scale) clamped to [-7, 7], stored as
// code + 8 in a nibble (even element in the low nibble).
#include <cmath>
#include <cstring>

#include <cuda_runtime.h>

#include "dd_ctx.h"
#include "dd_merge_kernel.cuh"

namespace ddm {

constexpr int kInt4Block = DD_INT4_BLOCK;     // elements per scale
constexpr int kQuantUnroll = 4;               // blocks a warp of the quantiser loads before it reduces
#ifndef DD_INT4_BATCH
#define DD_INT4_BATCH 8
#endif
constexpr int kInt4Batch = DD_INT4_BATCH;                 // participants whose loads a thread keeps in flight

// ---- learner side: quantise Theta - theta ---------------------------------------------
//
// One warp per block of 128 elements, 4 consecutive elements per lane: the block
// maximum is a warp-shuffle reduction, every lane packs its 4 codes into 16 bits.
template <bool BF16>
__global__ void __launch_bounds__(256)
quantize_int4_kernel(const float *__restrict__ theta, const void *__restrict__ learner,
                     unsigned long long n, unsigned char *__restrict__ codes, float *__restrict__ scales)
{
    const int lane = threadIdx.x & 31;
    const bool vec_ok = (((unsigned long long)theta | (unsigned long long)learner) & 15ull) == 0;
    const unsigned long long nblocks = (n + kInt4Block - 1) / kInt4Block;
    const unsigned long long warps = (unsigned long long)gridDim.x * (blockDim.x >> 5);
    unsigned long long b = (unsigned long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    // Whole blocks, kQuantUnroll at a time: every load is issued before the first reduction.
    if (vec_ok) {
        for (; b + (kQuantUnroll - 1) * warps < n / kInt4Block; b += kQuantUnroll * warps) {
            float4 t4[kQuantUnroll];
            float4 l4[kQuantUnroll];
#pragma unroll
            for (int u = 0; u < kQuantUnroll; ++u) {
                const unsigned long long e0 = (b + u * warps) * kInt4Block + 4ull * lane;
                t4[u] = __ldcs(reinterpret_cast<const float4 *>(theta + e0));
                if (BF16) {
                    const uint2 w = __ldcs(reinterpret_cast<const uint2 *>(
                        reinterpret_cast<const uint16_t *>(learner) + e0));
                    l4[u] = make_float4(__uint_as_float(w.x << 16), __uint_as_float(w.x & 0xffff0000u),
                                        __uint_as_float(w.y << 16), __uint_as_float(w.y & 0xffff0000u));
                } else {
                    l4[u] = __ldcs(reinterpret_cast<const float4 *>(
                        reinterpret_cast<const float *>(learner) + e0));
                }
            }
#pragma unroll
            for (int u = 0; u < kQuantUnroll; ++u) {
                const float d[4] = {__fsub_rn(t4[u].x, l4[u].x), __fsub_rn(t4[u].y, l4[u].y),
                                    __fsub_rn(t4[u].z, l4[u].z), __fsub_rn(t4[u].w, l4[u].w)};
                // The block maximum is taken on the bit patterns of |d|: they order like the values, and
                // a NaN (pattern above infinity's) wins, so a block that holds a NaN gets a NaN scale.
                const unsigned amax_bits = max(max(__float_as_uint(fabsf(d[0])), __float_as_uint(fabsf(d[1]))),
                                               max(__float_as_uint(fabsf(d[2])), __float_as_uint(fabsf(d[3]))));
                const float amax = __uint_as_float(__reduce_max_sync(0xffffffffu, amax_bits));
                const float scale = __fdiv_rn(amax, 7.0f);
                if (lane == 0) scales[b + u * warps] = scale;
                // round(d / scale) without a division per element: q0 = d * (1 / scale) is within
                // 1.1e-6 of the correctly rounded quotient (|quotient| <= 7), so both round to the same
                // integer unless q0 is that close to a half-integer; those elements, and blocks whose
                // scale is so small or large that the reciprocal leaves the normal range, take the
                // exact division.  The codes equal rint(fdiv(d, scale)) in every case.
                const bool fast = scale >= 1e-30f && scale <= 1e30f;
                const float rcp = __frcp_rn(scale);
                float q[4];
                bool exact = !fast;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const float q0 = d[k] * rcp;
                    q[k] = rintf(q0);
                    exact |= !(fabsf(q0 - q[k]) <= 0.5f - 4e-6f);
                }
                if (exact) {
#pragma unroll
                    for (int k = 0; k < 4; ++k) q[k] = scale > 0.0f ? rintf(__fdiv_rn(d[k], scale)) : 0.0f;
                }
                unsigned packed = 0;
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    packed |= (unsigned)((int)fminf(fmaxf(q[k], -7.0f), 7.0f) + 8) << (4 * k);
                *reinterpret_cast<unsigned short *>(codes + ((b + u * warps) * kInt4Block + 4ull * lane) / 2) =
                    (unsigned short)packed;
            }
        }
    }
    // the remaining blocks (and every block when the inputs are not 16-byte aligned), one at a time
    for (; b < nblocks; b += warps) {
        const unsigned long long e0 = b * kInt4Block + 4ull * lane;
        float d[4], T[4], th[4];
        unsigned amax_bits = 0u;
        if (vec_ok && e0 + 3 < n) {
            // 16 bytes of Theta and 8 (bf16) or 16 (fp32) bytes of the learner copy per lane
            const float4 t4 = __ldcs(reinterpret_cast<const float4 *>(theta + e0));
            T[0] = t4.x; T[1] = t4.y; T[2] = t4.z; T[3] = t4.w;
            if (BF16) {
                const uint2 w = __ldcs(reinterpret_cast<const uint2 *>(
                    reinterpret_cast<const uint16_t *>(learner) + e0));
                th[0] = __uint_as_float(w.x << 16); th[1] = __uint_as_float(w.x & 0xffff0000u);
                th[2] = __uint_as_float(w.y << 16); th[3] = __uint_as_float(w.y & 0xffff0000u);
            } else {
                const float4 l4 = __ldcs(reinterpret_cast<const float4 *>(
                    reinterpret_cast<const float *>(learner) + e0));
                th[0] = l4.x; th[1] = l4.y; th[2] = l4.z; th[3] = l4.w;
            }
        } else {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const unsigned long long e = e0 + k;
                T[k] = th[k] = 0.0f;
                if (e < n) {
                    T[k] = theta[e];
                    th[k] = BF16 ? __uint_as_float((unsigned)reinterpret_cast<const uint16_t *>(learner)[e] << 16)
                                 : reinterpret_cast<const float *>(learner)[e];
                }
            }
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            d[k] = __fsub_rn(T[k], th[k]);
            amax_bits = max(amax_bits, __float_as_uint(fabsf(d[k])));     // NaN wins, as above
        }
        const float amax = __uint_as_float(__reduce_max_sync(0xffffffffu, amax_bits));
        const float scale = __fdiv_rn(amax, 7.0f);
        if (lane == 0) scales[b] = scale;
        unsigned packed = 0;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            float q = scale > 0.0f ? rintf(__fdiv_rn(d[k], scale)) : 0.0f;
            q = fminf(fmaxf(q, -7.0f), 7.0f);
            packed |= (unsigned)((int)q + 8) << (4 * k);
        }
        // two bytes per lane; a ragged block writes only the bytes that hold elements
        const unsigned long long byte0 = e0 / 2;
        if (e0 + 3 < n) {
            *reinterpret_cast<unsigned short *>(codes + byte0) = (unsigned short)packed;
        } else if (e0 < n) {
            const unsigned long long left = n - e0;                 // 1..3 elements
            codes[byte0] = (unsigned char)(left >= 2 ? (packed & 0xffu) : (packed & 0x0fu));
            if (left == 3) codes[byte0 + 1] = (unsigned char)((packed >> 8) & 0x0fu);
        }
    }
}


// ---- syncer side: the merge with compressed outer gradients ------------------------------
//
// Delta = sum_j w_hat_j (code_j - 8) scale_j, then the usual outer step.  Participation
// and weights come from the same header code as every other merge.  A thread owns 16
// consecutive elements: 8 bytes of codes and one (block-shared) scale per participant,
// 64 bytes each of Theta and v.  Bytes per parameter: s (1/2 + 4/128) + 16.
struct ScalePtrs {
    const float *p[DD_MAX_LEARNERS];
};

// The element loop of the int4 merge.  WIDE: Theta and v start on 32-byte boundaries and are
// read and written with 256-bit accesses (two 128-bit ones otherwise).
template <bool WIDE>
__device__ __forceinline__ void int4_elements(Smem &sm, const float *const *sptr, const Common &c)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned long long n = sm.n;
    const unsigned long long nfull = n / 16;                      // whole 16-element steps
    const int s = sm.n_part;
    const float eta = c.eta, mu = c.mu;
    const bool heavy = (c.flags & DD_HEAVY_BALL) != 0;
    double a_d = 0.0, a_t = 0.0, a_m = 0.0;
    const float2 minus_c = make_float2(-8388616.0f, -8388616.0f);     // -(2^23 + 8)
    for (unsigned long long vi = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; vi < nfull;
         vi += (unsigned long long)gridDim.x * blockDim.x) {
        float2 acc[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) acc[k] = make_float2(0.0f, 0.0f);
        const unsigned long long blk = vi / (kInt4Block / 16);
        // kInt4Batch participants at a time: all their loads are issued before the first is used
#pragma unroll 1
        for (int j0 = 0; j0 < s; j0 += kInt4Batch) {
            uint2 words[kInt4Batch];
            float ws[kInt4Batch];
#pragma unroll
            for (int b = 0; b < kInt4Batch; ++b) {
                if (j0 + b < s) {
                    words[b] = __ldcs(reinterpret_cast<const uint2 *>(sm.ptr[j0 + b]) + vi);
                    ws[b] = __ldg(sptr[j0 + b] + blk);
                }
            }
#pragma unroll
            for (int b = 0; b < kInt4Batch; ++b) {
                if (j0 + b < s) {
                    const float w = sm.w[j0 + b] * ws[b];
                    const float2 ws2 = make_float2(w, w);
                    // nibble -> float without integer conversions: even nibbles in the bytes of `lo`,
                    // odd ones in `hi`; a byte permute drops each under the exponent of 2^23, giving
                    // 2^23 + code + 8, and one packed add removes 2^23 + 8.
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const unsigned word = h ? words[b].y : words[b].x;
                        const unsigned lo = word & 0x0f0f0f0fu, hi = (word >> 4) & 0x0f0f0f0fu;
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const float2 m = make_float2(
                                __uint_as_float(__byte_perm(lo, 0x4b000000u, 0x7650u + k)),
                                __uint_as_float(__byte_perm(hi, 0x4b000000u, 0x7650u + k)));
                            acc[4 * h + k] = __ffma2_rn(ws2, __fadd2_rn(m, minus_c), acc[4 * h + k]);
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const unsigned v8 = (unsigned)(2 * vi + h);            // index of the 8-element half
            float T[8], V[8];
            load_f32x8<WIDE>(sm.theta, v8, T);
            load_f32x8<WIDE>(sm.mom, v8, V);
            float dsq = 0.0f, tsq = 0.0f, msq = 0.0f;
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const float delta = (k & 1) ? acc[4 * h + (k >> 1)].y : acc[4 * h + (k >> 1)].x;
                const float vn = fmaf(mu, V[k], delta);
                const float u = heavy ? vn : fmaf(mu, vn, delta);
                const float tn = fmaf(-eta, u, T[k]);
                V[k] = vn;
                T[k] = tn;
                dsq = fmaf(delta, delta, dsq);
                tsq = fmaf(tn, tn, tsq);
                msq = fmaf(vn, vn, msq);
            }
            store_f32x8<WIDE>(sm.mom, v8, V);
            store_f32x8<WIDE>(sm.theta, v8, T);
            if (sm.out_bf16 != nullptr)
                st_stream16(reinterpret_cast<uint4 *>(sm.out_bf16) + v8,
                            make_uint4(pack_bf16x2(T[0], T[1]), pack_bf16x2(T[2], T[3]),
                                       pack_bf16x2(T[4], T[5]), pack_bf16x2(T[6], T[7])));
            a_d += (double)dsq;
            a_t += (double)tsq;
            a_m += (double)msq;
        }
    }
    // the ragged end (n mod 16 elements): one element per thread of the first CTA
    if (blockIdx.x == 0 && 16 * nfull + threadIdx.x < n) {
        const unsigned long long e = 16 * nfull + threadIdx.x;
        float delta = 0.0f;
        for (int j = 0; j < s; ++j) {
            const unsigned byte = reinterpret_cast<const unsigned char *>(sm.ptr[j])[e / 2];
            const int code = (int)((byte >> (4 * (e & 1))) & 15u) - 8;
            delta = fmaf(sm.w[j] * sptr[j][e / kInt4Block], (float)code, delta);
        }
        const float vn = fmaf(mu, sm.mom[e], delta);
        const float u = heavy ? vn : fmaf(mu, vn, delta);
        const float tn = fmaf(-eta, u, sm.theta[e]);
        sm.mom[e] = vn;
        sm.theta[e] = tn;
        if (sm.out_bf16 != nullptr) sm.out_bf16[e] = (uint16_t)(pack_bf16x2(tn, 0.0f) & 0xffffu);
        a_d += (double)delta * delta;
        a_t += (double)tn * tn;
        a_m += (double)vn * vn;
    }
    if (c.records != nullptr) {
        a_d = warp_sum(a_d);
        a_t = warp_sum(a_t);
        a_m = warp_sum(a_m);
        if (lane == 0) { sm.red[warp][0] = a_d; sm.red[warp][1] = a_t; sm.red[warp][2] = a_m; }
        flush_fragment<false>(sm, c);
    }
}

#ifndef DD_INT4_MINB
#define DD_INT4_MINB 3
#endif
__global__ void __launch_bounds__(256, DD_INT4_MINB)
merge_int4_kernel(const __grid_constant__ DevFrag frag, const __grid_constant__ ScalePtrs sp,
                  const __grid_constant__ Common c)
{
    __shared__ Smem sm;
    __shared__ const float *sptr[DD_MAX_LEARNERS];
    const int lane = threadIdx.x & 31;
    if (threadIdx.x < 32) {
        load_header<kModeMerge>(&frag, 0, blockIdx.x, c, sm);
        __syncwarp();
        for (int j = lane; j < sm.n_part; j += 32) sptr[j] = sp.p[sm.idx[j]];
    }
    __syncthreads();
    if (sm.status != DD_STATUS_OK) return;

    if (sm.wide) int4_elements<true>(sm, sptr, c);
    else int4_elements<false>(sm, sptr, c);
}

}  // namespace ddm

using namespace ddm;

extern "C" int dd_quantize_outer_gradient_int4(dd_ctx *ctx, const float *global, const void *learner,
                                               dd_dtype learner_dtype, size_t n, uint8_t *codes,
                                               float *scales, void *cuda_stream)
{
    if (!ctx || (learner_dtype != DD_F32 && learner_dtype != DD_BF16)) return DD_ERR_INVALID_ARG;
    if (n == 0) return DD_OK;
    if (!global || !learner || !codes || !scales) return DD_ERR_INVALID_ARG;
    if (((uintptr_t)codes & 1u) || ((uintptr_t)scales & 3u) || ((uintptr_t)global & 3u)) return DD_ERR_ALIGNMENT;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice, "cudaSetDevice");
    const unsigned long long nblocks = (n + kInt4Block - 1) / kInt4Block;
    unsigned long long grid = (nblocks + 7) / 8;
    const unsigned long long cap = (unsigned long long)ctx->sm_count * 8;
    if (grid > cap) grid = cap;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    if (learner_dtype == DD_BF16)
        quantize_int4_kernel<true><<<(unsigned)grid, 256, 0, stream>>>(global, learner, n, codes, scales);
    else
        quantize_int4_kernel<false><<<(unsigned)grid, 256, 0, stream>>>(global, learner, n, codes, scales);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(ctx, e, "quantize_int4_kernel launch");
    return DD_OK;
}

extern "C" int dd_merge_fragment_int4(dd_ctx *ctx, float *global, float *momentum,
                                      const uint8_t *const *code_ptrs, const float *const *scale_ptrs,
                                      int M, const uint64_t *tokens, const uint64_t *steps,
                                      uint64_t quorum_mask, int K, float outer_lr, float outer_mu,
                                      uint32_t flags, size_t n, void *out_bf16,
                                      dd_merge_record *record, void *cuda_stream)
{
    int rc = check_common(ctx, M, DD_BF16, outer_lr, outer_mu, flags);
    if (rc != DD_OK) return rc;
    if (flags & (DD_DIAG_PER_LEARNER | DD_DEBUG_EXPIRE_WAIT)) return DD_ERR_INVALID_ARG;
    if (!code_ptrs || !scale_ptrs) return DD_ERR_INVALID_ARG;
    DevFrag frag;
    rc = fill_fragment(frag, global, momentum, out_bf16, reinterpret_cast<const void *const *>(code_ptrs),
                       tokens, steps, quorum_mask, K, n, M, (n + 1) / 2);
    if (rc != DD_OK) return rc;
    ScalePtrs sp;
    std::memset(&sp, 0, sizeof sp);
    for (int m = 0; m < M; ++m) {
        sp.p[m] = scale_ptrs[m];
        const bool takes_part = ((frag.mask >> m) & 1ull) && tokens[m] > 0;
        if (takes_part && n > 0) {
            if (!scale_ptrs[m]) return DD_ERR_INVALID_ARG;
            if ((uintptr_t)scale_ptrs[m] & 3u) return DD_ERR_ALIGNMENT;
        }
    }
    if (n == 0 && record == nullptr) return DD_OK;

    DeviceGuard guard(ctx->device);
    if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice, "cudaSetDevice");
    const unsigned long long nvec = (n + 15) / 16;
    unsigned long long grid = (nvec + 255) / 256;
    const unsigned long long cap = (unsigned long long)ctx->sm_count * DD_INT4_MINB;   // resident CTAs of 256 threads per SM
    if (grid > cap) grid = cap;
    if (grid == 0) grid = 1;
    frag.tile_begin = 0;
    frag.tile_end = grid;               // every CTA reports its partial sums exactly once
    Common c;
    c.eta = outer_lr;
    c.mu = outer_mu;
    c.flags = flags;
    c.M = M;
    c.P = 1;
    c.total_tiles = grid;
    c.records = record;
    c.nq = kNumScalarDiag;
    if (record) {
        rc = ensure_workspace(ctx, 1, (size_t)c.nq, (size_t)cap);
        if (rc != DD_OK) return rc;
    }
    c.partials = ctx->partials;
    c.tickets = ctx->tickets;
    merge_int4_kernel<<<(unsigned)grid, 256, 0, (cudaStream_t)cuda_stream>>>(frag, sp, c);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(ctx, e, "merge_int4_kernel launch");
    return DD_OK;
}
