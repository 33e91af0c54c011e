// dd_broadcast_fragment: the learner side of a syncer update (Algorithm 1 step 3 and
// the appendix "Mixing learner and syncer params"): every selected learner copy
// becomes alpha * theta_m + (1 - alpha) * Theta'.  alpha = 0, the paper's choice,
// is a plain overwrite with the (rounded) global fragment.  One pass: Theta' is
// read once, each selected copy is read (alpha != 0) and written once.
#include <cmath>

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "dd_ctx.h"

namespace ddm {

struct BroadcastArgs {
    const float *theta;
    void *dst[DD_MAX_LEARNERS];
    int count;
    float alpha;
    unsigned long long n;
    int wide;                 // every selected copy starts on a 32-byte boundary
};

__device__ __forceinline__ unsigned bcast_pack_bf16x2(float lo, float hi)
{
    __nv_bfloat162 b = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<unsigned *>(&b);
}

template <bool BF16>
__global__ void __launch_bounds__(256)
broadcast_kernel(const __grid_constant__ BroadcastArgs a)
{
    const unsigned long long nfull = a.n / 8;
    const float alpha = a.alpha, beta = 1.0f - a.alpha;
    const bool mix = alpha != 0.0f;
    unsigned long long done = 0;          // 8-element steps covered by the wide loop
    if (BF16 && !mix && a.wide) {
        // Pure overwrite into 32-byte aligned bf16 copies: 16 elements per thread, one 32-byte store
        // per copy (with many output streams, 1 KB per warp and stream writes ~5 % faster than 512 B)
        const unsigned long long npair = nfull / 2;
        for (unsigned long long pi = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; pi < npair;
             pi += (unsigned long long)gridDim.x * blockDim.x) {
            const uint4 *tp = reinterpret_cast<const uint4 *>(a.theta) + 4 * pi;
            const uint4 t0 = __ldcs(tp), t1 = __ldcs(tp + 1), t2 = __ldcs(tp + 2), t3 = __ldcs(tp + 3);
            const unsigned w0 = bcast_pack_bf16x2(__uint_as_float(t0.x), __uint_as_float(t0.y));
            const unsigned w1 = bcast_pack_bf16x2(__uint_as_float(t0.z), __uint_as_float(t0.w));
            const unsigned w2 = bcast_pack_bf16x2(__uint_as_float(t1.x), __uint_as_float(t1.y));
            const unsigned w3 = bcast_pack_bf16x2(__uint_as_float(t1.z), __uint_as_float(t1.w));
            const unsigned w4 = bcast_pack_bf16x2(__uint_as_float(t2.x), __uint_as_float(t2.y));
            const unsigned w5 = bcast_pack_bf16x2(__uint_as_float(t2.z), __uint_as_float(t2.w));
            const unsigned w6 = bcast_pack_bf16x2(__uint_as_float(t3.x), __uint_as_float(t3.y));
            const unsigned w7 = bcast_pack_bf16x2(__uint_as_float(t3.z), __uint_as_float(t3.w));
            for (int j = 0; j < a.count; ++j)
                asm volatile("st.global.cs.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                             :: "l"(reinterpret_cast<char *>(a.dst[j]) + 32 * pi), "r"(w0), "r"(w1), "r"(w2),
                                "r"(w3), "r"(w4), "r"(w5), "r"(w6), "r"(w7)
                             : "memory");
        }
        done = 2 * npair;
    }
    for (unsigned long long vi = done + (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; vi < nfull;
         vi += (unsigned long long)gridDim.x * blockDim.x) {
        const uint4 *tp = reinterpret_cast<const uint4 *>(a.theta) + 2 * vi;
        const uint4 t0 = __ldcs(tp), t1 = __ldcs(tp + 1);
        const float T[8] = {__uint_as_float(t0.x), __uint_as_float(t0.y), __uint_as_float(t0.z),
                            __uint_as_float(t0.w), __uint_as_float(t1.x), __uint_as_float(t1.y),
                            __uint_as_float(t1.z), __uint_as_float(t1.w)};
        for (int j = 0; j < a.count; ++j) {
            float x[8];
            if (BF16) {
                uint4 *dp = reinterpret_cast<uint4 *>(a.dst[j]) + vi;
                if (mix) {
                    const uint4 r = __ldcs(dp);
                    const unsigned w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        x[2 * k] = fmaf(alpha, __uint_as_float(w[k] << 16), beta * T[2 * k]);
                        x[2 * k + 1] = fmaf(alpha, __uint_as_float(w[k] & 0xffff0000u), beta * T[2 * k + 1]);
                    }
                } else {
#pragma unroll
                    for (int k = 0; k < 8; ++k) x[k] = T[k];
                }
                __stcs(dp, make_uint4(bcast_pack_bf16x2(x[0], x[1]), bcast_pack_bf16x2(x[2], x[3]),
                                      bcast_pack_bf16x2(x[4], x[5]), bcast_pack_bf16x2(x[6], x[7])));
            } else {
                uint4 *dp = reinterpret_cast<uint4 *>(a.dst[j]) + 2 * vi;
                if (mix) {
                    const uint4 r0 = __ldcs(dp), r1 = __ldcs(dp + 1);
                    const float th[8] = {__uint_as_float(r0.x), __uint_as_float(r0.y), __uint_as_float(r0.z),
                                         __uint_as_float(r0.w), __uint_as_float(r1.x), __uint_as_float(r1.y),
                                         __uint_as_float(r1.z), __uint_as_float(r1.w)};
#pragma unroll
                    for (int k = 0; k < 8; ++k) x[k] = fmaf(alpha, th[k], beta * T[k]);
                } else {
#pragma unroll
                    for (int k = 0; k < 8; ++k) x[k] = T[k];
                }
                __stcs(dp, make_uint4(__float_as_uint(x[0]), __float_as_uint(x[1]), __float_as_uint(x[2]),
                                      __float_as_uint(x[3])));
                __stcs(dp + 1, make_uint4(__float_as_uint(x[4]), __float_as_uint(x[5]), __float_as_uint(x[6]),
                                          __float_as_uint(x[7])));
            }
        }
    }
    // ragged end: n mod 8 elements, one per thread of the first CTA
    const unsigned long long e = nfull * 8 + threadIdx.x;
    if (blockIdx.x == 0 && e < a.n) {
        const float T = a.theta[e];
        for (int j = 0; j < a.count; ++j) {
            if (BF16) {
                uint16_t *d = reinterpret_cast<uint16_t *>(a.dst[j]) + e;
                const float x = mix ? fmaf(alpha, __uint_as_float((unsigned)*d << 16), beta * T) : T;
                *d = (uint16_t)(bcast_pack_bf16x2(x, 0.0f) & 0xffffu);
            } else {
                float *d = reinterpret_cast<float *>(a.dst[j]) + e;
                *d = mix ? fmaf(alpha, *d, beta * T) : T;
            }
        }
    }
}

}  // namespace ddm

using namespace ddm;

extern "C" int dd_broadcast_fragment(dd_ctx *ctx, const float *global, void *const *learner_ptrs,
                                     int M, dd_dtype learner_dtype, uint64_t apply_mask, float alpha,
                                     size_t n, void *cuda_stream)
{
    if (!ctx || !learner_ptrs) return DD_ERR_INVALID_ARG;
    if (M > DD_MAX_LEARNERS) return DD_ERR_TOO_MANY_LEARNERS;
    if (M < 1 || (learner_dtype != DD_F32 && learner_dtype != DD_BF16)) return DD_ERR_INVALID_ARG;
    if (!std::isfinite(alpha) || (n > 0 && !global)) return DD_ERR_INVALID_ARG;
    if (((uintptr_t)global & 15u) != 0) return DD_ERR_ALIGNMENT;
    BroadcastArgs a;
    a.theta = global;
    a.count = 0;
    a.alpha = alpha;
    a.n = n;
    a.wide = 1;
    const size_t lb = (learner_dtype == DD_BF16 ? 2u : 4u) * n;
    for (int m = 0; m < M; ++m) {
        if (!((apply_mask >> m) & 1ull)) continue;
        void *p = learner_ptrs[m];
        if (!p && n > 0) return DD_ERR_INVALID_ARG;
        if (((uintptr_t)p & 15u) != 0) return DD_ERR_ALIGNMENT;
        const uintptr_t p0 = (uintptr_t)p, g0 = (uintptr_t)global;
        if (n > 0 && p0 < g0 + 4 * n && g0 < p0 + lb) return DD_ERR_ALIAS;
        if ((uintptr_t)p & 31u) a.wide = 0;
        a.dst[a.count++] = p;
    }
    if (a.count == 0 || n == 0) return DD_OK;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice, "cudaSetDevice");
    unsigned long long blocks = (n / 8 + 255) / 256;
    const unsigned long long cap = (unsigned long long)ctx->sm_count * 8;
    if (blocks > cap) blocks = cap;
    if (blocks == 0) blocks = 1;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    if (learner_dtype == DD_BF16) broadcast_kernel<true><<<(unsigned)blocks, 256, 0, stream>>>(a);
    else broadcast_kernel<false><<<(unsigned)blocks, 256, 0, stream>>>(a);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(ctx, e, "broadcast_kernel launch");
    return DD_OK;
}
