// Building blocks of the fused per-fragment merge kernel (sm_100a): participation
// -> weights -> outer gradients -> weighted reduce -> outer optimizer step -> norm
// diagnostics, one pass over HBM.  Algorithm 2 steps 2-3 with the Weight function
// of Section 3.2 and the weighted direct-averaging merge of the "Merging methods"
// appendix.  This file holds the per-fragment header (participation and weights),
// the ragged-tail code and the reduction of the diagnostics; the streaming part
// is in dd_merge_tma.cuh.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "dd_internal.h"

namespace ddm {

// What a launch does with a fragment.  The weighted direct average needs one
// launch (kModeMerge).  Radial-directional averaging ("Merging methods" appendix)
// needs three: per-participant norms, the mean direction u = sum_j (w_j/||D_j||) D_j
// written to a scratch array together with ||u||^2, and the outer step with
// Delta = (sum_j w_j ||D_j||) u / ||u||.
// With few participants two launches are enough: the Gram matrix of the outer gradients
// (dd_rda_gram.cuh), then the ordinary merge with weights derived from it (kModeMergeGram).
enum : int { kModeMerge = 0, kModeNorms = 1, kModeDir = 2, kModeApply = 3, kModeMergeGram = 4 };

// One 2 KB piece of a warp round as the producer lane needs it: where the piece of the row that
// starts at step 0 begins, how many bytes one 8-element step of it takes, which steps of the row it
// covers.  The piece of the row that starts at step v covers steps [first, first + cap) of that row
// and begins at src0 + v * step_bytes.
struct alignas(16) Piece {
    const char *src0;
    unsigned short step_bytes;           // 16 (bf16) or 32 (fp32)
    unsigned short first;                // first step of the row in this piece (0 or 64)
    unsigned short cap;                  // steps of the row in this piece (128 or 64)
    unsigned short pad_;
};
constexpr int kMaxPieces = 2 * DD_MAX_LEARNERS + 4;

struct Smem {
    const void *ptr[DD_MAX_LEARNERS];    // participant j's buffer (compacted)
    double wraw[DD_MAX_LEARNERS];        // raw weights, participant order
    float w[DD_MAX_LEARNERS];            // normalised weights, participant order
    unsigned char idx[DD_MAX_LEARNERS];  // participant j's learner id
    float *theta;
    float *mom;
    uint16_t *out_bf16;
    unsigned long long n;
    unsigned long long tile_begin;
    unsigned long long tile_end;
    int n_part;
    int status;
    int frag;
    int is_last;
    int wide;                            // Theta, v (and scratch) are 32-byte aligned: 256-bit accesses
    int kind;                            // DD_MERGE_AVG / DD_MERGE_RDA of this fragment
    float *scratch;                      // RDA: the mean direction u
    float cscale;                        // RDA apply: Delta = cscale * u
    void *push[DD_MAX_LEARNERS];         // copies that receive Theta' (compacted)
    int n_push;
    int any_failed;                      // a warp of this CTA gave up a bounded wait in (or before) this fragment
    double red[kWarps][kNumScalarDiag];  // per-warp ||Delta||^2, ||Theta'||^2, ||v'||^2 of this fragment
    double dm[kWarps][DD_MAX_LEARNERS];  // per-warp per-participant ||Theta-theta_m||^2
    Piece piece[kMaxPieces];             // the pieces of one warp round, in the order they are consumed
};

// ---- memory access helpers ---------------------------------------------------
//
// Every operand is read once and written once: loads and stores carry the
// streaming (evict-first) hint so that 30+ GB of learner data does not displace
// the state lines that are about to be rewritten.

__device__ __forceinline__ uint4 ld_stream16(const void *p)
{
    return __ldcs(reinterpret_cast<const uint4 *>(p));
}

__device__ __forceinline__ void st_stream16(void *p, uint4 v)
{
    __stcs(reinterpret_cast<uint4 *>(p), v);
}

// 8 consecutive floats (32 bytes).  WIDE: one 256-bit access (needs a 32-byte
// aligned address); otherwise two 128-bit accesses.
template <bool WIDE>
__device__ __forceinline__ void load_f32x8(const float *base, unsigned vi, float (&x)[8])
{
    const float *p = base + 8ull * vi;
    if (WIDE) {
        asm volatile("ld.global.cs.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=f"(x[0]), "=f"(x[1]), "=f"(x[2]), "=f"(x[3]), "=f"(x[4]), "=f"(x[5]),
                       "=f"(x[6]), "=f"(x[7])
                     : "l"(p));
    } else {
        const uint4 a = ld_stream16(p), b = ld_stream16(p + 4);
        x[0] = __uint_as_float(a.x); x[1] = __uint_as_float(a.y);
        x[2] = __uint_as_float(a.z); x[3] = __uint_as_float(a.w);
        x[4] = __uint_as_float(b.x); x[5] = __uint_as_float(b.y);
        x[6] = __uint_as_float(b.z); x[7] = __uint_as_float(b.w);
    }
}

template <bool WIDE>
__device__ __forceinline__ void store_f32x8(float *base, unsigned vi, const float (&x)[8])
{
    float *p = base + 8ull * vi;
    if (WIDE) {
        asm volatile("st.global.cs.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                     :: "l"(p), "f"(x[0]), "f"(x[1]), "f"(x[2]), "f"(x[3]), "f"(x[4]), "f"(x[5]),
                        "f"(x[6]), "f"(x[7])
                     : "memory");
    } else {
        st_stream16(p, make_uint4(__float_as_uint(x[0]), __float_as_uint(x[1]),
                                  __float_as_uint(x[2]), __float_as_uint(x[3])));
        st_stream16(p + 4, make_uint4(__float_as_uint(x[4]), __float_as_uint(x[5]),
                                      __float_as_uint(x[6]), __float_as_uint(x[7])));
    }
}

__device__ __forceinline__ unsigned pack_bf16x2(float lo, float hi)
{
    __nv_bfloat162 b = __floats2bfloat162_rn(lo, hi);     // cvt.rn.bf16x2.f32: .x = lo half
    return *reinterpret_cast<unsigned *>(&b);
}

__device__ __forceinline__ double warp_sum(double x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

__device__ __forceinline__ float warp_sum(float x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

// ---- step 1-2: participation and weights, by warp 0 ---------------------------
//
// S = { m : mask bit m and tokens[m] > 0 } in ascending order (ballot + popc gives
// each member its rank), quorum test |S| >= max(K,1), w = tokens (or
// tokens^2/steps), w_hat = w / sum_S w.  Integer work is exact; the token sum is
// an order-free uint64 butterfly, the tokens^2/steps sum is taken in rank order.
template <int MODE>
__device__ __forceinline__ void load_header(const DevFrag *f, int p, unsigned long long tile,
                                            const Common &c, Smem &sm)
{
    const int lane = threadIdx.x;                 // called by warp 0 only
    const unsigned lt = (1u << lane) - 1u;
    const int M = c.M;
    const unsigned long long mask = f->mask;
    const int m0 = lane, m1 = lane + 32;
    const unsigned long long tok0 = m0 < M ? f->tokens[m0] : 0ull;
    const unsigned long long tok1 = m1 < M ? f->tokens[m1] : 0ull;
    const bool p0 = m0 < M && ((mask >> m0) & 1ull) && tok0 > 0;
    const bool p1 = m1 < M && ((mask >> m1) & 1ull) && tok1 > 0;
    const unsigned b0 = __ballot_sync(0xffffffffu, p0);
    const unsigned b1 = __ballot_sync(0xffffffffu, p1);
    const int c0 = __popc(b0);
    const int n_part = c0 + __popc(b1);
    const int j0 = __popc(b0 & lt), j1 = c0 + __popc(b1 & lt);

    double w0 = 0.0, w1 = 0.0, W;
    if (!f->has_steps) {
        unsigned long long sum = (p0 ? tok0 : 0ull) + (p1 ? tok1 : 0ull);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        W = (double)sum;
        w0 = (double)tok0;
        w1 = (double)tok1;
    } else {
        if (p0) { double t = (double)tok0; w0 = t * t / (double)f->steps[m0]; sm.wraw[j0] = w0; }
        if (p1) { double t = (double)tok1; w1 = t * t / (double)f->steps[m1]; sm.wraw[j1] = w1; }
        __syncwarp();
        W = 0.0;
        if (lane == 0)
            for (int j = 0; j < n_part; ++j) W += sm.wraw[j];
        W = __shfl_sync(0xffffffffu, W, 0);
    }
    const int Kmin = f->K > 1 ? f->K : 1;
    const int status = n_part < Kmin ? DD_STATUS_QUORUM_NOT_MET
                                     : (!(W > 0.0) ? DD_STATUS_ZERO_WEIGHT : DD_STATUS_OK);
    if (p0) { sm.idx[j0] = (unsigned char)m0; sm.w[j0] = (float)(w0 / W); sm.ptr[j0] = f->ptrs[m0]; }
    if (p1) { sm.idx[j1] = (unsigned char)m1; sm.w[j1] = (float)(w1 / W); sm.ptr[j1] = f->ptrs[m1]; }
    // learners that receive Theta' in their own dtype: compacted like the participants
    const unsigned long long pm = f->push_mask;
    const bool q0 = m0 < M && ((pm >> m0) & 1ull), q1 = m1 < M && ((pm >> m1) & 1ull);
    const unsigned pb0 = __ballot_sync(0xffffffffu, q0);
    const unsigned pb1 = __ballot_sync(0xffffffffu, q1);
    if (q0) sm.push[__popc(pb0 & lt)] = const_cast<void *>(f->ptrs[m0]);
    if (q1) sm.push[__popc(pb0) + __popc(pb1 & lt)] = const_cast<void *>(f->ptrs[m1]);
    if (lane == 0) {
        sm.n_push = __popc(pb0) + __popc(pb1);
        sm.theta = f->theta;
        sm.mom = f->mom;
        sm.out_bf16 = f->out_bf16;
        sm.n = f->n;
        sm.tile_begin = f->tile_begin;
        sm.tile_end = f->tile_end;
        sm.n_part = n_part;
        sm.status = status;
        sm.frag = p;
        sm.wide = (((unsigned long long)f->theta | (unsigned long long)f->mom |
                    (unsigned long long)f->scratch) & 31ull) == 0;
        sm.kind = f->kind;
        sm.scratch = f->scratch;
        sm.cscale = 0.0f;
        sm.any_failed = 0;
    }
    for (int j = lane; j < kWarps * DD_MAX_LEARNERS; j += 32) (&sm.dm[0][0])[j] = 0.0;
    if (lane < kWarps * kNumScalarDiag) (&sm.red[0][0])[lane] = 0.0;
    __syncwarp();
    if ((MODE == kModeDir || MODE == kModeApply) && f->kind == DD_MERGE_RDA &&
        status == DD_STATUS_OK) {
        // The norms pass left ||Theta - theta_j||^2 in this fragment's record.
        const dd_merge_record *rec = c.records + p;
        const double n0 = j0 < n_part && p0 ? sqrt(__ldcg(&rec->delta_m_sq[j0])) : 0.0;
        const double n1 = p1 ? sqrt(__ldcg(&rec->delta_m_sq[j1])) : 0.0;
        if (MODE == kModeDir) {
            // direction weights a_j = w_hat_j / ||D_j||; a zero outer gradient has no direction
            if (p0) sm.w[j0] = n0 > 0.0 ? (float)((double)sm.w[j0] / n0) : 0.0f;
            if (p1) sm.w[j1] = n1 > 0.0 ? (float)((double)sm.w[j1] / n1) : 0.0f;
        } else {
            // radial part sum_j w_hat_j ||D_j|| over the mean direction's length
            double radial = (p0 ? (double)sm.w[j0] * n0 : 0.0) + (p1 ? (double)sm.w[j1] * n1 : 0.0);
            radial = warp_sum(radial);
            const double usq = __ldcg(&rec->delta_sq);
            if (lane == 0) sm.cscale = usq > 0.0 ? (float)(radial / sqrt(usq)) : 0.0f;
        }
        __syncwarp();
    }
    if (MODE == kModeMergeGram && f->kind == DD_MERGE_RDA && status == DD_STATUS_OK) {
        // Second launch of the two-launch radial-directional merge: with G the Gram matrix of the
        // outer gradients, ||D_j|| = sqrt(G_jj), a_j = w_hat_j / ||D_j|| (0 for a zero gradient),
        // ||u||^2 = a^T G a, and Delta = sum_j (c a_j) D_j with c = (sum_j w_hat_j ||D_j||) / ||u||:
        // the ordinary merge with other weights.  At most 8 participants: lane j owns participant j.
        const double *g = c.gram + (size_t)p * kGramPairsMax;
        const bool on = lane < n_part;
        const double wj = on ? (double)sm.w[lane] : 0.0;
        const double nj = on ? sqrt(__ldcg(g + lane * (lane + 1) / 2 + lane)) : 0.0;
        const double aj = nj > 0.0 ? wj / nj : 0.0;
        const double radial = warp_sum(wj * nj);
        double row = 0.0;
#pragma unroll
        for (int k = 0; k < DD_RDA_GRAM_MAX_PARTICIPANTS; ++k) {
            const double ak = __shfl_sync(0xffffffffu, aj, k);
            if (on && k < n_part) {
                const int hi = lane > k ? lane : k, lo = lane > k ? k : lane;
                row += ak * __ldcg(g + hi * (hi + 1) / 2 + lo);
            }
        }
        const double usq = warp_sum(on ? aj * row : 0.0);
        const double cs = usq > 0.0 ? radial / sqrt(usq) : 0.0;
        if (on) sm.w[lane] = (float)(cs * aj);
        __syncwarp();
    }
    // The CTA that owns the fragment's first tile publishes the header (once per
    // call: the later passes of a radial-directional merge leave it alone).
    const bool publish = (MODE == kModeMerge || MODE == kModeMergeGram)
                             ? f->kind == DD_MERGE_AVG
                             : (MODE == kModeNorms && f->kind == DD_MERGE_RDA);
    if (publish && c.records != nullptr && tile == f->tile_begin) {
        dd_merge_record *rec = c.records + p;
        for (int j = lane; j < DD_MAX_LEARNERS; j += 32) {
            const bool on = j < n_part && status == DD_STATUS_OK;
            rec->idx[j] = j < n_part ? sm.idx[j] : (unsigned char)0;
            rec->w_hat[j] = on ? sm.w[j] : 0.0f;
            rec->delta_m_sq[j] = 0.0;
        }
        if (lane == 0) {
            rec->status = status;
            rec->n_part = n_part;
            rec->w_total = status == DD_STATUS_QUORUM_NOT_MET ? 0.0 : W;
            rec->delta_sq = 0.0;
            rec->theta_sq = 0.0;
            rec->mom_sq = 0.0;
        }
    }
}

// Smallest fragment index >= lo whose tile range ends after `tile`.
__device__ __forceinline__ int find_frag(const DevFrag *frags, int lo, int P,
                                         unsigned long long tile)
{
    int hi = P - 1;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (tile < frags[mid].tile_end) hi = mid; else lo = mid + 1;
    }
    return lo;
}

// The ragged end of a fragment (n mod 8 elements), one element per lane of warp 0.
template <bool BF16, bool PL, int MODE>
__device__ __forceinline__ void process_tail(Smem &sm, const Common &c, unsigned long long first,
                                             int count, float &dsq, float &tsq, float &msq)
{
    const int lane = threadIdx.x & 31;
    const bool active = lane < count;
    const unsigned long long e = first + lane;
    const int s = sm.n_part;
    const float T = active ? sm.theta[e] : 0.0f;
    float acc = 0.0f;
    if (MODE != kModeApply) {
        for (int j = 0; j < s; ++j) {
            float th = 0.0f;
            if (active) {
                if (BF16) th = __uint_as_float((unsigned)reinterpret_cast<const uint16_t *>(sm.ptr[j])[e] << 16);
                else th = reinterpret_cast<const float *>(sm.ptr[j])[e];
            }
            const float d = th - T;
            acc = fmaf(sm.w[j], d, acc);
            if (PL) {
                const float q = warp_sum(d * d);
                if (lane == 0) sm.dm[0][j] += (double)q;
            }
        }
    }
    if (!active || MODE == kModeNorms) return;
    if (MODE == kModeDir) {
        sm.scratch[e] = -acc;
        dsq = fmaf(acc, acc, dsq);
        return;
    }
    const float delta = MODE == kModeApply ? sm.cscale * sm.scratch[e] : -acc;
    const float vn = fmaf(c.mu, sm.mom[e], delta);
    const float u = (c.flags & DD_HEAVY_BALL) ? vn : fmaf(c.mu, vn, delta);
    const float tn = fmaf(-c.eta, u, T);
    sm.mom[e] = vn;
    sm.theta[e] = tn;
    if (sm.out_bf16 != nullptr) sm.out_bf16[e] = (uint16_t)(pack_bf16x2(tn, 0.0f) & 0xffffu);
    for (int q = 0; q < sm.n_push; ++q) {
        if (BF16) reinterpret_cast<uint16_t *>(sm.push[q])[e] = (uint16_t)(pack_bf16x2(tn, 0.0f) & 0xffffu);
        else reinterpret_cast<float *>(sm.push[q])[e] = tn;
    }
    dsq = fmaf(delta, delta, dsq);
    tsq = fmaf(tn, tn, tsq);
    msq = fmaf(vn, vn, msq);
}

// ---- step 6: per-CTA partials, ticket, fixed-order final reduce ----------------
//
// Wait-free: every CTA that worked on the fragment stores its partial sums and
// draws a ticket (a release-acquire atomic); the CTA that draws the last ticket adds the
// partials in a fixed order (so the result does not depend on CTA timing) and
// re-arms the ticket for the next call.  The ticket word's top bit carries "some
// CTA gave up a bounded wait in this fragment": a CTA sets it before it draws its
// ticket, so the last CTA sees it from every CTA and reports DD_STATUS_WAIT_LIMIT
// after the header (written by the CTA of the fragment's first tile) is in place.
constexpr unsigned kTicketFailedBit = 0x80000000u;

// Ticket draw with release and acquire semantics at GPU scope: everything this CTA wrote before
// the barrier that precedes the call is visible to whoever draws a later ticket and then
// synchronises its own CTA.  One such atomic replaces a fence per writer plus a fence per reader.
__device__ __forceinline__ unsigned ticket_add_acq_rel(unsigned *addr, unsigned val)
{
    unsigned old;
    asm volatile("atom.add.acq_rel.gpu.global.u32 %0, [%1], %2;" : "=r"(old) : "l"(addr), "r"(val) : "memory");
    return old;
}

template <bool PL>
__device__ __forceinline__ void flush_fragment(Smem &sm, const Common &c)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned G = gridDim.x;
    const int s = sm.n_part, p = sm.frag;
    const int nq = c.nq;
    __syncthreads();
    double *part = c.partials + (size_t)p * nq * G;
    if (threadIdx.x < kNumScalarDiag) {
        double t = 0.0;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) t += sm.red[w][threadIdx.x];
        part[(size_t)threadIdx.x * G + blockIdx.x] = t;
    } else if (PL && threadIdx.x >= 32 && threadIdx.x < 32 + s) {
        const int j = threadIdx.x - 32;
        double t = 0.0;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) t += sm.dm[w][j];
        part[(size_t)(kNumScalarDiag + j) * G + blockIdx.x] = t;
    }
    __syncthreads();
    const unsigned long long ntiles = sm.tile_end - sm.tile_begin;
    if (threadIdx.x == 0) {
        const unsigned expected = ntiles < G ? (unsigned)ntiles : G;
        if (sm.any_failed) atomicOr(c.tickets + p, kTicketFailedBit);
        const unsigned ticket = ticket_add_acq_rel(c.tickets + p, 1u);
        sm.is_last = (ticket & ~kTicketFailedBit) == expected - 1u;
        if (ticket & kTicketFailedBit) sm.any_failed = 1;
    }
    __syncthreads();
    if (!sm.is_last) return;
    dd_merge_record *rec = c.records + p;
    const unsigned first = (unsigned)(sm.tile_begin % G);
    const int nq_used = kNumScalarDiag + (PL ? s : 0);
    for (int q = warp; q < nq_used; q += kWarps) {
        double t = 0.0;
        for (unsigned cta = lane; cta < G; cta += 32) {
            const unsigned off = cta >= first ? cta - first : cta + G - first;
            if (off < ntiles) t += __ldcg(part + (size_t)q * G + cta);
        }
        t = warp_sum(t);
        if (lane == 0) {
            if (q == 0) rec->delta_sq = t;
            else if (q == 1) rec->theta_sq = (c.flags & DD_DIAG_STATE) ? t : 0.0;
            else if (q == 2) rec->mom_sq = (c.flags & DD_DIAG_STATE) ? t : 0.0;
            else rec->delta_m_sq[q - kNumScalarDiag] = t;
        }
    }
    if (threadIdx.x == 0) {
        if (sm.any_failed) rec->status = DD_STATUS_WAIT_LIMIT;
        c.tickets[p] = 0u;
    }
}

}  // namespace ddm
