// First launch of the two-launch radial-directional merge (Appendix "Merging methods").
//
// With D_j = Theta - theta_j the merge needs ||D_j|| for every participant and the length
// of the mean direction u = sum_j a_j D_j, a_j = w_hat_j / ||D_j||.  Both follow from the
// s x s Gram matrix G_jk = <D_j, D_k>:  ||D_j||^2 = G_jj and ||u||^2 = a^T G a.  So one pass
// that reads Theta and the s copies once and accumulates the s (s + 1) / 2 products is
// enough; the second launch is then the ordinary fused merge with the weights
// c a_j, c = (sum_j w_hat_j ||D_j||) / ||u||, and the mean direction is never stored.
// Bytes per parameter: (s b + 4) + (s b + 16) instead of 2 (s b + 4) + 24 for the
// three-launch form.  The products run on the CUDA cores, which is why this path is taken
// for at most kGramMaxPart participants (36 fused multiply-adds per element at 8).
//
// Data movement: the products need every participant's values of the SAME elements at the
// same time, so the staging is CTA-wide here: a stage holds one sub-tile (1024 elements of
// bf16 copies, 512 of fp32 ones) of Theta and of every participant, filled by a producer
// warp with bulk asynchronous copies (one 2 KB piece per participant) and consumed by the
// eight other warps.  The ring is cut into as many stages as fit (three at 8 participants,
// eight at 2).  Full / empty mbarriers per stage; every wait has an iteration limit.
#pragma once

#include "dd_merge_tma.cuh"

#ifndef DD_GRAM_RING_KB
#define DD_GRAM_RING_KB 64
#endif

namespace ddm {

constexpr int kGramMaxPart = DD_RDA_GRAM_MAX_PARTICIPANTS;
constexpr int kGramPairs = kGramMaxPart * (kGramMaxPart + 1) / 2;
constexpr int kGramMaxStages = 8;                                 // stages the ring is cut into at most
constexpr int kGramThreads = kThreads + 32;                       // eight consumer warps and the producer warp
constexpr size_t kGramRingBytes = (size_t)DD_GRAM_RING_KB * 1024; // stages of Theta sub-tile + one piece per participant
constexpr int kGramFlushTiles = 128;                              // tiles a thread sums in fp32 before the fp64 hand-over

__device__ __forceinline__ void mbar_arrive(unsigned bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(bar) : "memory");
}

// Index of the pair (j, k), k <= j, in the packed lower triangle.
__host__ __device__ constexpr int gram_index(int j, int k) { return j * (j + 1) / 2 + k; }

struct GramShared {
    double acc[kWarps][kGramPairs];      // per-warp fp64 sums of this fragment
    int dead;                            // a bounded wait ran out somewhere in this CTA: nothing more is staged
};

// Per-CTA partial sums -> ticket -> fixed-order final reduce of the Gram matrix of fragment
// sm.frag (the same wait-free scheme as flush_fragment); every thread of the CTA calls it.
__device__ __forceinline__ void flush_gram(Smem &sm, GramShared &gs, const Common &c)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned G = gridDim.x;
    const int p = sm.frag, s = sm.n_part;
    const int npairs = s * (s + 1) / 2;
    __syncthreads();
    double *part = c.partials + (size_t)p * c.nq * G;
    if ((int)threadIdx.x < npairs) {
        double t = 0.0;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) t += gs.acc[w][threadIdx.x];
        part[(size_t)threadIdx.x * G + blockIdx.x] = t;
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
    for (int q = warp; q < npairs; q += kGramThreads / 32) {
        double t = 0.0;
        for (unsigned cta = lane; cta < G; cta += 32) {
            const unsigned off = cta >= first ? cta - first : cta + G - first;
            if (off < ntiles) t += __ldcg(part + (size_t)q * G + cta);
        }
        t = warp_sum(t);
        if (lane == 0) c.gram[(size_t)p * kGramPairs + q] = t;
    }
    __syncthreads();
    // the diagonal is the participants' squared norms: the record's per-learner diagnostics
    if ((int)threadIdx.x < s) rec->delta_m_sq[threadIdx.x] = c.gram[(size_t)p * kGramPairs + gram_index(threadIdx.x, threadIdx.x)];
    if (threadIdx.x == 0) {
        if (sm.any_failed) rec->status = DD_STATUS_WAIT_LIMIT;
        c.tickets[p] = 0u;
    }
}

// One consumer warp's share of a fragment: every stage of this CTA's tiles.  A thread owns four
// (bf16) or two (fp32) consecutive elements of every sub-tile and accumulates every pair's product.
// SMAX is the largest participant count the instance handles.  Up to kGramPackedMaxPart the sums
// are kept per even / odd element in register pairs and every product is one packed
// multiply-add (fma.rn.f32x2): half the arithmetic instructions, 2 x 21 accumulator registers at 6
// participants; the 2 x 36 of 8 participants do not fit beside the operands, so above that the
// sums are scalars.
constexpr int kGramPackedMaxPart = 6;
template <bool BF16, int SMAX>
__device__ __forceinline__ void gram_consume(Smem &sm, GramShared &gs, unsigned long long tile,
                                             unsigned long long mine, const unsigned char *stage_base,
                                             unsigned full_s, unsigned empty_s, int nst, unsigned stage_bytes,
                                             unsigned &phase_bits, bool &failed)
{
    constexpr bool PACKED = SMAX <= kGramPackedMaxPart;
    constexpr int E = BF16 ? 1024 : 512;               // elements per sub-tile: 2 KB of every copy
    constexpr int EPT = E / kThreads;                  // elements per consumer thread: 4 or 2
    constexpr int NP = EPT / 2;                        // pairs of elements per consumer thread
    constexpr int NPAIRS = SMAX * (SMAX + 1) / 2;
    constexpr int NACC = PACKED ? 2 * NPAIRS : NPAIRS; // floats of accumulators
    const unsigned G = gridDim.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int s = sm.n_part;
    const unsigned long long nelems = (sm.n / kVec) * kVec;
    const unsigned long long tile_end = sm.tile_end;
    const unsigned my = (unsigned)threadIdx.x * EPT;   // first element of this thread within a sub-tile
    float acc[NACC];                                   // PACKED: acc[2 q] even elements, acc[2 q + 1] odd ones
#pragma unroll
    for (int q = 0; q < NACC; ++q) acc[q] = 0.0f;
    auto hand_over = [&]() {                           // per-thread fp32 sums -> per-warp fp64 sums
#pragma unroll
        for (int j = 0; j < SMAX; ++j)
#pragma unroll
            for (int k = 0; k <= j; ++k) {
                const int q = gram_index(j, k);
                if (j < s) {
                    const float t = warp_sum(PACKED ? acc[2 * q] + acc[2 * q + 1] : acc[q]);
                    if (lane == 0) gs.acc[warp][q] += (double)t;
                }
                if (PACKED) acc[2 * q] = acc[2 * q + 1] = 0.0f;
                else acc[q] = 0.0f;
            }
    };
    int slot = 0, tiles_summed = 0;
    // 32-bit loop state (a fragment has at most 2^31 8-element steps, 2^21 tiles): the accumulators
    // and operands leave few registers
    constexpr unsigned kTileSteps = kTileElems / kVec;
    const unsigned nsteps = (unsigned)(sm.n / kVec);
    const unsigned ntiles = (unsigned)(tile_end - sm.tile_begin);
    for (unsigned tr = (unsigned)(tile - sm.tile_begin); tr < ntiles && !failed; tr += G) {
        // elements of this tile that go through the stages (the fragment's last tile may be short)
        const unsigned left = nsteps - tr * kTileSteps;
        const unsigned in_tile = (left < kTileSteps ? left : kTileSteps) * (unsigned)kVec;
        for (unsigned first = 0; first < in_tile; first += E) {
            const unsigned cnt = in_tile - first < (unsigned)E ? in_tile - first : (unsigned)E;
            const bool ok = mbar_wait_bounded(full_s + 8u * slot, (phase_bits >> slot) & 1u);
            if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
            const unsigned char *st = stage_base + (size_t)slot * stage_bytes;
            if (my < cnt) {
                float2 nT[NP], D[SMAX][NP];            // -Theta and the outer gradients, two elements per pair
                if (BF16) {
                    const float4 t4 = *reinterpret_cast<const float4 *>(st + threadIdx.x * 16);
                    nT[0] = make_float2(-t4.x, -t4.y);
                    nT[NP - 1] = make_float2(-t4.z, -t4.w);
                } else {
                    const float2 t2 = *reinterpret_cast<const float2 *>(st + threadIdx.x * 8);
                    nT[0] = make_float2(-t2.x, -t2.y);
                }
#pragma unroll
                for (int j = 0; j < SMAX; ++j) {
                    if (j < s) {
                        const uint2 x = *reinterpret_cast<const uint2 *>(st + E * 4 + j * kTmaChunk + threadIdx.x * 8);
                        if (BF16) {
                            D[j][0] = __fadd2_rn(make_float2(__uint_as_float(x.x << 16), __uint_as_float(x.x & 0xffff0000u)), nT[0]);
                            D[j][NP - 1] = __fadd2_rn(make_float2(__uint_as_float(x.y << 16), __uint_as_float(x.y & 0xffff0000u)), nT[NP - 1]);
                        } else {
                            D[j][0] = __fadd2_rn(make_float2(__uint_as_float(x.x), __uint_as_float(x.y)), nT[0]);
                        }
#pragma unroll
                        for (int k = 0; k <= j; ++k) {
                            const int q = gram_index(j, k);
                            if (PACKED) {
                                float2 a2 = make_float2(acc[2 * q], acc[2 * q + 1]);
#pragma unroll
                                for (int e = 0; e < NP; ++e) a2 = __ffma2_rn(D[j][e], D[k][e], a2);
                                acc[2 * q] = a2.x;
                                acc[2 * q + 1] = a2.y;
                            } else {
                                float a = acc[q];
#pragma unroll
                                for (int e = 0; e < NP; ++e) {
                                    a = fmaf(D[j][e].x, D[k][e].x, a);
                                    a = fmaf(D[j][e].y, D[k][e].y, a);
                                }
                                acc[q] = a;
                            }
                        }
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty_s + 8u * slot);
            phase_bits ^= 1u << slot;
            if (++slot == nst) slot = 0;
        }
        if (++tiles_summed == kGramFlushTiles) { hand_over(); tiles_summed = 0; }
    }
    // the ragged end of the fragment (n mod 8 elements): one element per lane of warp 0 of the CTA
    // that owns the last tile
    const int rem = (int)(sm.n % kVec);
    if (rem != 0 && warp == 0 && tile + (mine - 1) * G == tile_end - 1 && lane < rem && !failed) {
        const unsigned long long e = nelems + lane;
        const float T = sm.theta[e];
        float D[SMAX];
#pragma unroll
        for (int j = 0; j < SMAX; ++j) {
            if (j < s) {
                D[j] = (BF16 ? __uint_as_float((unsigned)reinterpret_cast<const uint16_t *>(sm.ptr[j])[e] << 16)
                             : reinterpret_cast<const float *>(sm.ptr[j])[e]) - T;
#pragma unroll
                for (int k = 0; k <= j; ++k) {
                    const int q = PACKED ? 2 * gram_index(j, k) : gram_index(j, k);
                    acc[q] = fmaf(D[j], D[k], acc[q]);
                }
            }
        }
    }
    hand_over();
}

// Two instances.  BOTH = true holds the packed consumer (fragments of up to kGramPackedMaxPart
// participants) and the scalar one (above); the launcher takes it when no fragment of the launch
// has more than kGramPackedMaxPart participants.  BOTH = false holds the scalar consumer alone
// and serves launches with 7 or 8 participants: inside the combined instance the scalar path is
// 10 % slower (registers), while the packed path measured 7 % FASTER there than in an instance of
// its own (same source, another schedule), which is why there is no packed-only instance.
template <bool BF16, bool BOTH>
__global__ void __launch_bounds__(kGramThreads, 2)
rda_gram_kernel(const DevFrag *__restrict__ frags, const __grid_constant__ Common c)
{
    constexpr int E = BF16 ? 1024 : 512;               // elements per sub-tile: 2 KB of every copy
    constexpr int kEsz = BF16 ? 2 : 4;
    __shared__ Smem sm;
    __shared__ GramShared gs;
    __shared__ unsigned long long full_bar[kGramMaxStages], empty_bar[kGramMaxStages];
    extern __shared__ __align__(128) unsigned char stage_base[];
    const unsigned G = gridDim.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const bool producer = warp == kWarps;
    if (threadIdx.x == 0) {
        for (int d = 0; d < kGramMaxStages; ++d) {
            mbar_init(full_bar + d, 1);                // the producer's arrival (plus the bytes it announces)
            mbar_init(empty_bar + d, kWarps);          // one arrival per consumer warp
        }
        gs.dead = 0;
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncthreads();
    const unsigned full_s = smem_addr(full_bar), empty_s = smem_addr(empty_bar), stage_s = smem_addr(stage_base);

    // Every stage barrier completes one phase per use, whatever the number of stages a fragment
    // cuts the ring into: bit d is the parity of barrier d's next use (producer and consumers count
    // alike, each for itself).
    unsigned phase_bits = 0;
    bool failed = false;                               // this warp gave up a bounded wait
    int cur = -1;
    unsigned long long tile = blockIdx.x;
    while (tile < c.total_tiles) {
        __syncthreads();
        if (threadIdx.x < 32) {
            cur = find_frag(frags, cur < 0 ? 0 : cur + 1, c.P, tile);
            load_header<kModeNorms>(frags + cur, cur, tile, c, sm);
        }
        for (int i = threadIdx.x; i < kWarps * kGramPairs; i += kGramThreads) (&gs.acc[0][0])[i] = 0.0;
        __syncthreads();
        cur = sm.frag;
        const unsigned long long tile_end = sm.tile_end;
        const unsigned long long mine = (tile_end - tile + G - 1) / G;
        const int s = sm.n_part;
        const bool worked_on = sm.status == DD_STATUS_OK && sm.kind == DD_MERGE_RDA && s <= kGramMaxPart;
        if (worked_on) {
            // a stage: the Theta sub-tile, then one 2 KB piece per participant; as many stages as fit
            const unsigned stage_bytes = (unsigned)(E * 4 + s * kTmaChunk);
            int nst = (int)(kGramRingBytes / stage_bytes);
            nst = nst > kGramMaxStages ? kGramMaxStages : nst;
            const unsigned long long nelems = (sm.n / kVec) * kVec;       // whole 8-element steps go through the stages
            const bool dead = gs.dead != 0;
            if (dead && threadIdx.x == 0) sm.any_failed = 1;               // an earlier failure leaves this fragment undone
            if (producer) {
                if (lane == 0 && !dead) {
                    const bool expire_hook = (c.flags & DD_DEBUG_EXPIRE_WAIT) != 0;
                    int slot = 0;
                    for (unsigned long long t = tile; t < tile_end && !failed; t += G) {
                        const unsigned long long e0 = (t - sm.tile_begin) * (unsigned long long)kTileElems;
                        const unsigned in_tile = (unsigned)(nelems - e0 < (unsigned long long)kTileElems ? nelems - e0 : kTileElems);
                        const char *theta_t = reinterpret_cast<const char *>(sm.theta + e0);
                        for (unsigned first = 0; first < in_tile && !failed; first += E) {
                            const unsigned cnt = in_tile - first < (unsigned)E ? in_tile - first : (unsigned)E;
                            // the slot is free once every consumer warp has left its previous use
                            if (!mbar_wait_bounded(empty_s + 8u * slot, ((phase_bits >> slot) & 1u) ^ 1u)) { failed = true; break; }
                            const unsigned fb = full_s + 8u * slot;
                            const unsigned dst = stage_s + (unsigned)slot * stage_bytes;
                            // (test hook) announce 16 bytes that no copy delivers: the consumers' wait must expire
                            const unsigned phantom = expire_hook && t == tile && first == 0 ? 16u : 0u;
                            mbar_arrive_expect_tx(fb, cnt * 4u + (unsigned)s * cnt * kEsz + phantom);
                            bulk_copy_g2s(dst, theta_t + first * 4u, cnt * 4u, fb);
                            for (int j = 0; j < s; ++j)
                                bulk_copy_g2s(dst + E * 4u + (unsigned)j * kTmaChunk,
                                              reinterpret_cast<const char *>(sm.ptr[j]) + (e0 + first) * kEsz, cnt * kEsz, fb);
                            phase_bits ^= 1u << slot;
                            if (++slot == nst) slot = 0;
                        }
                    }
                    if (failed) { gs.dead = 1; sm.any_failed = 1; }
                }
                __syncwarp();                            // the producer warp reconverges before the CTA-wide barriers
            } else if (!dead) {
                if (BOTH && s <= kGramPackedMaxPart)
                    gram_consume<BF16, kGramPackedMaxPart>(sm, gs, tile, mine, stage_base, full_s, empty_s, nst, stage_bytes, phase_bits, failed);
                else
                    gram_consume<BF16, kGramMaxPart>(sm, gs, tile, mine, stage_base, full_s, empty_s, nst, stage_bytes, phase_bits, failed);
                if (failed && lane == 0) { gs.dead = 1; sm.any_failed = 1; }
            }
            if (c.records != nullptr) flush_gram(sm, gs, c);
        }
        tile += mine * G;
    }
}

}  // namespace ddm
