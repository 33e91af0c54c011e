// The streaming part of the fused merge: operands are staged through shared
// memory by bulk asynchronous copies (cp.async.bulk: the TMA engine, no tensor
// map, every copy addressed to this CTA alone).  A warp owns a private ring of
// kTmaStages slots of 2 KB.  Its lane 0
// asks the copy engine for the next 2 KB piece -- 1024 bf16 elements of one
// learner copy, or 512 floats of Theta / v -- up to kTmaStages-1 pieces ahead of
// the piece the warp is consuming, each piece signalling its own mbarrier.  The
// loads therefore cost neither registers nor load/store-unit slots, and 2 KB
// requests keep HBM streaming with only 16 warps per SM.
//
// Synchronisation is warp-local: lanes wait on the slot's mbarrier (try_wait in
// a loop with an iteration limit; on giving up the warp records
// DD_STATUS_WAIT_LIMIT, waits -- again bounded -- for its copies in flight and
// leaves), and a slot is handed back to lane 0 by __syncwarp().  No CTA-wide
// barrier, no flag shared between CTAs.
#pragma once

#include "dd_merge_kernel.cuh"


namespace ddm {

constexpr int kTmaChunk = 2048;                           // bytes per slot / per bulk copy
constexpr int kSuperRow = 1024;                           // elements a warp merges per round (4 steps per lane)
constexpr size_t kTmaRingBytes = (size_t)kWarps * kTmaStages * kTmaChunk;
constexpr int kPlMaxParticipants = 48;                    // per-lane norm area: 1 KB per participant per CTA
constexpr int kPlFlushRows = 128;                         // rounds a lane sums in fp32 before the fp64 hand-over
constexpr int kWaitLimit = 1 << 18;                       // try_wait attempts before giving up
constexpr unsigned kWaitHintNs = 4000;                    // each attempt may sleep this long (~1 s in all)
static_assert(kTileElems == kWarps * kSuperRow, "one super-row per warp per tile");

__device__ __forceinline__ unsigned smem_addr(const void *p)
{
    return (unsigned)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void mbar_init(unsigned long long *bar, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_addr(bar)), "r"(count) : "memory");
}

// The issuing thread's arrival plus the number of bytes the copies will deliver.
// (These take 32-bit shared-space addresses so that the per-piece code does no
// generic-to-shared conversions.)
__device__ __forceinline__ void mbar_arrive_expect_tx(unsigned bar, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(bar), "r"(bytes) : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(unsigned bar, unsigned parity)
{
    unsigned ok;
    // The attempt suspends the thread until the phase completes or the hint expires.
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n"
                 " selp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(bar), "r"(parity), "r"(kWaitHintNs) : "memory");
    return ok != 0;
}

// Bounded wait for one phase of a slot's barrier.
__device__ __forceinline__ bool mbar_wait_bounded(unsigned bar, unsigned parity)
{
    for (int spins = 0; spins < kWaitLimit; ++spins)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}

// global -> this CTA's shared memory, 16-byte aligned on both sides, bytes % 16 == 0.
__device__ __forceinline__ void bulk_copy_g2s(unsigned dst, const void *src, unsigned bytes, unsigned bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// The same with an L2 eviction-priority hint for the lines the copy brings in.
__device__ __forceinline__ void bulk_copy_g2s_hint(unsigned dst, const void *src, unsigned bytes, unsigned bar,
                                                   unsigned long long policy)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                 :: "r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(policy) : "memory");
}

__device__ __forceinline__ unsigned long long l2_policy_evict_first()
{
    unsigned long long p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}

// With few participants the writes are a large share of the traffic (29 % at 6 participants, 44 % at
// 1) and the launch runs 2-3 % faster when every line read is marked evict-first in L2; from 8
// participants on the same hint costs 9 %, so it is given only below that.
constexpr int kEvictFirstMaxParticipants = 7;

// Ring position of a warp; survives from one fragment to the next (the ring is
// always drained in between, so producer and consumer meet at the same slot).
struct TmaRing {
    int islot = 0;           // next slot to fill
    int cslot = 0;           // next slot to consume
    unsigned phase_bits = 0; // bit d: parity of the phase the consumer waits for on slot d
    bool failed = false;     // a bounded wait gave up
};

// Slots of the ring a fragment uses (one fewer is in flight ahead of the consumer).  Measured on
// B200 at 2 CTAs per SM.  bf16 copies: with one piece in flight per warp (32 KB per SM) the launch
// is 3-7 % faster up to 7 participants, within 1.5 % either way from 8 to 16, and 2-4 % slower
// from 18 on.  fp32 copies: one piece in flight is 1-4 % faster at every count up to 24.  With a
// fused push the host picks the depth together with the grid (push_shape in the launcher).  The
// norms and direction passes of the three-launch radial-directional merge follow the same rule
// (-2 % on three launches at 6 participants); its apply pass, 40 % writes, runs shallow at two
// CTAs per SM and with the full ring when the host launches it with one (a probe of its pattern:
// 6.69 against 6.33 TB/s).  Every slot's barrier has its own phase parity, so the depth may change
// from one fragment to the next (the ring is drained in between).
template <bool BF16, int MODE>
__device__ __forceinline__ int ring_depth(int s, int n_push, const Common &c)
{
    if (kTmaStages < 3) return kTmaStages;
    if (MODE == kModeApply) return c.apply_depth;
    if (n_push > 0) return c.push_depth;
    return merge_ring_slots(BF16, s);
}

// Fills sm.piece for the current fragment (all threads of the CTA; a CTA barrier must follow).
// MODE is the mode the fragment is processed in.  The order is the order of consumption:
//   Theta[0:512) Theta[512:1024) | learner pieces (1 per bf16 copy, 2 per fp32 copy) | v[0:512) v[512:1024)
template <bool BF16, int MODE>
__device__ __forceinline__ void build_piece_table(Smem &sm)
{
    constexpr int LB = BF16 ? 1 : 2;
    constexpr bool kHasV = MODE == kModeMerge || MODE == kModeApply;
    const int nmid = MODE == kModeApply ? 2 : sm.n_part * LB;
    const int npieces = 2 + nmid + (kHasV ? 2 : 0);
    for (int i = threadIdx.x; i < npieces; i += kThreads) {
        Piece pc;
        pc.pad_ = 0;
        if (BF16 && MODE != kModeApply && i >= 2 && i < 2 + nmid) {
            pc.src0 = reinterpret_cast<const char *>(sm.ptr[i - 2]);
            pc.step_bytes = 16;
            pc.first = 0;
            pc.cap = (unsigned short)(kSuperRow / kVec);
        } else {
            // float32 operand (Theta, fp32 learner copy, stored direction, v): two halves of 64 steps
            const int q = i < 2 ? i : (i < 2 + nmid ? i - 2 : i - 2 - nmid);
            const void *base = i < 2 ? (const void *)sm.theta
                             : i >= 2 + nmid ? (const void *)sm.mom
                             : MODE == kModeApply ? (const void *)sm.scratch : sm.ptr[q >> 1];
            pc.first = (unsigned short)(64 * (q & 1));
            pc.src0 = reinterpret_cast<const char *>(base) + 32u * pc.first;
            pc.step_bytes = 32;
            pc.cap = 64;
        }
        sm.piece[i] = pc;
    }
}

// All tiles of the current fragment that belong to this CTA (tile, tile+G, ...):
// warp w merges super-row w of each of them.  Pieces per super-row, in order:
//   Theta[0:512) Theta[512:1024) | learner pieces (1 per bf16 copy, 2 per fp32 copy) | v[0:512) v[512:1024)
// The passes of a radial-directional merge use the same pipeline: the norms and
// direction passes have no v pieces; the apply pass reads the two halves of the
// stored direction u in place of the learner pieces.  PL adds the per-participant
// squared norms of the outer gradients (always on in the norms pass).
template <bool BF16, bool WIDE, int MODE, bool PL>
__device__ __forceinline__ void process_fragment_tma(Smem &sm, const Common &c,
                                                     unsigned long long tile, unsigned char *ring_base,
                                                     unsigned long long *bars, TmaRing &rs)
{
    constexpr int LB = BF16 ? 1 : 2;                      // 2 KB pieces per learner per super-row
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned G = gridDim.x;
    unsigned char *const ring = ring_base + (size_t)warp * kTmaStages * kTmaChunk;
    const unsigned ring_s = smem_addr(ring);                      // the same, as shared-space addresses
    const unsigned bar_s = smem_addr(bars + warp * kTmaStages);
    const bool expire_hook = (c.flags & DD_DEBUG_EXPIRE_WAIT) != 0;
    const unsigned nfull = (unsigned)(sm.n / kVec);
    const unsigned long long tile_begin = sm.tile_begin;
    const int s = sm.n_part;
    constexpr bool kHasV = MODE == kModeMerge || MODE == kModeApply;
    constexpr bool kNorms = PL || MODE == kModeNorms;
    // Per-participant squared norms: every lane keeps its own fp32 sum per participant in shared
    // memory (behind the rings) and the warp reduces them once per kPlFlushRows rounds, not once
    // per piece; without the area (more than kPlMaxParticipants) each piece is reduced at once.
    float *const pl = kNorms && c.pl_cap > 0 && sm.n_part <= c.pl_cap
                          ? reinterpret_cast<float *>(ring_base + kTmaRingBytes) + (size_t)warp * c.pl_cap * 32
                          : nullptr;
    int pl_rows = 0;
    auto pl_flush = [&]() {
        for (int j = 0; j < sm.n_part; ++j) {
            float t = pl[j * 32 + lane];
            pl[j * 32 + lane] = 0.0f;
            t = warp_sum(t);
            if (lane == 0) sm.dm[warp][j] += (double)t;
        }
        pl_rows = 0;
    };
    const int nmid = MODE == kModeApply ? 2 : s * LB;      // pieces between Theta and v
    const int npieces = 2 + nmid + (kHasV ? 2 : 0);
    const float *const theta = sm.theta;
    const float *const mom = sm.mom;

    // This warp's super-rows in the fragment start at step v_first and are row_stride steps apart.
    constexpr unsigned kRowSteps = kSuperRow / kVec;
    const unsigned row_stride = G * (unsigned)(kTileElems / kVec);
    const unsigned v_first = ((unsigned)(tile - tile_begin) * kWarps + (unsigned)warp) * kRowSteps;

    const int nst = ring_depth<BF16, MODE>(s, sm.n_push, c);
    rs.islot = rs.cslot = 0;                   // drained: both may restart at slot 0 whatever the depth was
    const bool evict_first = MODE == kModeMerge && s <= kEvictFirstMaxParticipants;
    const unsigned long long policy = l2_policy_evict_first();

    // ---- producer (lane 0): one piece per call ---------------------------------------
    unsigned iv0 = v_first;                    // first step of the super-row being requested
    int ipiece = 0;
    int outstanding = 0;
    auto issue = [&]() {
        if (rs.failed || iv0 >= nfull) return;
        if (lane == 0) {
            const Piece pc = sm.piece[ipiece];
            const unsigned cnt = min(kRowSteps, nfull - iv0);      // steps in this super-row
            const unsigned have = cnt > pc.first ? min(cnt - pc.first, (unsigned)pc.cap) : 0u;
            const unsigned bytes = have * pc.step_bytes;
            const char *src = pc.src0 + (unsigned long long)iv0 * pc.step_bytes;
            // (test hook) announce 16 bytes that no copy will deliver: the wait must expire
            const unsigned phantom = expire_hook && iv0 == v_first && ipiece == 0 ? 16u : 0u;
            mbar_arrive_expect_tx(bar_s + 8u * rs.islot, bytes + phantom);
            if (bytes != 0) {
                if (evict_first) bulk_copy_g2s_hint(ring_s + kTmaChunk * rs.islot, src, bytes, bar_s + 8u * rs.islot, policy);
                else bulk_copy_g2s(ring_s + kTmaChunk * rs.islot, src, bytes, bar_s + 8u * rs.islot);
            }
        }
        if (++ipiece == npieces) { ipiece = 0; iv0 += row_stride; }
        if (++rs.islot == nst) rs.islot = 0;
        ++outstanding;
    };
    // ---- consumer: the next piece is in rs.cslot once its barrier flips -----------------
    auto acquire = [&]() -> const unsigned char * {
        __syncwarp();                                              // the slot consumed last is free again
        if (!rs.failed) {
            issue();
            const bool ok = mbar_wait_bounded(bar_s + 8u * rs.cslot, (rs.phase_bits >> rs.cslot) & 1u);
            if (!__all_sync(0xffffffffu, ok)) rs.failed = true;    // the whole warp gives up together
        }
        return ring + rs.cslot * kTmaChunk;
    };
    auto release = [&]() {
        if (rs.failed) return;
        rs.phase_bits ^= 1u << rs.cslot;
        if (++rs.cslot == nst) rs.cslot = 0;
        --outstanding;
    };

#pragma unroll 1
    for (int p = 0; p < nst - 1; ++p) issue();

    const float eta = c.eta, mu = c.mu;
    const bool heavy = (c.flags & DD_HEAVY_BALL) != 0;
    const int n_push = sm.n_push;
#pragma unroll 1
    for (unsigned v0 = v_first; v0 < nfull && !rs.failed; v0 += row_stride) {
        const unsigned cnt = min(kRowSteps, nfull - v0);
        float2 nT[4][4], acc[4][4];
        // Theta: two pieces of 64 steps; lane owns steps r*32 + lane, r = 0..3
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const unsigned char *slot = acquire();
#pragma unroll
            for (int rr = 0; rr < 2; ++rr) {
                const int r = 2 * half + rr;
                const uint4 *p = reinterpret_cast<const uint4 *>(slot + (rr * 32 + lane) * 32);
                const uint4 a = p[0], b = p[1];
                nT[r][0] = make_float2(-__uint_as_float(a.x), -__uint_as_float(a.y));
                nT[r][1] = make_float2(-__uint_as_float(a.z), -__uint_as_float(a.w));
                nT[r][2] = make_float2(-__uint_as_float(b.x), -__uint_as_float(b.y));
                nT[r][3] = make_float2(-__uint_as_float(b.z), -__uint_as_float(b.w));
#pragma unroll
                for (int k = 0; k < 4; ++k) acc[r][k] = make_float2(0.0f, 0.0f);
            }
            release();
        }
        if (MODE == kModeApply) {
            // Delta = cscale * u: the stored mean direction, two halves
            const float cs = sm.cscale;
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const unsigned char *slot = acquire();
#pragma unroll
                for (int rr = 0; rr < 2; ++rr) {
                    const int r = 2 * half + rr;
                    const uint4 *p = reinterpret_cast<const uint4 *>(slot + (rr * 32 + lane) * 32);
                    const uint4 a = p[0], b = p[1];
                    acc[r][0] = make_float2(-cs * __uint_as_float(a.x), -cs * __uint_as_float(a.y));
                    acc[r][1] = make_float2(-cs * __uint_as_float(a.z), -cs * __uint_as_float(a.w));
                    acc[r][2] = make_float2(-cs * __uint_as_float(b.x), -cs * __uint_as_float(b.y));
                    acc[r][3] = make_float2(-cs * __uint_as_float(b.z), -cs * __uint_as_float(b.w));
                }
                release();
            }
        } else {
            // acc = sum_j w_j (theta_j - Theta) = -Delta; the difference first, then the weight
#pragma unroll 1
            for (int j = 0; j < s; ++j) {
                const float w = sm.w[j];
                const float2 w2 = make_float2(w, w);
                float2 q2 = make_float2(0.0f, 0.0f);
                if (BF16) {
                    const unsigned char *slot = acquire();
#pragma unroll
                    for (int r = 0; r < 4; ++r) {
                        const uint4 x = *reinterpret_cast<const uint4 *>(slot + r * 512 + lane * 16);
                        const unsigned word[4] = {x.x, x.y, x.z, x.w};
                        float2 qr = make_float2(0.0f, 0.0f);
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const float2 th = make_float2(__uint_as_float(word[k] << 16),
                                                          __uint_as_float(word[k] & 0xffff0000u));
                            const float2 d = __fadd2_rn(th, nT[r][k]);
                            if (MODE != kModeNorms) acc[r][k] = __ffma2_rn(w2, d, acc[r][k]);
                            if (kNorms) qr = __ffma2_rn(d, d, qr);          // even / odd elements side by side
                        }
                        if (kNorms && (unsigned)(r * 32 + lane) < cnt) q2 = __fadd2_rn(q2, qr);
                    }
                    release();
                } else {
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        const unsigned char *slot = acquire();
#pragma unroll
                        for (int rr = 0; rr < 2; ++rr) {
                            const int r = 2 * half + rr;
                            const uint4 *p = reinterpret_cast<const uint4 *>(slot + (rr * 32 + lane) * 32);
                            const uint4 a = p[0], b = p[1];
                            const float2 th[4] = {make_float2(__uint_as_float(a.x), __uint_as_float(a.y)),
                                                  make_float2(__uint_as_float(a.z), __uint_as_float(a.w)),
                                                  make_float2(__uint_as_float(b.x), __uint_as_float(b.y)),
                                                  make_float2(__uint_as_float(b.z), __uint_as_float(b.w))};
                            float2 qr = make_float2(0.0f, 0.0f);
#pragma unroll
                            for (int k = 0; k < 4; ++k) {
                                const float2 d = __fadd2_rn(th[k], nT[r][k]);
                                if (MODE != kModeNorms) acc[r][k] = __ffma2_rn(w2, d, acc[r][k]);
                                if (kNorms) qr = __ffma2_rn(d, d, qr);
                            }
                            if (kNorms && (unsigned)(r * 32 + lane) < cnt) q2 = __fadd2_rn(q2, qr);
                        }
                        release();
                    }
                }
                if (kNorms && !rs.failed) {
                    float q = q2.x + q2.y;
                    if (pl != nullptr) {
                        pl[j * 32 + lane] += q;
                    } else {
                        q = warp_sum(q);
                        if (lane == 0) sm.dm[warp][j] += (double)q;
                    }
                }
            }
        }
        if (kNorms && pl != nullptr && ++pl_rows == kPlFlushRows) pl_flush();
        if (MODE == kModeNorms) continue;

        float dsq = 0.0f, tsq = 0.0f, msq = 0.0f;
        if (MODE == kModeDir) {
            // the mean direction u = sum_j a_j (Theta - theta_j), kept for the apply pass
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const unsigned step = (unsigned)(r * 32 + lane);
                if (step < cnt && !rs.failed) {
                    float U[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        U[k] = -((k & 1) ? acc[r][k >> 1].y : acc[r][k >> 1].x);
                        dsq = fmaf(U[k], U[k], dsq);
                    }
                    store_f32x8<WIDE>(sm.scratch, v0 + step, U);
                }
            }
        } else {
            // v and the outer step: v' = mu v + Delta; Theta' = Theta - eta (Delta + mu v')
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const unsigned char *slot = acquire();
#pragma unroll
                for (int rr = 0; rr < 2; ++rr) {
                    const int r = 2 * half + rr;
                    const unsigned step = (unsigned)(r * 32 + lane);
                    const uint4 *p = reinterpret_cast<const uint4 *>(slot + (rr * 32 + lane) * 32);
                    const uint4 a = p[0], b = p[1];
                    float V[8] = {__uint_as_float(a.x), __uint_as_float(a.y), __uint_as_float(a.z),
                                  __uint_as_float(a.w), __uint_as_float(b.x), __uint_as_float(b.y),
                                  __uint_as_float(b.z), __uint_as_float(b.w)};
                    float T[8];
                    if (step < cnt && !rs.failed) {
#pragma unroll
                        for (int k = 0; k < 8; ++k) {
                            const float delta = -((k & 1) ? acc[r][k >> 1].y : acc[r][k >> 1].x);
                            const float vn = fmaf(mu, V[k], delta);
                            const float u = heavy ? vn : fmaf(mu, vn, delta);
                            const float tn = fmaf(-eta, u, -((k & 1) ? nT[r][k >> 1].y : nT[r][k >> 1].x));
                            V[k] = vn;
                            T[k] = tn;
                            dsq = fmaf(delta, delta, dsq);
                            tsq = fmaf(tn, tn, tsq);
                            msq = fmaf(vn, vn, msq);
                        }
                        const unsigned vi = v0 + step;
                        store_f32x8<WIDE>(sm.mom, vi, V);
                        store_f32x8<WIDE>(sm.theta, vi, T);
                        if (sm.out_bf16 != nullptr || (BF16 && n_push > 0)) {
                            const uint4 packed = make_uint4(pack_bf16x2(T[0], T[1]), pack_bf16x2(T[2], T[3]),
                                                            pack_bf16x2(T[4], T[5]), pack_bf16x2(T[6], T[7]));
                            if (sm.out_bf16 != nullptr)
                                st_stream16(reinterpret_cast<uint4 *>(sm.out_bf16) + vi, packed);
                            // fused push: Theta' replaces the selected learners' copies (in place: this
                            // warp has already consumed these elements of every copy it reads)
                            if (BF16)
                                for (int q = 0; q < n_push; ++q)
                                    st_stream16(reinterpret_cast<uint4 *>(sm.push[q]) + vi, packed);
                        }
                        if (!BF16)
                            for (int q = 0; q < n_push; ++q)
                                store_f32x8<false>(reinterpret_cast<float *>(sm.push[q]), vi, T);
                    }
                }
                release();
            }
        }
        if (c.records != nullptr) {
            dsq = warp_sum(dsq);
            tsq = warp_sum(tsq);
            msq = warp_sum(msq);
            if (lane == 0) {
                sm.red[warp][0] += (double)dsq;
                sm.red[warp][1] += (double)tsq;
                sm.red[warp][2] += (double)msq;
            }
        }
    }

    if (kNorms && pl != nullptr && pl_rows > 0) pl_flush();
    if (rs.failed) {
        // Give the copies still in flight a bounded chance to land before this
        // warp's slots can be reused or the CTA exits, and say what happened.
        for (int k = 0; k < outstanding; ++k) {
            (void)mbar_wait_bounded(bar_s + 8u * rs.cslot, (rs.phase_bits >> rs.cslot) & 1u);
            rs.phase_bits ^= 1u << rs.cslot;
            if (++rs.cslot == nst) rs.cslot = 0;
        }
        rs.islot = rs.cslot;
        if (lane == 0) sm.any_failed = 1;       // reported through the fragment's ticket (flush_fragment)
    }
}

// Kernel body of the staged merge.  MODE is what this launch does with fragments
// merged radial-directionally (kModeMerge for a plain launch); a fragment of kind
// DD_MERGE_AVG is skipped by the norms and direction passes and gets the ordinary
// fused merge in the apply pass, so one batch can mix both kinds.
template <bool BF16, int MODE, bool PL>
__device__ __forceinline__ void merge_body_tma(const DevFrag *frags, const Common &c)
{
    __shared__ Smem sm;
    __shared__ unsigned long long bars[kWarps * kTmaStages];
    extern __shared__ __align__(128) unsigned char ring_base[];
    const unsigned G = gridDim.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if ((PL || MODE == kModeNorms) && c.pl_cap > 0)   // per-lane norm sums start at zero (and are left so)
        for (int i = threadIdx.x; i < c.pl_cap * kWarps * 32; i += kThreads)
            reinterpret_cast<float *>(ring_base + kTmaRingBytes)[i] = 0.0f;
    if (lane == 0)
        for (int d = 0; d < kTmaStages; ++d) mbar_init(bars + warp * kTmaStages + d, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncthreads();

    TmaRing rs;
    int cur = -1;
    unsigned long long tile = blockIdx.x;
    while (tile < c.total_tiles) {
        __syncthreads();
        if (threadIdx.x < 32) {
            cur = find_frag(frags, cur < 0 ? 0 : cur + 1, c.P, tile);
            if (MODE == kModeApply && frags[cur].kind == DD_MERGE_AVG)
                load_header<kModeMerge>(frags + cur, cur, tile, c, sm);
            else
                load_header<MODE>(frags + cur, cur, tile, c, sm);
        }
        __syncthreads();
        cur = sm.frag;
        const unsigned long long tile_end = sm.tile_end;
        const unsigned long long mine = (tile_end - tile + G - 1) / G;      // this CTA's tiles in the fragment
        const bool plain = MODE == kModeMerge || MODE == kModeMergeGram ||
                           (MODE == kModeApply && sm.kind == DD_MERGE_AVG);
        const bool worked_on = sm.status == DD_STATUS_OK && (plain || sm.kind == DD_MERGE_RDA);
        if (worked_on) {
            if (plain) build_piece_table<BF16, kModeMerge>(sm);
            else build_piece_table<BF16, MODE>(sm);
            __syncthreads();
            // A warp whose ring failed in an earlier fragment skips its rows of this one too: the
            // fragment is incomplete and must say so.
            if (rs.failed && lane == 0 &&
                ((tile - sm.tile_begin) * kWarps + (unsigned)warp) * (unsigned long long)(kSuperRow / kVec) < sm.n / kVec)
                sm.any_failed = 1;
            const int rem = (int)(sm.n % kVec);
            const bool owns_tail = rem != 0 && warp == 0 && tile + (mine - 1) * G == tile_end - 1;
            float dsq = 0.0f, tsq = 0.0f, msq = 0.0f;
            if (plain) {
                if (!rs.failed) {
                    if (sm.wide) process_fragment_tma<BF16, true, kModeMerge, PL && MODE == kModeMerge>(sm, c, tile, ring_base, bars, rs);
                    else process_fragment_tma<BF16, false, kModeMerge, PL && MODE == kModeMerge>(sm, c, tile, ring_base, bars, rs);
                }
                if (owns_tail)
                    process_tail<BF16, PL && MODE == kModeMerge, kModeMerge>(sm, c, (sm.n / kVec) * kVec, rem, dsq, tsq, msq);
            } else {
                if (!rs.failed) {
                    if (sm.wide) process_fragment_tma<BF16, true, MODE, PL>(sm, c, tile, ring_base, bars, rs);
                    else process_fragment_tma<BF16, false, MODE, PL>(sm, c, tile, ring_base, bars, rs);
                }
                if (owns_tail) process_tail<BF16, PL, MODE>(sm, c, (sm.n / kVec) * kVec, rem, dsq, tsq, msq);
            }
            if (owns_tail && c.records != nullptr) {
                dsq = warp_sum(dsq);
                tsq = warp_sum(tsq);
                msq = warp_sum(msq);
                if (lane == 0) {
                    sm.red[0][0] += (double)dsq;
                    sm.red[0][1] += (double)tsq;
                    sm.red[0][2] += (double)msq;
                }
            }
            if (c.records != nullptr) {
                if (plain) flush_fragment<PL && MODE == kModeMerge>(sm, c);
                else flush_fragment<PL>(sm, c);
            }
        }
        tile += mine * G;
    }
}

}  // namespace ddm
