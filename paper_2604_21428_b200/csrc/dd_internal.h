// Internal layout shared by the host launcher and the device code of libddmerge.
// Not part of the public ABI.
#pragma once

#include <cstdint>

#include "dd_merge.h"

namespace ddm {

constexpr int kThreads = 256;            // threads per CTA
constexpr int kWarps = kThreads / 32;
constexpr int kVec = 8;                  // elements one thread handles per step
constexpr int kStepsPerLane = 4;         // 8-element steps a lane handles per warp round
constexpr int kTileElems = kThreads * kVec * kStepsPerLane;   // 8192 elements per tile: 1024 per warp
constexpr int kNumScalarDiag = 3;        // delta_sq, theta_sq, mom_sq
constexpr unsigned long long kMaxFragmentElems = 1ull << 34;   // 8-element steps are indexed in 32 bits
// Radial-directional merges of at most this many participants take the two-launch form through
// the participants' Gram matrix (its s (s + 1) / 2 products run on the CUDA cores).
#define DD_RDA_GRAM_MAX_PARTICIPANTS 8
constexpr int kGramPairsMax = DD_RDA_GRAM_MAX_PARTICIPANTS * (DD_RDA_GRAM_MAX_PARTICIPANTS + 1) / 2;

// Ring slots a warp uses for a plain merge (one fewer copy is in flight ahead of the consumer):
// the shallow ring for fp32 copies and for up to kShallowMaxParticipantsBf16 bf16 copies, the full
// one above.  One definition for the kernel and for the host's dd_launch_shape.
#ifndef DD_TMA_STAGES
#define DD_TMA_STAGES 3
#endif
#ifndef DD_SHALLOW_MAX_BF16
#define DD_SHALLOW_MAX_BF16 7
#endif
constexpr int kTmaStages = DD_TMA_STAGES;
constexpr int kShallowMaxParticipantsBf16 = DD_SHALLOW_MAX_BF16;
#ifdef __CUDACC__
__host__ __device__
#endif
constexpr int merge_ring_slots(bool bf16, int participants)
{
    return kTmaStages < 3 ? kTmaStages : ((!bf16 || participants <= kShallowMaxParticipantsBf16) ? 2 : kTmaStages);
}
// A merge with a fused push: from this share of writes in the bytes moved on, one CTA per SM with
// the full ring; below, the ordinary grid with the shallow ring.
constexpr double kPushHeavyWriteShare = 0.45;

// One fragment as the kernel sees it.  Raw counters, mask and pointers travel to
// the device; participation and weights are derived there.
struct alignas(16) DevFrag {
    float *theta;
    float *mom;
    uint16_t *out_bf16;
    unsigned long long n;
    unsigned long long tile_begin;       // first flat tile index of this fragment
    unsigned long long tile_end;         // one past its last tile (always > tile_begin)
    unsigned long long mask;
    int K;
    int has_steps;
    float *scratch;                      // radial-directional merge: n floats for the mean direction
    int kind;                            // DD_MERGE_AVG or DD_MERGE_RDA
    int n_part_host;                     // |S| as the host counted it (sizes the per-lane norm area)
    unsigned long long push_mask;        // learners whose copy is overwritten with Theta' (fused push)
    unsigned long long pad2_;
    const void *ptrs[DD_MAX_LEARNERS];
    unsigned long long tokens[DD_MAX_LEARNERS];
    unsigned long long steps[DD_MAX_LEARNERS];
};

struct Common {
    float eta;
    float mu;
    unsigned flags;
    int M;
    int P;
    unsigned long long total_tiles;
    dd_merge_record *records;            // device, nullable
    double *partials;                    // [P][nq][grid] per-CTA partial sums
    unsigned *tickets;                   // [P] completion counters, zero between calls
    int nq;                              // quantities per fragment in `partials`
    double *gram = nullptr;              // [P][kGramPairsMax] Gram matrices (lower triangle) of the two-launch RDA
    int pl_cap = 0;                      // participants the per-lane norm area holds (0: none)
    int push_depth = 2;                  // ring slots a fragment with a fused push uses (3 when the launch runs 1 CTA per SM)
    int apply_depth = 2;                 // ring slots of the radial-directional apply pass (3 when it runs 1 CTA per SM)
};

}  // namespace ddm
