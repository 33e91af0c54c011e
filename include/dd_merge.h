/*
 * dd_merge.h -- C ABI of libddmerge: the Decoupled DiLoCo syncer's per-fragment
 * merge on one NVIDIA B200 (sm_100a).
 *
 * For one parameter fragment the syncer (Algorithm 2, steps 2-3) takes the copies
 * theta_m held by the M learners, keeps the learners that reported in time
 * (minimum quorum K and grace window, Section 3.2), weights their outer
 * gradients Theta - theta_m by the token/step counters (the Weight display,
 * Section 3.2), merges them (weighted direct averaging, Appendix "Merging
 * methods") and applies the outer optimizer, SGD with Nesterov momentum (Eq. 1,
 * Eq. 2), to the global fragment Theta and its momentum v.  The whole chain runs
 * in one fused CUDA kernel that reads every participating operand once.
 *
 * Conventions common to every call
 *   - Pointers marked [device] are device addresses on the context's GPU;
 *     pointers marked [host] are ordinary host memory.  Every buffer is borrowed:
 *     the library allocates only its own context workspace.
 *   - Theta and v are float32 and are updated IN PLACE.  Learner copies are
 *     read-only, contiguous, all float32 or all bf16 (dd_dtype).
 *   - Device base pointers must be 16-byte aligned (32-byte aligned Theta and v
 *     get 256-bit accesses).  n is arbitrary up to 2^34 elements per fragment
 *     (DD_ERR_TOO_LARGE beyond).
 *   - Calls enqueue work on the given CUDA stream (a cudaStream_t passed as
 *     void*; NULL = the legacy default stream) and return without waiting.  Host
 *     arrays are consumed before the call returns.
 *   - Return value: DD_OK (0) or a negative dd_error.  Conditions that depend on
 *     the data -- quorum not met, zero total weight -- are not errors: the call
 *     returns DD_OK, writes dd_merge_record.status != 0 and leaves Theta and v
 *     untouched (the syncer "keeps waiting", Algorithm 2 step 1).
 *   - Nothing here aborts, throws, traps or spins without bound on the device.
 */
#ifndef DD_MERGE_H
#define DD_MERGE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define DD_MAX_LEARNERS 64

typedef struct dd_ctx dd_ctx;

typedef enum { DD_F32 = 0, DD_BF16 = 1 } dd_dtype;

/* How the per-learner outer gradients of a fragment are merged (Appendix "Merging methods"). */
typedef enum { DD_MERGE_AVG = 0, DD_MERGE_RDA = 1 } dd_merge_kind;

typedef enum {
    DD_OK = 0,
    DD_ERR_INVALID_ARG = -1,        /* null where not allowed, M / K / P out of range, non-finite lr or mu */
    DD_ERR_ALIGNMENT = -2,          /* a device pointer is not 16-byte aligned */
    DD_ERR_ALIAS = -3,              /* a participating learner buffer overlaps Theta, v or out_bf16 */
    DD_ERR_TOO_MANY_LEARNERS = -4,  /* M > DD_MAX_LEARNERS */
    DD_ERR_CUDA = -5,               /* a CUDA runtime call failed; see dd_last_cuda_error */
    DD_ERR_TOO_LARGE = -6           /* a size exceeds what the entry point supports */
} dd_error;

/* dd_merge_record.status */
enum {
    DD_STATUS_OK = 0,
    DD_STATUS_QUORUM_NOT_MET = 1,   /* fewer than max(K,1) participants; nothing written */
    DD_STATUS_ZERO_WEIGHT = 2,      /* weights sum to zero; nothing written */
    DD_STATUS_WAIT_LIMIT = 3        /* a bounded device-side wait gave up; fragment state is unspecified */
};

/* flags */
enum {
    DD_HEAVY_BALL = 1u << 0,        /* Theta' = Theta - lr v' instead of the Nesterov form */
    DD_DIAG_PER_LEARNER = 1u << 1,  /* also ||Theta - theta_m||^2 for every participant */
    DD_DIAG_STATE = 1u << 2,        /* also ||Theta'||^2 and ||v'||^2 */
    DD_RDA_THREE_PASS = 1u << 3,    /* radial-directional merges: always the three-launch form (see dd_merge_fragment_rda) */
    /* Test hook for the error path.  Production callers must never set it: every warp's
     * first bulk copy is made to wait for bytes that never come, so its bounded wait
     * expires (about a second, up to three for the launch), every fragment the launch
     * could not finish reports DD_STATUS_WAIT_LIMIT in its record and the kernel returns
     * normally with the context still usable.  Needs records; the state of those
     * fragments is unspecified afterwards.  Rejected by the int4 and allocation-free
     * entry points. */
    DD_DEBUG_EXPIRE_WAIT = 1u << 30
};

/*
 * Written by the device, one per fragment; readable by the host once the stream
 * has been synchronised.  Participants are listed in ascending learner id.
 */
typedef struct {
    int32_t status;
    int32_t n_part;                         /* |S|, S = { m : mask bit m and tokens[m] > 0 } */
    uint8_t idx[DD_MAX_LEARNERS];           /* first n_part entries valid */
    float   w_hat[DD_MAX_LEARNERS];         /* normalised weights, aligned with idx */
    double  w_total;                        /* sum of the raw weights over S */
    double  delta_sq;                       /* ||Delta||_2^2 of the merged outer gradient */
    double  theta_sq;                       /* ||Theta'||_2^2   (DD_DIAG_STATE) */
    double  mom_sq;                         /* ||v'||_2^2       (DD_DIAG_STATE) */
    double  delta_m_sq[DD_MAX_LEARNERS];    /* ||Theta - theta_m||_2^2, aligned with idx (DD_DIAG_PER_LEARNER) */
} dd_merge_record;

/*
 * Context: binds a GPU and owns a small workspace (per-CTA partial sums of the
 * norm diagnostics, completion tickets, a ring of descriptor staging slots).
 * One context serves one host thread at a time; calls issued through one
 * context on DIFFERENT streams must not overlap on the GPU, because they
 * share that workspace.  device < 0 selects the current device.
 */
int dd_create(dd_ctx **ctx, int device);
int dd_destroy(dd_ctx *ctx);

/*
 * One syncer update of one fragment (Algorithm 2 steps 2-3).
 *
 *   S      = { m < M : bit m of quorum_mask set and tokens[m] > 0 }      (Section 3.2; Section 4:
 *            an absent learner is a learner of weight 0)
 *   w_m    = tokens[m] * (tokens[m] / steps[m]);  tokens[m] when steps == NULL   (Weight, Section 3.2)
 *   w^_m   = w_m / sum_{m in S} w_m
 *   Delta  = sum_{m in S} w^_m (Theta - theta_m)          (weighted direct averaging, Appendix)
 *   v'     = outer_mu v + Delta
 *   Theta' = Theta - outer_lr (Delta + outer_mu v')       (SGD with Nesterov momentum, Section 2)
 *
 * If |S| < max(K, 1) the record says DD_STATUS_QUORUM_NOT_MET and nothing else
 * is written.  Buffers of learners outside S are never dereferenced (their
 * pointers may be NULL or dangling, their contents NaN).
 *
 *   global, momentum  [device] float32[n], in/out
 *   learner_ptrs      [host]   M device pointers to learner_dtype[n]
 *   tokens, steps     [host]   uint64[M]; steps may be NULL; tokens[m] > 0 with
 *                              steps[m] == 0, or participants' tokens summing past
 *                              2^64 - 1, is DD_ERR_INVALID_ARG
 *   quorum_mask       bit m = learner m reported in time (bits >= M ignored)
 *   K                 minimum quorum, 0 <= K <= M (0 acts as 1)
 *   out_bf16          [device] optional bf16[n]: round-to-nearest-even copy of
 *                     Theta' (the payload broadcast back to the learners)
 *   record            [device] optional; without it no diagnostics are computed
 *
 * The call enqueues one kernel on cuda_stream and returns.  The first call on a
 * context that passes a record allocates the context's diagnostics workspace, sized
 * once for any single-fragment call (every M, every flag); from then on
 * dd_merge_fragment neither allocates nor synchronises, so it may be recorded into
 * a CUDA graph by stream capture (host arrays are consumed before it returns).
 * Only a batched call with many fragments can make the workspace grow later, which
 * synchronises the device.
 */
int dd_merge_fragment(dd_ctx *ctx, float *global, float *momentum,
                      const void *const *learner_ptrs, int M, dd_dtype learner_dtype,
                      const uint64_t *tokens, const uint64_t *steps,
                      uint64_t quorum_mask, int K, float outer_lr, float outer_mu,
                      uint32_t flags, size_t n, void *out_bf16,
                      dd_merge_record *record, void *cuda_stream);

/*
 * Many fragments in ONE kernel launch.  Fragments may differ in size, mask and
 * counters (the counters are kept per learner and per fragment, Section 3.1);
 * M, dtype, lr, mu and flags are shared.  Semantics per fragment are exactly
 * those of dd_merge_fragment.  descs and the arrays it points to are host
 * memory and are consumed before return.
 */
typedef struct {
    float *global;                      /* [device] float32[n] in/out */
    float *momentum;                    /* [device] float32[n] in/out */
    void *out_bf16;                     /* [device] optional bf16[n] */
    const void *const *learner_ptrs;    /* [host] M device pointers */
    const uint64_t *tokens;             /* [host] uint64[M] */
    const uint64_t *steps;              /* [host] uint64[M] or NULL */
    uint64_t quorum_mask;
    int32_t K;
    uint64_t n;
} dd_fragment_desc;

int dd_merge_fragments_batched(dd_ctx *ctx, const dd_fragment_desc *descs, int P, int M,
                               dd_dtype learner_dtype, float outer_lr, float outer_mu,
                               uint32_t flags, dd_merge_record *records /* [device] P records or NULL */,
                               void *cuda_stream);

/*
 * Merge and push in one pass.  Algorithm 2 ends a fragment's synchronisation by sending
 * the new global fragment to every learner, which overwrites its copy (alpha = 0 in the
 * learner-side mixing of the Appendix).  When the learner copies the syncer reads are also
 * the buffers the learners resume from, these calls do both: every learner m with bit m of
 * push_mask set has its copy replaced by Theta' rounded to learner_dtype (round to
 * nearest even for bf16), in the same kernel that merges, so Theta' is not read back a
 * second time.  A learner may be pushed to without being merged (it was late or down) and
 * merged without being pushed to.  If the quorum is not met nothing is pushed.
 *
 *   learner_ptrs[m] of a pushed learner is written: it must be non-NULL, 16-byte aligned
 *   and must not overlap global, momentum, out_bf16, or the copy of another learner that
 *   is read or pushed (DD_ERR_ALIAS).  Bits of push_mask at or above M are ignored.
 * Everything else is as in dd_merge_fragment / dd_merge_fragments_batched;
 * push_masks is a host array of P masks.
 */
int dd_merge_fragment_push(dd_ctx *ctx, float *global, float *momentum,
                           void *const *learner_ptrs, int M, dd_dtype learner_dtype,
                           const uint64_t *tokens, const uint64_t *steps,
                           uint64_t quorum_mask, int K, float outer_lr, float outer_mu,
                           uint32_t flags, size_t n, uint64_t push_mask, void *out_bf16,
                           dd_merge_record *record, void *cuda_stream);
int dd_merge_fragments_batched_push(dd_ctx *ctx, const dd_fragment_desc *descs,
                                    const uint64_t *push_masks, int P, int M,
                                    dd_dtype learner_dtype, float outer_lr, float outer_mu,
                                    uint32_t flags, dd_merge_record *records, void *cuda_stream);

/*
 * Radial-directional averaging (RDA, Appendix "Merging methods"): the merged outer
 * gradient keeps the weighted mean NORM of the per-learner outer gradients
 * D_m = Theta - theta_m and takes the direction of their weighted mean direction,
 *
 *   Delta = ( sum_m w^_m ||D_m|| ) * phi( sum_m w^_m phi(D_m) ),   phi(x) = x / ||x||,
 *
 * so that ||Delta|| does not shrink like 1/sqrt(M) when the D_m are nearly
 * orthogonal; the outer step is the same as for dd_merge_fragment.  (The printed
 * weighted formula shows the mean vector in the first factor; it is read as the
 * weighted mean of the norms, by analogy with the unweighted one.)
 * A participant with D_m = 0 adds its (zero) norm to the radial mean and nothing
 * to the direction; if the mean direction vanishes, Delta = 0.
 *
 * Learner copies are read twice, in one of two forms:
 *   - at most 8 participants: two launches on cuda_stream.  The first accumulates the
 *     Gram matrix G_jk = <D_j, D_k> of the outer gradients (||D_j||^2 = G_jj, and the
 *     mean direction's squared length is a^T G a with a_j = w^_j / ||D_j||); the second
 *     is the ordinary fused merge with the weights c a_j, c = (sum_j w^_j ||D_j||) /
 *     sqrt(a^T G a).  Nothing is stored in between but the matrix; bytes per parameter
 *     = 2 s b_theta + 20.  `scratch` is not used.
 *   - more participants, or DD_RDA_THREE_PASS: three launches -- norms, mean direction
 *     (kept in `scratch`), outer step; bytes per parameter = 2 (s b_theta + 4) + 24.
 * In a batch every fragment takes the same form: two launches only if no
 * radial-directional fragment has more than 8 participants.
 *
 *   scratch   [device] n floats (16-byte aligned), or NULL: the context allocates
 *             and keeps one when the three-launch form needs it (growing it
 *             synchronises the device)
 *   record    as for dd_merge_fragment; delta_m_sq is always filled, delta_sq is
 *             ||Delta||^2 of the RDA result.  DD_DIAG_PER_LEARNER is implied.
 * Everything else is as in dd_merge_fragment.
 */
int dd_merge_fragment_rda(dd_ctx *ctx, float *global, float *momentum,
                          const void *const *learner_ptrs, int M, dd_dtype learner_dtype,
                          const uint64_t *tokens, const uint64_t *steps,
                          uint64_t quorum_mask, int K, float outer_lr, float outer_mu,
                          uint32_t flags, size_t n, void *out_bf16,
                          dd_merge_record *record, float *scratch, void *cuda_stream);

/*
 * Many fragments, each merged by the kind given in merge_kinds[p] (host array of
 * dd_merge_kind values as bytes; NULL = all RDA).  The paper's main runs average
 * the embedding directly and use RDA everywhere else (Section 5 set-up): this call
 * does both in the same three launches.  scratch holds, back to back, n_p rounded
 * up to 8 floats for every RDA fragment (scratch_elems = its capacity in floats;
 * NULL/0 = context-owned).
 */
int dd_merge_fragments_batched_rda(dd_ctx *ctx, const dd_fragment_desc *descs, int P, int M,
                                   dd_dtype learner_dtype, float outer_lr, float outer_mu,
                                   uint32_t flags, const uint8_t *merge_kinds,
                                   dd_merge_record *records, float *scratch,
                                   size_t scratch_elems, void *cuda_stream);

/*
 * The batched radial-directional merge with the push of dd_merge_fragment_push: the apply
 * pass, which no longer reads the learner copies, overwrites those selected by
 * push_masks[p] (host array of P masks) with Theta'.  Same rules for pushed copies.
 */
int dd_merge_fragments_batched_rda_push(dd_ctx *ctx, const dd_fragment_desc *descs,
                                        const uint64_t *push_masks, int P, int M,
                                        dd_dtype learner_dtype, float outer_lr, float outer_mu,
                                        uint32_t flags, const uint8_t *merge_kinds,
                                        dd_merge_record *records, float *scratch, size_t scratch_elems,
                                        void *cuda_stream);

/*
 * One pass of the batched radial-directional merge, for a fragment that is sharded by
 * element range over several GPUs.  The merge needs two whole-fragment quantities that a
 * shard cannot know, so the caller runs the passes one by one on every shard and sums
 * across the shards in between (the paper's RDA likewise all-reduces the norms first and
 * the directions second, Appendix "Merging methods"):
 *
 *   DD_RDA_PASS_NORMS      writes records[p].delta_m_sq[j] = ||Theta - theta_j||^2 of the shard
 *                          -> sum delta_m_sq[0 .. n_part) over the shards, in place
 *   DD_RDA_PASS_DIRECTION  reads delta_m_sq; writes the shard's mean direction to scratch and
 *                          its squared length to records[p].delta_sq
 *                          -> sum delta_sq over the shards, in place
 *   DD_RDA_PASS_APPLY      reads delta_m_sq and delta_sq; outer step (and push, if push_masks is
 *                          given); writes the shard's ||Delta||^2, ||Theta'||^2, ||v'||^2
 *                          -> sum those three for whole-fragment diagnostics
 *
 * records and scratch are required and must be the same memory in all three calls, as must
 * every other argument.  Fragments of kind DD_MERGE_AVG are merged by the apply pass alone.
 * With a single shard the three calls equal dd_merge_fragments_batched_rda[_push].
 */
enum { DD_RDA_PASS_NORMS = 0, DD_RDA_PASS_DIRECTION = 1, DD_RDA_PASS_APPLY = 2 };
int dd_merge_fragments_batched_rda_pass(dd_ctx *ctx, const dd_fragment_desc *descs,
                                        const uint64_t *push_masks /* may be NULL */, int P, int M,
                                        dd_dtype learner_dtype, float outer_lr, float outer_mu,
                                        uint32_t flags, const uint8_t *merge_kinds,
                                        dd_merge_record *records, float *scratch, size_t scratch_elems,
                                        int pass, void *cuda_stream);

/*
 * int4 compression of outer gradients (Appendix "Outer gradients compression": 16 -> 4
 * bits per value before the merge, comparable quality; 2 and 1 bit are not).  The paper
 * prints no quantiser; this library's reading, fixed here so that both ends agree:
 *   - blocks of DD_INT4_BLOCK consecutive elements, the last one possibly shorter;
 *   - D = Theta - theta_m in float32; scale = max|D| / 7 (float32), one per block;
 *   - code = D / scale rounded to nearest (ties to even), clamped to [-7, 7]; a block of
 *     zeros has scale 0 and codes 0;
 *   - a non-finite D poisons its block, as it would poison an uncompressed merge: a NaN
 *     makes the block's scale NaN (all codes 0), an infinity makes it infinite (finite
 *     elements get code 0, infinite ones -7), so every element of the block decodes to a
 *     non-finite value; other blocks are unaffected;
 *   - element i's code + 8 sits in nibble (i & 1) of byte i / 2 (even element low).
 *
 * dd_quantize_outer_gradient_int4 is the learner side:
 *   global [device] float32[n]; learner [device] learner_dtype[n];
 *   codes [device] (n + 1) / 2 bytes, 2-byte aligned; scales [device] float32[ceil(n / 128)].
 *
 * dd_merge_fragment_int4 is dd_merge_fragment with the outer gradients arriving
 * compressed: Delta = sum_{m in S} w^_m (code_m - 8) scale_m, same outer step, same
 * participation, weights, record and errors.  code_ptrs / scale_ptrs are host arrays
 * of M device pointers (16- and 4-byte aligned).  DD_DIAG_PER_LEARNER is not offered.
 * Bytes per merged parameter: s (1/2 + 4/128) + 16.
 */
#define DD_INT4_BLOCK 128
int dd_quantize_outer_gradient_int4(dd_ctx *ctx, const float *global, const void *learner,
                                    dd_dtype learner_dtype, size_t n, uint8_t *codes, float *scales,
                                    void *cuda_stream);
int dd_merge_fragment_int4(dd_ctx *ctx, float *global, float *momentum,
                           const uint8_t *const *code_ptrs, const float *const *scale_ptrs, int M,
                           const uint64_t *tokens, const uint64_t *steps, uint64_t quorum_mask,
                           int K, float outer_lr, float outer_mu, uint32_t flags, size_t n,
                           void *out_bf16, dd_merge_record *record, void *cuda_stream);

/*
 * The same update for a fragment whose operands live in HOST memory -- the
 * paper's syncer pulls each learner's fragment from that learner's host RAM and
 * keeps the global state off the accelerators (Section 4, system overview).
 * The fragment is cut into chunks of chunk_elems elements (0 = library default:
 * an eighth of the fragment in whole 2^20 elements, between 2^20 and 2^24; else a
 * multiple of 8) that are pipelined through three sets of device staging buffers
 * owned by the context (each holds one chunk of every operand: 8 + 2 + the
 * participants' payload bytes per element): host-to-device copies, the fused kernel and device-to-host
 * copies of successive chunks overlap.  Only copies of participating learners
 * are transferred.
 *
 *   global, momentum, out_bf16, record, learner_ptrs[m]   all [host]; page-locked
 *        memory is needed for the copies to run at full PCIe speed and to overlap.
 *   The call first waits (on the device) for work already queued on cuda_stream,
 *   and it BLOCKS the calling thread until the results are in host memory.
 *   record (optional) is the record of the whole fragment: squared norms are
 *   summed over the chunks in chunk order.
 * Everything else is as in dd_merge_fragment.
 */
int dd_merge_fragment_host(dd_ctx *ctx, float *global, float *momentum,
                           const void *const *learner_ptrs, int M, dd_dtype learner_dtype,
                           const uint64_t *tokens, const uint64_t *steps,
                           uint64_t quorum_mask, int K, float outer_lr, float outer_mu,
                           uint32_t flags, size_t n, void *out_bf16,
                           dd_merge_record *record, size_t chunk_elems, void *cuda_stream);

/*
 * Host-buffer variants of the batched merge and of the int4 merge (Section 4, system overview:
 * the syncer pulls the fragments from the learners' host RAM; Appendix "Outer gradients
 * compression": 4 bits per value on the wire).  Same pipeline as dd_merge_fragment_host; the
 * chunks of successive fragments follow one another without a pause.
 *
 * dd_merge_fragments_batched_host: descs[p].global, .momentum, .out_bf16 and every
 *   descs[p].learner_ptrs[m] are HOST pointers here; records is a HOST array of P records
 *   (or NULL).  Per fragment the semantics are those of dd_merge_fragment_host.
 *
 * dd_merge_fragment_int4_host: code_ptrs[m] / scale_ptrs[m] are HOST pointers to the codes
 *   ((n + 1) / 2 bytes) and scales (ceil(n / 128) floats) that dd_quantize_outer_gradient_int4
 *   defines; global, momentum, out_bf16, record are host memory.  chunk_elems (0 = library
 *   default) must be a multiple of 128 so that no chunk splits a quantisation block.  Only
 *   s (1/2 + 4/128) + 8 bytes per parameter cross the bus on the way in, against 2 s + 8 for
 *   bf16 copies.  DD_DIAG_PER_LEARNER is not offered.
 *
 * Both block the calling thread until the results are in host memory.
 */
int dd_merge_fragments_batched_host(dd_ctx *ctx, const dd_fragment_desc *descs, int P, int M,
                                    dd_dtype learner_dtype, float outer_lr, float outer_mu,
                                    uint32_t flags, dd_merge_record *records /* [host] P records or NULL */,
                                    size_t chunk_elems, void *cuda_stream);
int dd_merge_fragment_int4_host(dd_ctx *ctx, float *global, float *momentum,
                                const uint8_t *const *code_ptrs, const float *const *scale_ptrs, int M,
                                const uint64_t *tokens, const uint64_t *steps, uint64_t quorum_mask,
                                int K, float outer_lr, float outer_mu, uint32_t flags, size_t n,
                                void *out_bf16, dd_merge_record *record, size_t chunk_elems,
                                void *cuda_stream);

/*
 * The batched merge for callers that cannot allocate device memory.  (The paper
 * has no counterpart to this entry point; it exists for deployment reasons only.)
 *
 * Some hosts of this library may not call cudaMalloc: a syncer living inside a
 * training process whose framework allocator has already claimed nearly all of
 * the GPU, a loop that cannot tolerate the device-wide synchronisation that
 * cudaMalloc / cudaFree imply, or a service with a no-allocation-after-start-up
 * rule.  This call takes no dd_ctx and calls neither cudaMalloc nor cudaFree nor
 * any other allocating routine.  Its scratch memory (device copy of the fragment
 * descriptors, per-CTA partial sums of the norm diagnostics, completion tickets)
 * is a fixed array of DD_NOALLOC_SCRATCH_BYTES inside the library's device
 * image; every GPU on which the library runs holds that array until the process
 * exits.
 *
 * Semantics per fragment are those of dd_merge_fragments_batched, on the CURRENT
 * device, with these limits:
 *   - P <= DD_NOALLOC_MAX_FRAGMENTS, else DD_ERR_TOO_LARGE (nothing is launched);
 *   - DD_DIAG_PER_LEARNER is not offered (DD_ERR_INVALID_ARG);
 *   - the grid is capped at 592 CTAs.
 * The first call on a device does the set-up: it resolves the array's device
 * address (one cudaGetSymbolAddress) and sizes the grid; with lazy module
 * loading it is also the moment the CUDA runtime loads this library's device
 * image, array included, onto that GPU, which can fail on a GPU that is already
 * full.  Make that first call at start-up, and before any stream capture
 * begins.  (Nothing is said here, either way, about recording later calls by
 * stream capture.)  All calls on a device share the one array, and it
 * keeps the previous call's contents: the call itself clears what has to start
 * at zero, but two calls that overlap on the GPU (different streams, or
 * different host threads without ordering) race on it and give wrong results.
 * Calls on one stream are safe back to back.  descs and the arrays it points to
 * are host memory and are consumed before return; the call may wait for earlier
 * work on cuda_stream while it hands the descriptors to the driver.
 */
#define DD_NOALLOC_MAX_FRAGMENTS 32
#define DD_NOALLOC_SCRATCH_BYTES (512 * 1024)
int dd_merge_fragments_batched_noalloc(const dd_fragment_desc *descs, int P, int M,
                                       dd_dtype learner_dtype, float outer_lr, float outer_mu,
                                       uint32_t flags, dd_merge_record *records /* [device] P records or NULL */,
                                       void *cuda_stream);

/*
 * The learner side of a syncer update (Algorithm 1 step 3; Appendix "Mixing learner
 * and syncer params"): for every learner m whose bit is set in apply_mask,
 *     theta_m <- alpha * theta_m + (1 - alpha) * Theta'
 * in the learner dtype (round to nearest even for bf16).  alpha = 0 -- what the
 * paper settles on -- overwrites the copy with the global fragment.  Learners whose
 * bit is clear are not touched (their pointers may be NULL).  Resetting the
 * per-fragment counters is the caller's bookkeeping.
 *
 *   global        [device] float32[n], read only
 *   learner_ptrs  [host]   M device pointers to learner_dtype[n], updated in place
 */
int dd_broadcast_fragment(dd_ctx *ctx, const float *global, void *const *learner_ptrs, int M,
                          dd_dtype learner_dtype, uint64_t apply_mask, float alpha, size_t n,
                          void *cuda_stream);

/*
 * Quorum with grace window (Section 3.2, "Adaptive Quorum Window"), host only.
 * arrival_s[m] is when learner m's report arrived (+inf = never).  The syncer
 * may proceed at t_K, the K-th earliest arrival, and then waits grace_s longer:
 * every learner with arrival <= t_K + grace_s is admitted.  Returns DD_OK and the
 * mask, or DD_OK with *mask_out = 0 and *n_admitted = 0 when fewer than
 * max(K,1) reports ever arrived.
 */
int dd_select_quorum(const double *arrival_s, int M, int K, double grace_s,
                     uint64_t *mask_out, int *n_admitted);

/*
 * Largest admissible grace window: gamma * (tau * xi_step - (xi_quorum + xi_sync)),
 * clamped at 0 (the slack equation of Section 3.2).
 */
double dd_grace_window(double tau, double xi_step, double xi_quorum, double xi_sync,
                       double gamma);

/*
 * Adaptive grace window (Section 3.2): the durations of a learner step, of reaching
 * the quorum and of a synchronisation are tracked by exponential moving averages,
 *     x <- beta * x + (1 - beta) * observation     (the first observation initialises x)
 * and the window is dd_grace_window(tau, xi_step, xi_quorum, xi_sync, gamma).  The
 * paper names the averages but not their coefficient: beta is the caller's.
 * Plain data, host only; 0 <= beta < 1, 0 <= gamma < 1.
 */
typedef struct {
    double tau, gamma, beta;
    double xi_step, xi_quorum, xi_sync;
    int32_t n_obs;
} dd_grace_controller;
int dd_grace_controller_init(dd_grace_controller *gc, double tau, double gamma, double beta);
int dd_grace_controller_observe(dd_grace_controller *gc, double step_s, double quorum_s, double sync_s);
double dd_grace_controller_window(const dd_grace_controller *gc);   /* 0 before the first observation */

/*
 * Fragmentation planner (Appendix "Fragmentation strategies"), host only: assigns
 * each of the model's Q tensors to one of P fragments.
 *
 *   DD_FRAG_LAYER     fragment 0 holds every non-transformer tensor; transformer
 *                     layer l (0-based) goes to fragment 1 + (l mod (P-1)) -- strided
 *                     selection; needs 2 <= P and P-1 <= number of layers.
 *   DD_FRAG_TENSOR    fragment 0 holds every non-transformer tensor; the i-th (0-based,
 *                     in the given order) transformer tensor goes to 1 + (i mod (P-1)).
 *   DD_FRAG_BALANCED  greedy number partitioning over ALL tensors: in descending order
 *                     of size (ties: given order) each tensor joins the fragment whose
 *                     total is smallest (ties: lowest index).  The largest fragment is
 *                     at most 4/3 of the best possible.
 *
 *   size_bits    [host] Q tensor sizes in bits
 *   layer        [host] Q entries: 0-based transformer layer of the tensor, or -1 for a
 *                non-transformer tensor (embedding, final norm, head); may be NULL for
 *                DD_FRAG_BALANCED
 *   fragment_of  [host] out, Q fragment indices in [0, P)
 *   fragment_bits[host] out, optional, P totals
 * Returns DD_OK or DD_ERR_INVALID_ARG (P < 1, Q < 0, a strategy's requirement unmet).
 */
typedef enum { DD_FRAG_LAYER = 0, DD_FRAG_TENSOR = 1, DD_FRAG_BALANCED = 2 } dd_frag_strategy;
int dd_plan_fragments(const uint64_t *size_bits, const int32_t *layer, int Q, int P,
                      dd_frag_strategy strategy, int32_t *fragment_of, uint64_t *fragment_bits);

/* Text for a dd_error / the most recent CUDA error string seen by ctx. */
const char *dd_status_string(int rc);
const char *dd_last_cuda_error(const dd_ctx *ctx);

/* Launch geometry chosen by the context (for reporting): CTAs, threads per CTA, elements per tile. */
int dd_launch_geometry(const dd_ctx *ctx, dd_dtype learner_dtype, int *grid, int *block, int *tile);

/*
 * How a merge of `participants` copies of learner_dtype, fused with a push to `pushed` copies
 * (0 = plain merge) and with or without the bf16 copy of Theta', is launched on a B200: persistent
 * CTAs per SM (2, or 1 for a push whose writes are 45 % or more of the bytes moved) and ring slots
 * each warp uses (2 = one 2 KB copy in flight ahead of the consumer, 3 = two).  Pure host function
 * (no context, no GPU); it reports the rule the launcher and the kernel apply, for benchmarks that
 * want to reproduce the kernel's data movement.  The paper has no counterpart.
 * Returns DD_OK or DD_ERR_INVALID_ARG (dtype, participants outside 1..DD_MAX_LEARNERS, pushed
 * outside 0..DD_MAX_LEARNERS).
 */
int dd_launch_shape(dd_dtype learner_dtype, int participants, int pushed, int with_out_bf16,
                    int *ctas_per_sm, int *ring_slots);

#ifdef __cplusplus
}
#endif
#endif /* DD_MERGE_H */
