/*
 * lvspec.h - C ABI of the B200 (sm_100a) hot path of the LVSpec verify step.
 *
 * Two operations, in the order a verify step runs them:
 *
 *   lvspec_verify_attention  the target model's verification attention: the
 *       gamma (= the paper's K, Eq. 1) draft-token queries of each sequence
 *       attend over that sequence's KV cache, which video tokens dominate;
 *       fused into the softmax is the share of each query's probability that
 *       lands on the visual-token span ("visual mass"), the relevance score
 *       this library feeds to the acceptance rule.
 *
 *   lvspec_loose_accept      the loose acceptance pass over the target logits:
 *       vocabulary-wide argmax per draft position, then the rule of Sec. 3.2
 *       and 3.3 (Eq. 5-7) and the accepted length of Eq. 2.
 *
 * Around them, each documented at its declaration: the attention on a paged
 * cache, with several visual spans, and on a draft-token tree; the acceptance
 * pass with the emit step, with host buffers, and without any allocation; the
 * paper's own relevance score (Eq. 4) as an alternative input to the rule.
 *
 * Conventions
 *   - "device" pointers are CUDA global memory of the context's device; "host"
 *     pointers are ordinary host memory.  The caller owns every buffer it
 *     passes; the library neither frees nor keeps them past the call.
 *   - All tensors are dense, row-major, innermost dimension contiguous, with the
 *     shapes given at each call; device tensors must be 16-byte aligned.
 *   - Device calls enqueue work on the context's stream and return without
 *     synchronising.  The return value reports argument and launch errors only.
 *     A call refused for its arguments (INVALID_ARG, UNSUPPORTED) has launched
 *     nothing.
 *   - A context owns scratch memory on its device and is not thread-safe.
 *     Calls on one context must not overlap on the GPU with each other unless
 *     they are ordered on the same stream.
 *   - There is no CPU fallback: without a CUDA device lvspec_create fails.
 */
#ifndef LVSPEC_H_
#define LVSPEC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    LVSPEC_OK = 0,
    LVSPEC_ERR_INVALID_ARG = 1,  /* null pointer, bad shape, span or length out of range */
    LVSPEC_ERR_UNSUPPORTED = 2,  /* a shape the kernels do not cover (see each call) */
    LVSPEC_ERR_WORKSPACE = 3,    /* scratch memory could not be allocated, or would have to grow
                                    during a stream capture (see lvspec_reserve) */
    LVSPEC_ERR_CUDA = 4,         /* a CUDA runtime call failed; see lvspec_last_error */
    LVSPEC_ERR_TIMEOUT = 5       /* a bounded device-side wait ran out */
} lvspec_status_t;

/* Bits of the device status word (lvspec_device_status). */
#define LVSPEC_DEV_WAIT_EXPIRED 0x1u /* a bounded barrier wait gave up; results invalid */
#define LVSPEC_DEV_NAN_LOGIT    0x2u /* a NaN logit was seen (it was ranked as -inf) */

#define LVSPEC_MAX_BATCH 128   /* sequences per call */
#define LVSPEC_MAX_ROWS  128   /* gamma * (Hq / Hkv): query rows sharing one KV head */
#define LVSPEC_MAX_GAMMA 64    /* draft tokens per sequence */

typedef struct lvspec_ctx lvspec_ctx_t; /* opaque */

/* Shape of one verification-attention call. */
typedef struct {
    int32_t batch;       /* B, 1..LVSPEC_MAX_BATCH */
    int32_t gamma;       /* draft queries per sequence, 1..LVSPEC_MAX_GAMMA */
    int32_t n_q_heads;   /* Hq */
    int32_t n_kv_heads;  /* Hkv, divides Hq; gamma * Hq / Hkv <= LVSPEC_MAX_ROWS */
    int32_t head_dim;    /* D: 64 or 128 */
    int32_t kv_capacity; /* Lmax: cache slots allocated per (sequence, KV head) */
    int32_t n_split;     /* KV splits per (sequence, KV head); 0 lets the library choose */
    int32_t kernel;      /* LVSPEC_KERNEL_* ; 0 = default */
} lvspec_attn_shape_t;

#define LVSPEC_KERNEL_DEFAULT 0
#define LVSPEC_KERNEL_SIMT    1 /* plain CUDA-core kernel: any supported shape */
#define LVSPEC_KERNEL_TCGEN05 2 /* TMA + tcgen05 tensor-core kernel: kv_capacity >= 128 (the default then) */

/* Parameters of the rule.  n_loose >= 0 gives the number of loosened positions
 * directly; n_loose < 0 derives it from lambda as floor(lambda * gamma + 1e-9)
 * (Sec. 3.2: the lambda*K positions of lowest relevance; the paper runs
 * lambda = 0.7, K = 10, i.e. 7 loosened positions). */
typedef struct {
    double lambda;   /* in [0, 1]; used when n_loose < 0 */
    int32_t n_loose; /* -1, or 0..gamma */
    int32_t reserved;
} lvspec_thresholds_t;

/* ---- context -------------------------------------------------------------- */

/* Creates a context on CUDA device `device` (it becomes the current device of
 * the calling thread during each call).  Allocates the scratch memory the
 * kernels need (a few MiB, grown on demand by later calls) and zeroes it.
 * Errors: INVALID_ARG (null out pointer, bad ordinal), CUDA (no device or
 * driver), WORKSPACE.
 * The attention kernels of a context are launched "programmatically dependent"
 * on the kernel before them in the stream (their set-up overlaps that kernel's
 * tail; they still wait for it to finish before they read any input).  The
 * environment variable LVSPEC_NO_PDL=1, read here, makes them plain launches. */
lvspec_status_t lvspec_create(lvspec_ctx_t **ctx, int device);

/* Synchronises the context's stream, frees its scratch memory and the context. */
lvspec_status_t lvspec_destroy(lvspec_ctx_t *ctx);

/* Sets the CUDA stream (a cudaStream_t passed as void*; NULL = default stream)
 * that later calls enqueue on. */
lvspec_status_t lvspec_set_stream(lvspec_ctx_t *ctx, void *cuda_stream);

/* Synchronises the stream, reads and clears the device status word.
 * `flags` (host) receives the LVSPEC_DEV_* bits.  Returns LVSPEC_ERR_TIMEOUT if
 * LVSPEC_DEV_WAIT_EXPIRED is set, LVSPEC_ERR_CUDA if the sync failed. */
lvspec_status_t lvspec_device_status(lvspec_ctx_t *ctx, uint32_t *flags);
/* The same call under the name "last device status": what the kernels launched
 * since the previous reading have reported. */
lvspec_status_t lvspec_last_device_status(lvspec_ctx_t *ctx, uint32_t *flags);

/* Text of the last error recorded on this context (never NULL; valid until the
 * next call on the context).  `ctx` may be NULL: then the text describes why
 * the last lvspec_create on this thread failed. */
const char *lvspec_last_error(const lvspec_ctx_t *ctx);

const char *lvspec_status_string(lvspec_status_t status);

/* Number of kernels this context has launched since it was created. */
uint64_t lvspec_launch_count(const lvspec_ctx_t *ctx);

/* KV splits the library would use for `shape` with the longest sequence
 * `max_kv_len` (what n_split = 0 resolves to); 0 on invalid input. */
int32_t lvspec_attention_splits(const lvspec_ctx_t *ctx, const lvspec_attn_shape_t *shape,
                                int32_t max_kv_len);
/* The same for lvspec_verify_attention_fp8 (half the bytes per tile: it takes more splits). */
int32_t lvspec_attention_splits_fp8(const lvspec_ctx_t *ctx, const lvspec_attn_shape_t *shape,
                                    int32_t max_kv_len);

/* Scratch memory.  A context owns one scratch buffer on its device (split
 * partials of the attention, argmax partials of the acceptance pass, cosines of
 * the relevance score; never results).  A call that needs more than the context
 * holds grows it: that synchronises the context's stream, frees and allocates,
 * and so must not happen inside a CUDA-graph stream capture.  A caller that
 * captures its calls, or that wants every allocation done at start-up, sizes the
 * buffer first:
 *
 *   lvspec_*_workspace_bytes  bytes of scratch the call of that shape needs
 *       (attention: any of the lvspec_verify_attention* forms with `shape`, the
 *       longest sequence `max_kv_len` and the split choice `shape->n_split`;
 *       accept: any of the lvspec_loose_accept* forms that take a context;
 *       relevance: lvspec_visual_relevance).  0 on invalid input.
 *   lvspec_reserve            grows the buffer to at least `workspace_bytes`
 *       (the largest of the figures above); never shrinks it.
 *   lvspec_workspace_capacity bytes the context holds now.
 *
 * While the context's stream is being captured, a call that would have to grow
 * the buffer returns LVSPEC_ERR_WORKSPACE instead, launches nothing and leaves
 * the capture valid; lvspec_reserve does the same.  The *_host forms also own
 * device staging memory for their copies; they synchronise anyway and are not
 * meant for capture. */
size_t lvspec_attention_workspace_bytes(const lvspec_ctx_t *ctx, const lvspec_attn_shape_t *shape,
                                        int32_t max_kv_len);
size_t lvspec_accept_workspace_bytes(const lvspec_ctx_t *ctx, int32_t batch, int32_t gamma,
                                     int32_t vocab);
size_t lvspec_relevance_workspace_bytes(const lvspec_ctx_t *ctx, int32_t batch, int32_t gamma,
                                        int32_t n_visual, int32_t dim);
size_t lvspec_workspace_capacity(const lvspec_ctx_t *ctx);
lvspec_status_t lvspec_reserve(lvspec_ctx_t *ctx, size_t workspace_bytes);

/* Self-test of the bounded device-side waits.  Every barrier wait in the kernels
 * of this library has a time limit (about two seconds); a wait that runs out
 * raises LVSPEC_DEV_WAIT_EXPIRED and lets the kernel return, so that a lost
 * arrival cannot hang the GPU.  This call enqueues one warp that waits, through
 * the same code but with a limit of `limit_ms` milliseconds (1..2000), on a
 * barrier nothing ever completes.  Afterwards lvspec_device_status reports
 * LVSPEC_ERR_TIMEOUT once, and the context is as usable as before. */
lvspec_status_t lvspec_selftest_wait_expiry(lvspec_ctx_t *ctx, int32_t limit_ms);

/* ---- verification attention ---------------------------------------------------
 *
 * Operation (Eq. 1: the K draft tokens are verified by the target model in one
 * parallel pass; the attention is scaled-dot-product attention, App. "Baseline
 * Details").  For sequence b, draft query g in [0, gamma), query head h:
 *
 *   visible(b, g) = kv_len[b] - gamma + g + 1      (the draft tokens occupy the
 *                   last gamma slots of the cache and see each other causally)
 *   s_j   = <q[b,g,h,:], k_cache[b, h / (Hq/Hkv), j, :]> / sqrt(D),  j < visible
 *   p_j   = softmax_j(s_j)
 *   out[b,g,h,:]        = sum_j p_j * v_cache[b, h / (Hq/Hkv), j, :]
 *   visual_mass[b,g,h]  = sum of p_j over j in [span_start, span_end), j < visible
 *
 *   q            device, bf16  [B, gamma, Hq, D]
 *   k_cache      device, bf16  [B, Hkv, Lmax, D]
 *   v_cache      device, bf16  [B, Hkv, Lmax, D]
 *   kv_len       host,  int32  [B]      gamma <= kv_len[b] <= Lmax, counts the draft slots
 *   visual_span  host,  int32  [B][2]   0 <= start <= end <= kv_len[b] - gamma
 *   out          device, bf16  [B, gamma, Hq, D]   (written)
 *   visual_mass  device, fp32  [B, gamma, Hq]      (written)
 *
 * Products are bf16 x bf16 accumulated in fp32; the softmax, its sums and the
 * visual mass are fp32; `out` is rounded to bf16 once at the end.  kv_len and
 * visual_span are read during the call and may be reused as soon as it returns.
 *
 * Errors: INVALID_ARG for null pointers, misaligned device pointers, Hq not a
 * multiple of Hkv, lengths or spans outside the ranges above, batch or gamma
 * beyond the LVSPEC_MAX_* limits; UNSUPPORTED for head_dim other than 64 / 128
 * or more than LVSPEC_MAX_ROWS query rows per KV head; WORKSPACE / CUDA.
 */
lvspec_status_t lvspec_verify_attention(lvspec_ctx_t *ctx, const lvspec_attn_shape_t *shape,
                                        const void *q, const void *k_cache, const void *v_cache,
                                        const int32_t *kv_len, const int32_t *visual_span,
                                        void *out, float *visual_mass);

/* lvspec_verify_attention on a cache with the caller's own layout: any layout in which
 * the head_dim channels of one (sequence, KV head, position) are contiguous.  Element
 * (b, h, j, c) of the K cache sits at k_cache + b * k_strides->batch + h * k_strides->head
 * + j * k_strides->position + c (in bf16 elements), V likewise with v_strides.  The dense
 * [B, Hkv, Lmax, D] layout of lvspec_verify_attention is {Hkv * Lmax * D, Lmax * D, D};
 * a position-major cache [B, Lmax, Hkv, D] is {Lmax * Hkv * D, D, Hkv * D}; K and V
 * interleaved in one buffer [B, Hkv, Lmax, 2, D] is {2 * Hkv * Lmax * D, 2 * Lmax * D, 2 * D}
 * for both, with v_cache = k_cache + D.  Strides must be positive multiples of 8 elements
 * (16 bytes), the position stride at least D.  The same operation, arithmetic and
 * results as lvspec_verify_attention (Eq. 1); the tensor-core kernel reads the layout
 * through its TMA descriptors, the plain kernel through the same strides. */
typedef struct {
    int64_t batch;    /* elements between sequences */
    int64_t head;     /* elements between KV heads */
    int64_t position; /* elements between cache positions */
} lvspec_kv_strides_t;
lvspec_status_t lvspec_verify_attention_strided(lvspec_ctx_t *ctx, const lvspec_attn_shape_t *shape,
                                                const lvspec_kv_strides_t *k_strides,
                                                const lvspec_kv_strides_t *v_strides, const void *q,
                                                const void *k_cache, const void *v_cache,
                                                const int32_t *kv_len, const int32_t *visual_span,
                                                void *out, float *visual_mass);

/* Draft-token trees (App. "Exploration on Draft Token Trees": a static tree of
 * branches with K draft tokens each; every branch is verified loosely on its
 * own and the branch with the longest accepted length is kept).
 *
 * lvspec_verify_attention_tree is lvspec_verify_attention for such a tree:
 * shape->gamma counts ALL draft queries, gamma = n_branches * K; the gamma draft
 * slots at the end of the cache hold the branches one after the other; query g
 * (branch g / K) sees the context before the draft slots and the slots of its
 * own branch up to itself, nothing of the other branches.  All else, limits
 * included (gamma * Hq / Hkv <= LVSPEC_MAX_ROWS), is as for
 * lvspec_verify_attention; n_branches = 1 is that call.
 *
 * The acceptance pass then treats the branches as sequences of their own:
 * lvspec_loose_accept with batch = B * n_branches and gamma = K on logits
 * [B, n_branches, K, V], drafts [B, n_branches, K] and the attention's
 * visual_mass [B, n_branches * K, Hq] read as [B * n_branches, K, Hq]; the
 * loosened set is taken among the K positions of a branch.
 * lvspec_select_branch picks, per sequence, the branch with the longest accepted
 * length (the first among equals):
 *   accept_len   device, int32 [B, n_branches]
 *   best_branch  device, int32 [B]   (written)
 *   best_len     device, int32 [B]   (written)
 * B * n_branches <= LVSPEC_MAX_BATCH. */
lvspec_status_t lvspec_verify_attention_tree(lvspec_ctx_t *ctx, const lvspec_attn_shape_t *shape,
                                             int32_t n_branches, const void *q, const void *k_cache,
                                             const void *v_cache, const int32_t *kv_len,
                                             const int32_t *visual_span, void *out, float *visual_mass);
lvspec_status_t lvspec_select_branch(lvspec_ctx_t *ctx, int32_t batch, int32_t n_branches,
                                     const int32_t *accept_len, int32_t *best_branch, int32_t *best_len);

/* lvspec_verify_attention with SEVERAL visual spans per sequence (a video whose
 * frames are separated by text: time stamps, captions).  The paper scores a draft
 * token against the visual tokens as a set (Eq. 4); on this path the score is the
 * attention mass on them, so the set is the union of the spans:
 *
 *   visual_mass[b,g,h] = sum of p_j over j in the union of the spans, j < visible
 *
 *   visual_spans  host, int32 [B][n_spans][2]: [start, end) each, sorted and
 *                 disjoint within a sequence, inside 0..kv_len[b]-gamma; an empty
 *                 span (start == end) is padding.  At most 241 spans per sequence.
 *
 * `out` and all else are as for lvspec_verify_attention.  The attention kernels run
 * on the hull of the spans; one more small kernel per sequence then takes off the
 * mass of the positions between them (these are few), which it recomputes in fp32
 * from q, k and the softmax denominators.  n_split = 1 is UNSUPPORTED with
 * LVSPEC_KERNEL_TCGEN05 (the denominators come from the merge of the splits; the
 * automatic choice takes care of it). */
lvspec_status_t lvspec_verify_attention_spans(lvspec_ctx_t *ctx, const lvspec_attn_shape_t *shape,
                                              const void *q, const void *k_cache, const void *v_cache,
                                              const int32_t *kv_len, int32_t n_spans,
                                              const int32_t *visual_spans, void *out, float *visual_mass);

/* lvspec_verify_attention on a PAGED cache (a serving engine's layout; the paper's
 * runs keep one contiguous cache per sequence, Sec. "Experimental Setup", so this is a
 * layout variant of Eq. 1, not another operation).  K and V live in pools of
 * fixed-size pages shared by all sequences:
 *
 *   k_pool, v_pool  device, bf16  [n_pages, Hkv, page_size, D]
 *   block_table     device, int32 [B, kv_capacity / page_size]: pool page of each
 *                   logical page of a sequence; logical position j of sequence b
 *                   is row j % page_size of page block_table[b][j / page_size]
 *
 * shape->kv_capacity is the logical capacity per sequence, a whole number of
 * pages; page_size is a multiple of 128 (one tile never straddles pages).  Only
 * the entries of pages that hold positions below kv_len[b] are read; an entry
 * outside 0..n_pages-1 is not an error: its positions read as zeros.  The block
 * table is read on the device during the call (it may be written by the kernel
 * before this call in the stream).  All else is as for lvspec_verify_attention:
 * same arithmetic, same results bit for bit as on the equivalent contiguous cache.
 * UNSUPPORTED for head_dim other than 128 and for LVSPEC_KERNEL_SIMT. */
lvspec_status_t lvspec_verify_attention_paged(lvspec_ctx_t *ctx, const lvspec_attn_shape_t *shape,
                                              int32_t page_size, int32_t n_pages, const void *q,
                                              const void *k_pool, const void *v_pool,
                                              const int32_t *block_table, const int32_t *kv_len,
                                              const int32_t *visual_span, void *out, float *visual_mass);

/* lvspec_verify_attention on an FP8 cache.  The paper's premise is that the target's
 * pass over the long visual KV cache is bound by memory traffic (Sec. 1; the T_t^K
 * term of the speed-up formula in Sec. 2.2): a cache stored in 8 bits halves it.  The
 * operation is that of Eq. 1 as above, on the cache values
 *
 *   k[b,h,j,:] = k_scale[b,h] * decode(k_cache[b,h,j,:]),   v likewise,
 *
 * where decode is the OCP 8-bit floating-point format E4M3 (1 sign, 4 exponent bits
 * with bias 7, 3 mantissa bits; no infinities, codes 0x7F / 0xFF are NaN, largest value
 * 448):
 *
 *   k_cache, v_cache  device, uint8  [B, Hkv, Lmax, D]   E4M3 codes
 *   k_scale, v_scale  device, fp32   [B, Hkv]            read during the call
 *
 * q, out and everything else are as for lvspec_verify_attention (q and out stay bf16).
 * Arithmetic: the 8-bit tiles go to the tensor cores as they are; q and the
 * probabilities are each split into two E4M3 terms (leading four significant bits and
 * the rest) so that they lose no more than they would as bf16; accumulation is fp32.
 * Range: E4M3 has 17 binades.  A row's reference is set so that the largest score of the
 * split's first tile has probability 2^3, and moves up (with a rescale of the
 * accumulators) when a later score exceeds that by more than 2^5.  A probability keeps
 * eight significant bits down to 2^5 below the first tile's largest, four bits down to
 * 2^9 below, and vanishes 2^12 below it: a row that holds most of its mass that far (8
 * nats) under its largest score is beyond this call; the bf16 call has no such limit.
 * Tolerances against the plain definition on the decoded cache: those of the bf16 call.
 * UNSUPPORTED for head_dim other than 128, for LVSPEC_KERNEL_SIMT, for more than 80
 * query rows per KV head (gamma * Hq / Hkv), and for kv_capacity < 128. */
lvspec_status_t lvspec_verify_attention_fp8(lvspec_ctx_t *ctx, const lvspec_attn_shape_t *shape,
                                            const void *q, const void *k_cache, const void *v_cache,
                                            const float *k_scale, const float *v_scale,
                                            const int32_t *kv_len, const int32_t *visual_span,
                                            void *out, float *visual_mass);

/* Same operation on HOST buffers: copies q, the caches, and the results through
 * device staging memory the context owns (grown on demand), on the context's
 * stream, and synchronises before returning.  All seven arrays are host
 * pointers with the shapes above (out is bf16, visual_mass fp32). */
lvspec_status_t lvspec_verify_attention_host(lvspec_ctx_t *ctx, const lvspec_attn_shape_t *shape,
                                             const void *q, const void *k_cache,
                                             const void *v_cache, const int32_t *kv_len,
                                             const int32_t *visual_span, void *out,
                                             float *visual_mass);

/* ---- loose acceptance ---------------------------------------------------------
 *
 * Operation, per sequence b (Sec. 3.2, 3.3):
 *   1. y_i = argmax_v target_logits[b,i,v]; ties go to the lowest v; a NaN
 *      logit ranks as -inf (and raises LVSPEC_DEV_NAN_LOGIT); a row with
 *      nothing above -inf gives y_i = 0.
 *   2. score_i = sum_h visual_mass[b,i,h], added in index order in fp64.
 *      n_mass_heads = 1 takes a ready per-position score instead (for
 *      instance the paper's own relevance score of Eq. 4).
 *   3. Loosened set I' = the first n' positions when positions are ordered by
 *      (score ascending, position ascending) (Eq. 5).  NaN scores are not
 *      supported.
 *   4. accepted_i = (draft_i == y_i) or (i in I') or (y_i == draft_k for some k
 *      with |k - i| <= shift_window, 0 <= k < gamma)  (Eq. 6; Eq. 7 when
 *      shift_window >= gamma - 1; shift_window = 0 switches the
 *      position-shift tolerance off).
 *   5. accept_len[b] = number of leading accepted positions (Eq. 2), 0..gamma.
 *
 *   target_logits  device, fp32  [B, gamma, V]
 *   draft_tokens   device, int32 [B, gamma]
 *   visual_mass    device, fp32  [B, gamma, n_mass_heads]
 *   thresholds     host
 *   accept_len     device, int32 [B]            (written)
 *
 * All decisions are exact integer / IEEE comparisons: the result is
 * bit-identical to the definition above.
 * Errors: INVALID_ARG (null or misaligned pointers, batch/gamma/vocab/heads
 * < 1 or beyond limits, lambda outside [0,1], n_loose > gamma, shift_window
 * < 0); WORKSPACE / CUDA.
 */
lvspec_status_t lvspec_loose_accept(lvspec_ctx_t *ctx, int32_t batch, int32_t gamma,
                                    int32_t vocab, int32_t n_mass_heads,
                                    const float *target_logits, const int32_t *draft_tokens,
                                    const float *visual_mass,
                                    const lvspec_thresholds_t *thresholds, int32_t shift_window,
                                    int32_t *accept_len);

/* As lvspec_loose_accept, with two optional extra outputs (either may be NULL):
 *   target_tokens  device, int32 [B, gamma]   y_i of step 1
 *   accepted       device, uint8 [B, gamma]   accepted_i of step 4 */
lvspec_status_t lvspec_loose_accept_ex(lvspec_ctx_t *ctx, int32_t batch, int32_t gamma,
                                       int32_t vocab, int32_t n_mass_heads,
                                       const float *target_logits, const int32_t *draft_tokens,
                                       const float *visual_mass,
                                       const lvspec_thresholds_t *thresholds,
                                       int32_t shift_window, int32_t *accept_len,
                                       int32_t *target_tokens, uint8_t *accepted);

/* As lvspec_loose_accept, plus the emit step: what the verify step hands back
 * to the decoding loop.  The paper defines the accepted length tau (Eq. 2) and
 * is silent on the rest; this is the usual speculative-decoding bookkeeping
 * under the rule's decisions.  The first tau draft tokens are kept as they are
 * (also where they were accepted by loosening or by shift tolerance: the later
 * target rows were computed with these very tokens in the context).  If a
 * position was rejected (tau < gamma), the target's own token y_tau of that
 * position follows as the correction; with tau = gamma there is no further
 * target row to take a bonus token from.
 *   kv_len      device, int32 [B]          optional (NULL together with new_kv_len)
 *   emitted     device, int32 [B, gamma]   (written) tokens, -1 beyond n_emitted
 *   n_emitted   device, int32 [B]          (written) min(tau + 1, gamma)
 *   new_kv_len  device, int32 [B]          (written) kv_len - gamma + tau: the cache
 *               keeps the accepted draft slots; the correction token has no K/V
 *               yet and is the next step's input */
lvspec_status_t lvspec_loose_accept_emit(lvspec_ctx_t *ctx, int32_t batch, int32_t gamma,
                                         int32_t vocab, int32_t n_mass_heads,
                                         const float *target_logits, const int32_t *draft_tokens,
                                         const float *visual_mass,
                                         const lvspec_thresholds_t *thresholds,
                                         int32_t shift_window, const int32_t *kv_len,
                                         int32_t *accept_len, int32_t *emitted, int32_t *n_emitted,
                                         int32_t *new_kv_len);

/* Same operation on HOST buffers (see lvspec_verify_attention_host). */
lvspec_status_t lvspec_loose_accept_host(lvspec_ctx_t *ctx, int32_t batch, int32_t gamma,
                                         int32_t vocab, int32_t n_mass_heads,
                                         const float *target_logits, const int32_t *draft_tokens,
                                         const float *visual_mass,
                                         const lvspec_thresholds_t *thresholds,
                                         int32_t shift_window, int32_t *accept_len);

/* ---- the paper's own relevance score -------------------------------------------
 *
 * Sec. 3.1, Eq. 4: the visual relevance A_s of draft token k is the mean of the
 * N largest cosine similarities between its final-layer hidden state H_D[k] and
 * the final-layer hidden states H_V[j] of the visual tokens (Eq. 3; the paper
 * runs N = 10).  The result feeds lvspec_loose_accept as `visual_mass` with
 * n_mass_heads = 1, in place of the attention's visual mass.
 *
 * H_V is fixed after prefill, so the reciprocal norms of its rows are computed
 * once (lvspec_row_inv_norms) and passed to every step's call.
 *
 *   lvspec_row_inv_norms:
 *     x         device, bf16  [rows, dim]     dim a multiple of 8
 *     inv_norm  device, fp32  [rows]          (written) 1 / ||x_r||, 0 for a zero row
 *
 *   lvspec_visual_relevance:
 *     h_draft          device, bf16  [B, gamma, dim]       H_D of this step
 *     h_visual         device, bf16  [B, n_visual, dim]    H_V
 *     visual_inv_norm  device, fp32  [B, n_visual]         from lvspec_row_inv_norms
 *     top_n            N >= 1; min(N, n_visual) similarities are averaged
 *     relevance        device, fp32  [B, gamma]            (written) A_s
 *
 * A zero vector has cosine 0 with everything.  Dot products are bf16 x bf16
 * accumulated in fp32 on the tensor cores; norms, cosines and the Top-N mean are
 * fp32.  dim must be a multiple of 64, n_visual >= 1, gamma <= LVSPEC_MAX_GAMMA.
 * Errors: INVALID_ARG (null or misaligned pointers, sizes out of range),
 * UNSUPPORTED (dim not a multiple of 64), WORKSPACE / CUDA.
 */
lvspec_status_t lvspec_row_inv_norms(lvspec_ctx_t *ctx, int64_t rows, int32_t dim, const void *x,
                                     float *inv_norm);
lvspec_status_t lvspec_visual_relevance(lvspec_ctx_t *ctx, int32_t batch, int32_t gamma,
                                        int32_t n_visual, int32_t dim, const void *h_draft,
                                        const void *h_visual, const float *visual_inv_norm,
                                        int32_t top_n, float *relevance);

/* ---- loose acceptance without any allocation ---------------------------------
 *
 * The paper has no counterpart of this call: it is the operation of
 * lvspec_loose_accept, offered to callers that are not allowed to allocate
 * device memory: an inference server whose own pool already owns the GPU's
 * memory, a process that must stay inside a memory budget fixed at start-up, or
 * a latency-critical loop that cannot afford the device-wide synchronisation a
 * cudaMalloc or cudaFree may bring.  It takes no context.  Its scratch memory
 * (argmax partials, per-sequence tickets, a status word: about 66 KB) is a
 * fixed array inside the library's device image; every GPU on which the
 * library's code is loaded holds that array until the process ends.
 *
 * Arguments, operation and results are those of lvspec_loose_accept, except:
 *   - work is enqueued on `cuda_stream` (a cudaStream_t passed as void*; NULL =
 *     the default stream) of the CALLER'S CURRENT DEVICE, and all pointers must
 *     belong to that device;
 *   - batch * gamma must not exceed LVSPEC_STATIC_MAX_ROWS; larger calls are
 *     refused with LVSPEC_ERR_UNSUPPORTED and launch nothing;
 *   - a NaN logit still ranks as -inf, but is not reported (there is no context
 *     to read a status word from);
 *   - `error_text` (host, may be NULL) receives a NUL-terminated description of
 *     at most error_text_len bytes when the call fails, "" when it succeeds.
 *
 * The call itself never calls cudaMalloc, cudaFree or any allocating routine.
 * The first call on each device looks up the device address of the array
 * (cudaGetSymbolAddress); make that first call outside any stream capture.
 * Later calls only enqueue two kernels (one clears the tickets).
 *
 * All calls on a device share the one array, and it keeps whatever the last
 * call left in it; each call clears the part that has to start at zero.  Two
 * calls whose kernels can overlap on the GPU (different streams, or several
 * host threads without stream ordering between them) race on it and give
 * wrong results: order them on one stream or with events. */
#define LVSPEC_STATIC_MAX_ROWS  1024  /* batch * gamma */
#define LVSPEC_STATIC_MAX_SLOTS 8192  /* argmax partials the array holds */
lvspec_status_t lvspec_loose_accept_static(void *cuda_stream, int32_t batch, int32_t gamma,
                                           int32_t vocab, int32_t n_mass_heads,
                                           const float *target_logits,
                                           const int32_t *draft_tokens, const float *visual_mass,
                                           const lvspec_thresholds_t *thresholds,
                                           int32_t shift_window, int32_t *accept_len,
                                           char *error_text, size_t error_text_len);

#ifdef __cplusplus
}
#endif
#endif /* LVSPEC_H_ */
