// Internal declarations shared by the translation units of liblvspec.so.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "lvspec.h"

// Time stamps for performance work, compiled in only with -DLVSPEC_TRACE (a separate
// build of the library: `python -m paper_2604_05650_b200.trace`; the shipped library has
// none of it).  The attention and merge kernels then write into a buffer of 64-bit words
// the caller provides through lvspec_trace_set_buffer (device memory; word 0 counts the
// records, records of 8 words follow from word 8):
//   CTA records   {kind (1 attention, 2 merge), q pointer of the call, CTA index,
//                  %globaltimer at CTA entry, past the prologue / the grid-dependency wait,
//                  all K.Q^T issued (attention only), end of the CTA's work, unused}
//   tile records  of the one attention CTA (split 3, KV head 2, sequence 0), from word
//                 8 + 8 * kTraceCtaRecords on: per role r (0 first softmax warp, 1 K.Q^T
//                 issuer, 2 P.V issuer, 3 inside the first softmax warp's pass), tile i < 32, eight clock64 stamps at
//                 ((r * 32 + i) * 8): see the LVSPEC_TILE_TS uses in verify_attn_tc.cu
#ifdef LVSPEC_TRACE
constexpr int kTraceCtaRecords = 4000;
// every translation unit with stamps holds its own copy of the buffer address
static __device__ unsigned long long *g_lvspec_trace = nullptr;
namespace lvspec {
cudaError_t trace_set_buffer_attention(unsigned long long *device_words);
cudaError_t trace_set_buffer_merge(unsigned long long *device_words);
}
__device__ __forceinline__ unsigned long long lvspec_trace_now()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
#define LVSPEC_TILE_TS(tr, role, tile, slot) \
    do { if ((tr) && (tile) < 32) (tr)[(((role) * 32 + (tile)) * 8) + (slot)] = clock64(); } while (0)
#else
#define LVSPEC_TILE_TS(tr, role, tile, slot) do { } while (0)
#endif

namespace lvspec {

// Per-sequence lengths travel as kernel parameters (the C ABI takes them as
// host arrays), so a launch needs no host->device copy of its own.
struct SeqInfo {
    int32_t kv_len[LVSPEC_MAX_BATCH];
    int32_t span_start[LVSPEC_MAX_BATCH];
    int32_t span_end[LVSPEC_MAX_BATCH];
};

struct AttnParams {
    const uint16_t *q;     // [B, gamma, Hq, D] bf16
    const uint16_t *k;     // [B, Hkv, Lmax, D] bf16
    const uint16_t *v;
    uint16_t *out;         // [B, gamma, Hq, D] bf16
    float *mass;           // [B, gamma, Hq]
    float *part_o;         // [B, Hkv, n_split, M, D] fp32, unnormalised
    float *part_stat;      // [B, Hkv, n_split, M, 4]: m (log2 units), l, l_vis, unused
    float *lse2;           // optional [B, gamma, Hq]: log2 of the softmax denominator, written by the combine
    uint32_t *status;      // device status word
    int32_t B, gamma, Hq, Hkv, D, Lmax, G, M, n_split;
    int32_t pdl;           // launch programmatically dependent on the previous kernel
    int32_t branch_len;    // draft tokens per tree branch (= gamma for a plain chain)
    // Paged cache (page_size > 0): k and v are pools [n_pages, Hkv, page_size, D]; logical
    // page j of sequence b is pool page block_table[b * pages_per_seq + j]
    const int32_t *block_table;
    int32_t page_size, pages_per_seq, n_pages;
    float scale_log2;      // log2(e) / sqrt(D)
    // fp8 cache (fp8 != 0): k and v point to E4M3 codes, one byte per element, and a
    // cache element is code * scale with one scale per (sequence, KV head)
    int32_t fp8;
    const float *k_scale;  // [B, Hkv]
    const float *v_scale;  // [B, Hkv]
    // Cache strides in elements (the head_dim channels of a position are contiguous):
    // element (b, h, j, c) of k sits at k + b * k_sb + h * k_sh + j * k_sp + c.  The dense
    // [B, Hkv, Lmax, D] cache has sp = D, sh = Lmax * D, sb = Hkv * Lmax * D; a page pool
    // [n_pages, Hkv, page_size, D] has sp = D, sh = page_size * D, sb = Hkv * page_size * D.
    int64_t k_sb, k_sh, k_sp, v_sb, v_sh, v_sp;
};

// Does draft query `qi` see the cache position with tail index t = pos - (kv_len -
// gamma)?  t < 0 is the context before the draft slots: always visible.  Among
// the draft slots a query sees its own branch up to itself (branches of
// `branch_len` slots sit one after the other; a plain chain is one branch).
__host__ __device__ inline bool draft_query_sees(int qi, int t, int branch_len)
{
    return qi >= t && (t < 0 || (qi / branch_len) * branch_len <= t);
}

// Partial results of one KV split, rows r = g * G + hg.
static inline size_t part_o_elems(const AttnParams &p)
{
    return (size_t)p.B * p.Hkv * p.n_split * p.M * p.D;
}
static inline size_t part_stat_elems(const AttnParams &p)
{
    return (size_t)p.B * p.Hkv * p.n_split * p.M * 4;
}

cudaError_t launch_attn_simt(const AttnParams &p, const SeqInfo &seq, cudaStream_t stream,
                             int *launches);
bool attn_tc_supported(const AttnParams &p);
cudaError_t launch_attn_tc(const AttnParams &p, const SeqInfo &seq, cudaStream_t stream,
                           int *launches);
cudaError_t launch_attn_combine(const AttnParams &p, cudaStream_t stream, int *launches);

// Several visual spans: the attention runs on their hull, then the probability mass of
// the positions between the spans (at most kMaxGaps ranges per sequence) is taken off.
constexpr int kMaxGaps = 240;
struct GapParams {
    const uint16_t *q;     // [B, gamma, Hq, D]
    const uint16_t *k;     // [B, Hkv, Lmax, D]
    const float *lse2;     // [B, gamma, Hq]
    float *mass;           // [B, gamma, Hq], corrected in place
    int32_t b, gamma, Hq, Hkv, D, Lmax, G, M;
    float scale_log2;
    int32_t n_gaps;
    int32_t gap_start[kMaxGaps];        // first cache position of each gap
    int32_t gap_first[kMaxGaps + 1];    // gaps laid end to end: index of each gap's first position; [n_gaps] = total
};
cudaError_t launch_gap_mass(const GapParams &p, cudaStream_t stream, int *launches);

struct AcceptParams {
    const float *logits;      // [B, gamma, V]
    const int32_t *draft;     // [B, gamma]
    const float *mass;        // [B, gamma, Hm]
    int32_t *accept_len;      // [B]
    int32_t *target;          // optional [B, gamma]
    uint8_t *accepted;        // optional [B, gamma]
    const int32_t *kv_len;    // optional [B]: cache lengths going in (emit step)
    int32_t *emitted;         // optional [B, gamma]: accepted draft tokens, then the correction token, then -1
    int32_t *n_emitted;       // optional [B]
    int32_t *new_kv_len;      // optional [B] (with kv_len)
    float *part_val;          // [B, gamma, n_vsplit]
    int32_t *part_idx;        // [B, gamma, n_vsplit]
    uint32_t *counters;       // [B], zero between calls
    uint32_t *status;
    int32_t B, gamma, V, Hm, n_loose, window, n_vsplit;
};
cudaError_t launch_loose_accept(const AcceptParams &p, cudaStream_t stream, int *launches);
cudaError_t launch_select_branch(const int32_t *accept_len, int B, int R, int32_t *best_branch,
                                 int32_t *best_len, cudaStream_t stream, int *launches);

struct RelevanceParams {
    const uint16_t *h_draft;    // [B, K, d] bf16
    const uint16_t *h_visual;   // [B, lv, d] bf16
    const float *v_inv_norm;    // [B, lv]
    float *cos_t;               // scratch [B, K, lv_pad]: Top-N candidates or all cosines, one row per draft token
    float *relevance;           // [B, K]
    uint32_t *counters;         // [B, K] candidates appended so far; zero between calls
    uint32_t *status;
    int32_t B, K, lv, d, top_n;
    int32_t lv_pad;             // lv rounded up to a multiple of 4
    int32_t n_sm;
};
cudaError_t launch_row_inv_norms(const uint16_t *x, long long rows, int dim, float *out,
                                 cudaStream_t stream, int *launches);
cudaError_t launch_visual_relevance(const RelevanceParams &p, cudaStream_t stream, int *launches);
size_t relevance_scratch_bytes(int B, int K, int lv, int d);
cudaError_t launch_wait_expiry(uint32_t *status, unsigned long long limit_ns, cudaStream_t stream,
                               int *launches);

}  // namespace lvspec
