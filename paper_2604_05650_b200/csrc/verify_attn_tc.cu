// Verification attention with fused visual mass: TMA + tcgen05 kernel (D = 128 or 64).
//
// One CTA owns one KV split of one (sequence, KV head) and the M = gamma * G
// query rows that read this head.  The GQA-grouped queries are the small side
// of the problem, so the products are taken transposed: per tile of 128 cache
// positions
//     S^T[pos, n] = K_tile[pos, :] . Q[n, :]          (MMA M = 128 positions, N = rows)
//     O^T[d, n]  += V_tile[:, d]^T . P^T[:, n]        (MMA M = 128 channels,  N = rows)
//     L[0..1, n] += [1; in_span]   . P^T[:, n]        (MMA M = 64: row 0 = l, row 1 = l_vis)
// so every TMEM lane of S^T is one cache position (all softmax threads do
// useful exponentials) and the padded dimension is N (granularity 16), not M.
// The softmax denominators l and the visual-span numerators l_vis come out of
// the tensor core as two extra accumulator rows fed by a constant 0/1 tile.
//
// The reference exponent m[n] of a row is the score of the first position of
// the split and stays fixed while scores stay within 2^60 of it; only when a
// score runs past that guard is the tile's maximum taken (a cross-lane
// reduction in this layout) and the accumulators rescaled.  fp32 and bf16
// share the exponent range, so nothing is lost in between.
//
// Warp roles (480 threads): warp 0 = TMA producer, warp 1 = issuer of the
// K.Q^T MMAs and TMEM owner, warp 14 = issuer of the P.V and sum MMAs (one
// thread each; two issuers because a single thread's issue rate, not the tensor
// pipe, bounded the loop), warps 2-13 = three softmax groups of four warps.
// The groups take the tiles in turn (tile i belongs to group i % 3; a thread is
// one cache position, TMEM lane quarter = warp % 4, and works through all N
// columns of its tile), so the latencies of one tile (TMEM load, barrier,
// hand-over) hide behind the exponentials of the two tiles the other groups are
// on; S^T has a TMEM buffer per tile in flight.  The reference exponents m[] are
// shared.  Tiles are handed to the P.V issuer strictly in order, through a
// counter of committed tiles: a group may move m (and rescale the accumulators)
// only while its tile is the oldest uncommitted one, and announces the move in an
// epoch counter; a group whose turn comes compares the epoch with the one it read
// m under and computes its tile once more if m has moved meanwhile.
// K and V tiles sit in separate shared-memory rings,
// each slot two 128-position x 64-channel boxes with the 128-byte swizzle; Q
// arrives by TMA in the same layout.  Every mbarrier wait is bounded; a wait
// that gives up raises LVSPEC_DEV_WAIT_EXPIRED.
//
// fp8 cache (kFp8): K and V are E4M3 codes with one scale per (sequence, KV head), half
// the bytes per position.  An MMA takes both operands in one kind, so the 8-bit tiles
// are multiplied as they are (kind::f8f6f4, K = 32 per instruction) and the bf16
// side is brought to them without losing its bits: a value is split into the E4M3
// number holding its leading four significant bits and the E4M3 number nearest to the
// rest (the next four), both exact for bf16 inputs in the normal range.  Q (scaled by a
// power of two so that its largest magnitude sits below 256) is split once per CTA into
// two operand tiles, and K.Q^T takes both in one accumulation (8 MMAs of K = 32 over the
// 2 x 128 channels); a probability is split by the softmax threads, head and rest sit
// in neighbouring columns of P^T, and V^T.P^T and the sum products run with N = 2 x
// rows: accumulator column 2n holds the head's part of row n, column 2n + 1 the rest's,
// added once in the epilogue.  Probabilities are kept within E4M3's range by the
// reference exponent: the largest score of the split's first tile gets probability 2^3,
// and a later score that would pass 2^8 moves the reference up.  The K scale folds into the
// softmax scale, the V scale into the epilogue.
//
// head_dim 64: one 64-channel box per K or V tile and four K.Q^T steps; the P.V product
// keeps its 128 rows, of which the upper 64 read what follows the box in shared memory
// and fill TMEM lanes nobody reads.
#include <cuda.h>
#include <cuda_bf16.h>

#include <cstdio>
#include <cstdlib>
#include <type_traits>

#include "lvspec_internal.h"
#include "sm100_ptx.cuh"

#ifdef LVSPEC_TRACE
cudaError_t lvspec::trace_set_buffer_attention(unsigned long long *device_words)
{
    return cudaMemcpyToSymbol(g_lvspec_trace, &device_words, sizeof device_words);
}
#endif

namespace lvspec {
namespace {

using namespace ptx;

constexpr int kTilePos = 128;
constexpr int kSoftmaxGroups = 3;           // groups of 4 warps, each on its own share of the columns
constexpr int kSoftmaxWarp0 = 2;            // first softmax warp
constexpr int kSoftmaxWarps = 4 * kSoftmaxGroups;
constexpr int kSoftmaxThreads = 32 * kSoftmaxWarps;
constexpr int kPvWarp = kSoftmaxWarp0 + kSoftmaxWarps;   // issues the P.V and sum MMAs
constexpr int kThreads = 32 * (kPvWarp + 1);
constexpr int kMaxChunks = (LVSPEC_MAX_ROWS / 8 + kSoftmaxGroups - 1) / kSoftmaxGroups;   // per group that shares the columns
constexpr uint32_t kBoxBytes = 16384;       // 128 positions x 64 channels bf16, or x 128 channels E4M3
constexpr uint32_t kSlotBytes = 2 * kBoxBytes;   // a bf16 tile; an fp8 tile is one box
constexpr uint32_t kA2Bytes = 2048;         // one 64 x 16 (bf16) or 64 x 32 (E4M3) constant tile
constexpr float kGuard = 60.f;              // log2 units above m before a rescale
constexpr float kGuard8 = 8.f;              // fp8 cache: probabilities stay below 2^8 (E4M3 ends at 448)
constexpr float kHead8 = 3.f;               // fp8 cache: the largest score of a row in the split's first tile has probability 2^3
constexpr float kMFloor = -1.0e30f;
constexpr int kQBarrier = 1 + kSoftmaxGroups;   // named barrier over all softmax threads
constexpr int kMaxRowsFp8 = 80;             // fp8 cache: 6 accumulator columns per padded row in 512

struct TcConfig {
    int n_pad;   // MMA N: rows padded to a multiple of 16
    int ks, vs, pb;   // K slots, V slots, P buffers
    int sb;           // S^T buffers in TMEM (2 or 3)
    int tmem_cols;
    int page_slots;   // paged cache: pool pages of this split's tiles, one entry per tile
    int slot_bytes;   // one K or V tile: 32 KB bf16, 16 KB fp8
};

// Byte offsets of the shared-memory regions (relative to a 1024-aligned base).
struct SmemMap {
    uint32_t k, v, q, p, a2, m, dl, tmx, vis, bars, misc, pages, total;
};
__host__ __device__ inline SmemMap smem_map(const TcConfig &c)
{
    SmemMap s;
    uint32_t o = 0;
    s.k = o;    o += c.ks * c.slot_bytes;
    s.v = o;    o += c.vs * c.slot_bytes;
    s.q = o;    o += c.n_pad * 256;
    s.p = o;    o += c.pb * c.n_pad * 256;
    s.a2 = o;   o += 4 * kA2Bytes;
    s.m = o;    o += c.n_pad * 4;
    s.dl = o;   o += c.n_pad * 4;
    s.tmx = o;  o += 4 * c.n_pad * 4;
    s.vis = o;  o += c.n_pad * 8;
    s.bars = o; o += 8 * (2 * c.ks + 2 * c.vs + 4 * kSoftmaxGroups + 4);
    s.misc = o; o += 16 + 4 * kSoftmaxWarps;     // TMEM address, abort flag, epoch of m, committed tiles, per-warp maxima of |q|
    s.pages = o; o += 4 * c.page_slots;
    s.total = o;
    return s;
}

struct TcParams {
    AttnParams a;
    TcConfig cfg;
};

// Position in a ring of n slots and the parity of the round: the per-tile loops count
// instead of dividing.
struct Ring {
    int idx, n;
    uint32_t parity;
    __device__ __forceinline__ Ring(int n_) : idx(0), n(n_), parity(0) {}
    __device__ __forceinline__ void next()
    {
        if (++idx == n) {
            idx = 0;
            parity ^= 1u;
        }
    }
};

__device__ __forceinline__ bool wait_unconditional(uint32_t bar, uint32_t parity)
{
    // used while tearing down: time-bounded, ignores the abort flag
    const uint64_t t0 = global_timer_ns();
    while (!mbar_try_wait(bar, parity))
        if (global_timer_ns() - t0 > 1000000000ull) return false;
    return true;
}

// named barrier over the 128 threads of one softmax group (ids 1, 2, ...)
__device__ __forceinline__ void group_sync(int id)
{
    asm volatile("bar.sync %0, 128;" ::"r"(id) : "memory");
}
__device__ __forceinline__ bool group_any(int id, bool pred)
{
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %2, 0;\n\t"
        "bar.red.or.pred p, %1, 128, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(out)
        : "r"(id), "r"((uint32_t)pred)
        : "memory");
    return out != 0;
}

// Accumulator values of the 8 rows of column chunk c8 in this warp's lanes: with an fp8
// cache every row has two columns (the products with the probabilities' leading bits and
// with the rest), added here.
template <bool kFp8>
__device__ __forceinline__ void load_acc8(uint32_t taddr, int c8, float (&v)[8])
{
    if (kFp8) {
        uint32_t a[8], b[8];
        tmem_ld_x8(taddr + c8 * 16, a);
        tmem_ld_x8(taddr + c8 * 16 + 8, b);
        tmem_wait_ld();
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            v[k] = __uint_as_float(a[2 * k]) + __uint_as_float(a[2 * k + 1]);
            v[4 + k] = __uint_as_float(b[2 * k]) + __uint_as_float(b[2 * k + 1]);
        }
    } else {
        uint32_t a[8];
        tmem_ld_x8(taddr + c8 * 8, a);
        tmem_wait_ld();
#pragma unroll
        for (int k = 0; k < 8; ++k) v[k] = __uint_as_float(a[k]);
    }
}

template <bool kFp8>
__device__ __forceinline__ void mma_ss(uint32_t d, uint64_t a, uint64_t b, uint32_t idesc, uint32_t acc)
{
    if (kFp8) mma_f8_ss(d, a, b, idesc, acc);
    else mma_f16_ss(d, a, b, idesc, acc);
}

// Which draft slots a column's query sees: tail indices [lo, hi] (its own branch up to
// itself); the context before the draft slots (tail index < 0) is visible to all.
__device__ __forceinline__ bool column_sees(int2 lohi, int t)
{
    return t < 0 || (unsigned)(t - lohi.x) <= (unsigned)(lohi.y - lohi.x);
}

// exp2 of eight scaled scores of one position, packed to bf16; returns their maximum
// kMask: 0 = every column sees the position; 1 = plain chain of draft tokens (query
// col / G sees tail index t iff it is not below t); 2 = draft tree (table look-up)
// kFp8: each probability goes out as two E4M3 values in neighbouring bytes, its leading
// four significant bits and the rest (see the head of this file).
template <int kMask, bool kFp8>
__device__ __forceinline__ float exp_chunk(const uint32_t (&r)[8], const float *m8, float scale,
                                           const int2 *vis8, int col0, int G, int t, uint4 &dst)
{
    const float4 ma = *reinterpret_cast<const float4 *>(m8);
    const float4 mb = *reinterpret_cast<const float4 *>(m8 + 4);
    const float mm[8] = {ma.x, ma.y, ma.z, ma.w, mb.x, mb.y, mb.z, mb.w};
    float x[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) x[k] = fmaf(__uint_as_float(r[k]), scale, -mm[k]);
    if (kMask == 1) {
#pragma unroll
        for (int k = 0; k < 8; ++k) x[k] = ((col0 + k) / G >= t) ? x[k] : -INFINITY;
    } else if (kMask == 2) {
#pragma unroll
        for (int k = 0; k < 8; ++k) x[k] = column_sees(vis8[k], t) ? x[k] : -INFINITY;
    }
    float mx = fmaxf(fmaxf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3])),
                     fmaxf(fmaxf(x[4], x[5]), fmaxf(x[6], x[7])));
    uint4 pk;
    if (kFp8) {
        uint32_t w[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const float pr = ex2(x[k]);
            const float hd = e4m3_head(pr);
            w[k] = pack_e4m3x2(hd, pr - hd);
        }
        pk.x = w[0] | (w[1] << 16);
        pk.y = w[2] | (w[3] << 16);
        pk.z = w[4] | (w[5] << 16);
        pk.w = w[6] | (w[7] << 16);
    } else {
        pk.x = pack_bf16x2(ex2(x[0]), ex2(x[1]));
        pk.y = pack_bf16x2(ex2(x[2]), ex2(x[3]));
        pk.z = pack_bf16x2(ex2(x[4]), ex2(x[5]));
        pk.w = pack_bf16x2(ex2(x[6]), ex2(x[7]));
    }
    dst = pk;
    return mx;
}

// One pass over this thread's position: exp2 of all n8 column chunks of S^T (four TMEM
// loads in flight per wait), the packed probabilities stored to this position's place in
// the P^T buffer; returns the largest scaled score.  kMask != 0: the tile reaches into the
// draft slots, so columns are masked by what their query may see; the common tile carries
// none of that.  The loop stays rolled: three groups run it at different places, and
// the instruction cache holds the short form better.
template <int kMask, bool kFp8>
__device__ __forceinline__ float softmax_pass(uint32_t s_addr, int n8, const float *m_s, float scale,
                                              const int2 *vis_s, int G, int t, uint8_t *prow, long long *tr,
                                              int tile)
{
    float gmax = -INFINITY;
#pragma unroll 1
    for (int cb = 0; cb < n8; cb += 4) {
        uint32_t r[4][8];
        LVSPEC_TILE_TS(tr, 3, tile, (cb >> 2) * 3);         // asks for four chunks of S^T
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (cb + u < n8) tmem_ld_x8(s_addr + (cb + u) * 8, r[u]);
        tmem_wait_ld();
        LVSPEC_TILE_TS(tr, 3, tile, (cb >> 2) * 3 + 1);     // has them
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (cb + u < n8) {
                uint4 pk;
                gmax = fmaxf(gmax, exp_chunk<kMask, kFp8>(r[u], m_s + (cb + u) * 8, scale, vis_s + (cb + u) * 8,
                                                          (cb + u) * 8, G, t, pk));
                *reinterpret_cast<uint4 *>(prow + (cb + u) * 2048) = pk;
            }
        LVSPEC_TILE_TS(tr, 3, tile, (cb >> 2) * 3 + 2);     // their probabilities stored
    }
    return gmax;
}

// The same for a group that works on a share of the columns, chunks [c_lo, c_hi), of every
// tile: exp2 of its chunks of S^T (up to
// four TMEM loads in flight per wait), packed probabilities into pk, returns the
// largest scaled score.  kMask != 0: the tile reaches into the draft slots, so
// columns are masked by what their query may see; the common tile carries none of that.
template <int kMask, bool kFp8>
__device__ __forceinline__ float softmax_pass_share(uint32_t s_addr, int c_lo, int c_hi, const float *m_s,
                                              float scale, const int2 *vis_s, int G, int t,
                                              uint4 (&pk)[kMaxChunks])
{
    float gmax = -INFINITY;
#pragma unroll
    for (int h = 0; h < (kMaxChunks + 3) / 4; ++h) {
        const int cb = c_lo + 4 * h;
        if (cb < c_hi) {
            uint32_t r[4][8];
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (4 * h + u < kMaxChunks && cb + u < c_hi) tmem_ld_x8(s_addr + (cb + u) * 8, r[u]);
            tmem_wait_ld();
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (4 * h + u < kMaxChunks && cb + u < c_hi)
                    gmax = fmaxf(gmax, exp_chunk<kMask, kFp8>(r[u], m_s + (cb + u) * 8, scale, vis_s + (cb + u) * 8,
                                                              (cb + u) * 8, G, t, pk[4 * h + u]));
        }
    }
    return gmax;
}
// kTree: the draft slots hold several branches (the visibility table is only built
// and read then; the plain chain keeps its arithmetic mask).  kPaged: K and V are page
// pools and a tile's position in them comes from the sequence's block table.
// kFp8: E4M3 cache (tmap_q is not used: q is split into its two E4M3 tiles by the CTA).
// kTurns: the softmax groups take the tiles in turn; otherwise all groups work on every
// tile, each on a share of its columns (shorter per tile, and so at the two ends of a
// CTA's stream, but the per-tile overheads are paid by all twelve warps: the form for few
// query rows, where the stream is bound by HBM either way).
template <bool kTree, bool kPaged, bool kFp8, bool kTurns>
__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(const TcParams P, const SeqInfo seq, const __grid_constant__ CUtensorMap tmap_k,
               const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ CUtensorMap tmap_q)
{
    // bytes of one K or V tile: two 64-channel boxes at head_dim 128 (bf16), one box at
    // head_dim 64 and for an fp8 tile of 128 channels
    const uint32_t kSlot = (uint32_t)P.cfg.slot_bytes;
    const bool two_boxes = kSlot == kSlotBytes;
    const int D = P.a.D;
    extern __shared__ uint8_t smem_raw[];
    const AttnParams &p = P.a;
    const TcConfig cfg = P.cfg;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
#ifdef LVSPEC_TRACE
    unsigned long long *rec = nullptr;      // this CTA's record (one thread writes it)
    long long *tile_tr = nullptr;           // per-tile stamps of the one traced CTA (lane 0 of its warps)
    if (g_lvspec_trace && tid == 32) {
        const unsigned long long idx = atomicAdd(g_lvspec_trace, 1ull);
        if (idx < (unsigned long long)kTraceCtaRecords) {
            rec = g_lvspec_trace + 8 + idx * 8;
            rec[0] = 1;
            rec[1] = (unsigned long long)P.a.q;
            rec[2] = blockIdx.x + 1000 * blockIdx.y + 1000000 * blockIdx.z;
            rec[3] = lvspec_trace_now();
        }
    }
    if (g_lvspec_trace && blockIdx.x == 3 && blockIdx.y == 2 && blockIdx.z == 0 && lane == 0)
        tile_tr = reinterpret_cast<long long *>(g_lvspec_trace + 8 + 8 * kTraceCtaRecords);   // 4 roles x 32 tiles x 8 stamps
#else
    constexpr long long *tile_tr = nullptr;
#endif
    // the TMA unit fetches the descriptors while everything else is set up; a warp that
    // has nothing to do in the prologue asks for them, not the producer (whose first
    // load is what the whole CTA waits for)
    if (warp == kPvWarp) {
        if (lane == 0) prefetch_tensormap(&tmap_k);
        if (lane == 1 && !kFp8) prefetch_tensormap(&tmap_q);
        if (lane == 2) prefetch_tensormap(&tmap_v);
    }
    const int split = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
    const int L = seq.kv_len[b], vs = seq.span_start[b], ve = seq.span_end[b];
    const int M = p.M, G = p.G, gamma = p.gamma, NP = cfg.n_pad;
    const int n8 = (M + 7) >> 3;

    // tiles [t_begin, t_begin + T) of this split: equal shares, sizes differ by at most one
    const int n_tiles = (L + kTilePos - 1) / kTilePos;
    const int t_base = n_tiles / p.n_split, t_rem = n_tiles - t_base * p.n_split;
    const int t_begin = split * t_base + min(split, t_rem);
    const int T = t_base + (split < t_rem ? 1 : 0);

    const size_t unit = ((size_t)b * p.Hkv + kvh) * p.n_split + split;
    float *part_o = p.part_o + unit * (size_t)M * P.a.D;
    float *part_stat = p.part_stat + unit * (size_t)M * 4;
    if (T <= 0) {   // a split with no tile: contributes nothing
        if (tid == 0) {
            grid_dependency_wait();
            grid_launch_dependents();
        }
        __syncthreads();
        for (int r = tid; r < M; r += kThreads)
            *reinterpret_cast<float4 *>(part_stat + r * 4) = make_float4(kMFloor, 0.f, 0.f, 0.f);
        return;
    }

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gbase = smem_raw + (base - smem_u32(smem_raw));
    const SmemMap sm = smem_map(cfg);
    float *m_s = reinterpret_cast<float *>(gbase + sm.m);
    float *dl_s = reinterpret_cast<float *>(gbase + sm.dl);
    float *tmx_s = reinterpret_cast<float *>(gbase + sm.tmx);
    int2 *vis_s = reinterpret_cast<int2 *>(gbase + sm.vis);
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(gbase + sm.misc);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(gbase + sm.misc + 4);
    // how often the reference exponents m[] have been set or moved; tiles handed to the P.V issuer
    volatile uint32_t *epoch_s = reinterpret_cast<volatile uint32_t *>(gbase + sm.misc + 8);
    volatile uint32_t *committed_s = reinterpret_cast<volatile uint32_t *>(gbase + sm.misc + 12);

    // barrier addresses
    const uint32_t bar0 = base + sm.bars;
    auto k_full = [&](int s) { return bar0 + 8 * s; };
    auto k_empty = [&](int s) { return bar0 + 8 * (cfg.ks + s); };
    auto v_full = [&](int s) { return bar0 + 8 * (2 * cfg.ks + s); };
    auto v_empty = [&](int s) { return bar0 + 8 * (2 * cfg.ks + cfg.vs + s); };
    const uint32_t bar1 = bar0 + 8 * (2 * cfg.ks + 2 * cfg.vs);
    // The hand-over barriers of tile i are those of index i % 3, whatever the number of
    // S^T and P^T buffers: a parity wait tells a phase from its neighbours only, so whoever
    // waits for a phase must know the phase before it to be over.  Each of these
    // barriers belongs to the tiles of one softmax group, which sees its phases in order.
    auto s_full = [&](int i) { return bar1 + 8 * (i % kSoftmaxGroups); };
    auto s_free = [&](int i) { return bar1 + 8 * (kSoftmaxGroups + i % kSoftmaxGroups); };
    auto p_full = [&](int i) { return bar1 + 8 * (2 * kSoftmaxGroups + i % kSoftmaxGroups); };
    auto p_free = [&](int i) { return bar1 + 8 * (3 * kSoftmaxGroups + i % kSoftmaxGroups); };
    auto hand_parity = [](int i) { return (uint32_t)(i / kSoftmaxGroups) & 1u; };
    const uint32_t drain_bar = bar1 + 8 * (4 * kSoftmaxGroups);
    const uint32_t done_bar = drain_bar + 8;
    const uint32_t q_full = drain_bar + 16;
    const uint32_t pv_done = drain_bar + 24;
    const int bh = b * p.Hkv + kvh;

    // the cache is read once per call: it should not push the split partials out of L2
    const uint64_t stream_policy = l2_evict_first_policy();
    // where tile i of this split sits in the [sequences or pages, heads, positions, 128]
    // maps: (position, sequence or page)
    volatile int32_t *page_s = reinterpret_cast<volatile int32_t *>(gbase + sm.pages);
    auto tile_at = [&](int i, int &pos0, int &map_row) {
        pos0 = (t_begin + i) * kTilePos;
        map_row = b;
        if (kPaged) {
            // a page holds a whole number of tiles; an entry outside the pool reads as zeros
            pos0 -= (pos0 / p.page_size) * p.page_size;
            map_row = page_s[i];
        }
    };
    auto load_k = [&](int i) {
        const int ks = i % cfg.ks;
        int pos0, map_row;
        tile_at(i, pos0, map_row);
        mbar_arrive_expect_tx(k_full(ks), kSlot);
        tma_load_4d_hint(base + sm.k + ks * kSlot, &tmap_k, k_full(ks), 0, pos0, kvh, map_row, stream_policy);
        if (two_boxes)
            tma_load_4d_hint(base + sm.k + ks * kSlot + kBoxBytes, &tmap_k, k_full(ks), 64, pos0, kvh, map_row,
                             stream_policy);
    };
    auto load_v = [&](int i) {
        const int vsl = i % cfg.vs;
        int pos0, map_row;
        tile_at(i, pos0, map_row);
        mbar_arrive_expect_tx(v_full(vsl), kSlot);
        tma_load_4d_hint(base + sm.v + vsl * kSlot, &tmap_v, v_full(vsl), 0, pos0, kvh, map_row, stream_policy);
        if (two_boxes)
            tma_load_4d_hint(base + sm.v + vsl * kSlot + kBoxBytes, &tmap_v, v_full(vsl), 64, pos0, kvh, map_row,
                             stream_policy);
    };

    // ------------------------------------------------------------------ prologue
    // The producer thread sets the barriers up and starts the first loads at
    // once; the other warps prepare shared memory and TMEM meanwhile.
    int first_k = 0, first_v = 0;   // loads issued before the CTA-wide barrier
    if (warp == 0) {
        {
            // one barrier per lane, all at once (an mbarrier.init costs about a hundred
            // cycles): barriers sit in the order k_full, k_empty, v_full, v_empty,
            // s_full[3], s_free[3], p_full[3], p_free[3], drain, done, q_full, pv_done
            const int n_kv = 2 * cfg.ks + 2 * cfg.vs;
            constexpr int n_sp = 4 * kSoftmaxGroups;
            const int n_bars = n_kv + n_sp + 4;
            for (int i = lane; i < n_bars; i += 32) {
                const int j = i - n_kv;          // index among the barriers after the rings
                uint32_t count = 1;
                if (j >= kSoftmaxGroups && j < 3 * kSoftmaxGroups) count = kTurns ? 4 : kSoftmaxWarps;   // s_free, p_full: the warps that work on a tile
                else if (j == n_sp + 1) count = kSoftmaxWarps + 1;              // done
                else if (kFp8 && j == n_sp + 2) count = kSoftmaxWarps;          // q_full: the warps that split q
                mbar_init(bar0 + 8 * i, count);
            }
            if (lane == 0) {
                *abort_flag = 0;
                *epoch_s = 0;
                *committed_s = 0;
            }
            mbar_fence_init();
            fence_proxy_async_smem();
        }
        __syncwarp();
        if (kPaged) {
            // the block table too may come from the kernel before this one: the warp reads
            // this split's entries (one per tile) after the wait, then lane 0 goes on
            grid_dependency_wait();
            const int32_t *row = p.block_table + (size_t)b * p.pages_per_seq;
            for (int i = lane; i < T; i += 32) page_s[i] = __ldg(row + ((t_begin + i) * kTilePos) / p.page_size);
            __syncwarp();
        }
        if (lane == 0) {
            // inputs may come from the kernel before this one in the stream
            grid_dependency_wait();
            // the first K tile comes from HBM and is needed first: it goes out before Q
            first_k = min(T, cfg.ks);
            first_v = min(T, cfg.vs);
            load_k(0);
            if (!kFp8) {
                mbar_arrive_expect_tx(q_full, (uint32_t)(M * D) * 2u);
                tma_load_4d(base + sm.q, &tmap_q, q_full, 0, kvh * G, 0, b);
                if (two_boxes) tma_load_4d(base + sm.q + NP * 128, &tmap_q, q_full, 64, kvh * G, 0, b);
            }
            for (int i = 0; i < first_v; ++i) {
                if (i > 0 && i < first_k) load_k(i);
                load_v(i);
            }
            for (int i = max(first_v, 1); i < first_k; ++i) load_k(i);    // a K ring deeper than the V ring
        }
        __syncwarp();
    } else if (warp == 1) {
        tmem_alloc(base + sm.misc, (uint32_t)cfg.tmem_cols);
        tmem_relinquish();
    } else if (warp < kPvWarp) {
        const int idx = tid - 64;   // 0..kSoftmaxThreads-1
        // rows M..NP-1 of Q are padding: zero them (the TMA boxes cover rows < M only;
        // with an fp8 cache the split of q below writes every row)
        for (int i = idx; !kFp8 && i < (NP - M) * 16; i += kSoftmaxThreads) {
            const int r = M + (i >> 4), c = i & 15, h = c >> 3, cc = c & 7;
            *reinterpret_cast<uint4 *>(gbase + sm.q + h * (NP * 128) + r * 128 + cc * 16) =
                make_uint4(0, 0, 0, 0);
        }
        // P buffers start as zeros (columns beyond the last chunk stay zero)
        for (uint32_t i = idx * 16; i < (uint32_t)(cfg.pb * NP * 256); i += kSoftmaxThreads * 16)
            *reinterpret_cast<uint4 *>(gbase + sm.p + i) = make_uint4(0, 0, 0, 0);
        for (int n = idx; n < NP; n += kSoftmaxThreads) {
            m_s[n] = kFp8 ? kMFloor : 0.f;
            if (kTree) {
                // the draft slots column n's query sees: its branch's first slot .. its own slot
                const int qi = n / G;
                vis_s[n] = qi < gamma ? make_int2((qi / p.branch_len) * p.branch_len, qi)
                                      : make_int2(1 << 30, (1 << 30) - 1);
            }
        }
        // constant 64 x 16 tiles (K-major, no swizzle: the 8 positions of chunk c
        // at c * 1024, row r at (r / 8) * 128 + (r % 8) * 16).  Row 0 = ones (sums
        // l), row 1 = 1 inside the visual span (sums l_vis), rows 2.. = 0.
        // tile 0: block inside the span, 1: outside, 2: the 16-block holding the
        // span start, 3: the 16-block holding the span end
        // (fp8 cache: the tiles are 64 x 32 E4M3, 16 positions per 16-byte chunk, and the
        // boundary tiles cover the 32-block holding the span's start / end)
        for (uint32_t i = idx * 16; i < 4 * kA2Bytes; i += kSoftmaxThreads * 16) {
            const int tile = i / kA2Bytes, off = i % kA2Bytes;
            const int c = off / 1024, rr = (off % 1024) / 16;   // rr = row index 0..63
            uint4 val = make_uint4(0, 0, 0, 0);
            if (rr < 2) {
                constexpr int kPer = kFp8 ? 16 : 8;             // positions per 16-byte chunk
                uint32_t w[4] = {0, 0, 0, 0};
#pragma unroll
                for (int k = 0; k < kPer; ++k) {
                    int ind = 1;
                    if (rr == 1) {
                        if (tile == 0) ind = 1;
                        else if (tile == 1) ind = 0;
                        else {
                            const int pos = ((tile == 2 ? vs : ve) & ~(2 * kPer - 1)) + c * kPer + k;
                            ind = (pos >= vs && pos < ve) ? 1 : 0;
                        }
                    }
                    if (kFp8) w[k >> 2] |= (ind ? 0x38u : 0u) << (8 * (k & 3));       // E4M3 1.0
                    else w[k >> 1] |= (ind ? 0x3F80u : 0u) << (16 * (k & 1));         // bf16 1.0
                }
                val = make_uint4(w[0], w[1], w[2], w[3]);
            }
            *reinterpret_cast<uint4 *>(gbase + sm.a2 + i) = val;
        }
        fence_proxy_async_smem();
    }
    // nobody polls a barrier while the grid before this one is still running
    grid_dependency_wait();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
#ifdef LVSPEC_TRACE
    if (rec) rec[4] = lvspec_trace_now();
#endif
    const uint32_t tmem_base = *tmem_slot;
    // accumulator columns: the S^T buffers, then O^T and the sums (fp8 cache: two columns per row)
    constexpr int kAccCols = kFp8 ? 2 : 1;
    const uint32_t tm_s0 = tmem_base, tm_o = tmem_base + cfg.sb * NP, tm_l = tm_o + kAccCols * NP;
    float scale_cta = p.scale_log2;     // softmax scale of this CTA (fp8 cache: with the K scale and q's shift)
    float v_scale = 1.f;
    if (kFp8 && warp >= kSoftmaxWarp0 && warp < kPvWarp) {
        // ---- q as two E4M3 operand tiles (128-byte swizzle, one 128-byte row per query row)
        // chunk = 8 channels of one row (16 bytes of bf16 in, 8 + 8 bytes out)
        const int idx = tid - 32 * kSoftmaxWarp0;
        const int n_chunks = NP * 16;
        constexpr int kMine = (kMaxRowsFp8 * 16 + kSoftmaxThreads - 1) / kSoftmaxThreads;
        uint4 qv[kMine];
        float amax = 0.f;
#pragma unroll
        for (int u = 0; u < kMine; ++u) {
            const int ch = idx + u * kSoftmaxThreads;
            qv[u] = make_uint4(0, 0, 0, 0);
            if (ch < n_chunks) {
                const int n = ch >> 4, c = ch & 15;
                if (n < M) {
                    const int g = n / G, hg = n - g * G;
                    qv[u] = __ldg(reinterpret_cast<const uint4 *>(
                        p.q + (((size_t)b * gamma + g) * p.Hq + kvh * G + hg) * 128 + c * 8));
                }
                const uint32_t w[4] = {qv[u].x, qv[u].y, qv[u].z, qv[u].w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    amax = fmaxf(amax, fabsf(__uint_as_float(w[k] << 16)));
                    amax = fmaxf(amax, fabsf(__uint_as_float(w[k] & 0xFFFF0000u)));
                }
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
        volatile float *wmax = reinterpret_cast<volatile float *>(gbase + sm.misc + 16);
        if (lane == 0) wmax[warp - kSoftmaxWarp0] = amax;
        asm volatile("bar.sync %0, %1;" ::"r"(kQBarrier), "r"(kSoftmaxThreads) : "memory");
        amax = 0.f;
#pragma unroll
        for (int u = 0; u < kSoftmaxWarps; ++u) amax = fmaxf(amax, wmax[u]);
        // power of two that brings the largest magnitude into [128, 256) (NaN or Inf in q:
        // no shift; the result is then NaN as it would be with any cache)
        int shift = 0;
        if (amax > 0.f && amax < INFINITY) shift = 7 - ((int)((__float_as_uint(amax) >> 23) & 0xFF) - 127);
        shift = max(-100, min(100, shift));
        const float up = __uint_as_float((uint32_t)(127 + shift) << 23);
#pragma unroll
        for (int u = 0; u < kMine; ++u) {
            const int ch = idx + u * kSoftmaxThreads;
            if (ch < n_chunks) {
                const int n = ch >> 4, c = ch & 15;
                const uint32_t w[4] = {qv[u].x, qv[u].y, qv[u].z, qv[u].w};
                uint32_t hd[4], rs[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const float x0 = __uint_as_float(w[k] << 16) * up, x1 = __uint_as_float(w[k] & 0xFFFF0000u) * up;
                    const float h0 = e4m3_head(x0), h1 = e4m3_head(x1);
                    hd[k] = pack_e4m3x2(h0, h1);
                    rs[k] = pack_e4m3x2(x0 - h0, x1 - h1);
                }
                const uint32_t off = n * 128 + (((c >> 1) ^ (n & 7)) << 4) + ((c & 1) << 3);
                *reinterpret_cast<uint2 *>(gbase + sm.q + off) = make_uint2(hd[0] | (hd[1] << 16), hd[2] | (hd[3] << 16));
                *reinterpret_cast<uint2 *>(gbase + sm.q + NP * 128 + off) =
                    make_uint2(rs[0] | (rs[1] << 16), rs[2] | (rs[3] << 16));
            }
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(q_full);
        scale_cta = p.scale_log2 * __ldg(p.k_scale + bh) * __uint_as_float((uint32_t)(127 - shift) << 23);
        v_scale = __ldg(p.v_scale + bh);
    }

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int nk = first_k, nv = first_v;   // loads issued so far
            // K and V slots free up at different times: poll both, never block on one
            uint64_t idle_since = 0;
            uint32_t spin = 0;
            while (nk < T || nv < T) {
                bool progress = false;
                if (nk < T && mbar_test_wait(k_empty(nk % cfg.ks), ((nk / cfg.ks) - 1) & 1)) {
                    load_k(nk);
                    ++nk;
                    progress = true;
                }
                if (nv < T && mbar_test_wait(v_empty(nv % cfg.vs), ((nv / cfg.vs) - 1) & 1)) {
                    load_v(nv);
                    ++nv;
                    progress = true;
                }
                if (progress) {
                    idle_since = 0;
                } else {
                    if (*abort_flag) break;
                    if ((++spin & 255u) == 0) {
                        const uint64_t now = global_timer_ns();
                        if (idle_since == 0) idle_since = now;
                        else if (now - idle_since > 2000000000ull) {
                            *abort_flag = 1;
                            break;
                        }
                    }
                }
            }
            if (*abort_flag) {
                // wait (bounded) for the copies still in flight before the CTA leaves
                wait_unconditional(q_full, 0);
                for (int j = max(0, nk - cfg.ks); j < nk; ++j)
                    wait_unconditional(k_full(j % cfg.ks), (j / cfg.ks) & 1);
                for (int j = max(0, nv - cfg.vs); j < nv; ++j)
                    wait_unconditional(v_full(j % cfg.vs), (j / cfg.vs) & 1);
            }
        }
    } else if (warp == 1) {
        // -------------------------------------------------------------- MMA issuer
        // The whole warp runs the loop and one elected lane issues: the descriptors are
        // then the same in every lane and the compiler can keep them where the MMA
        // instruction takes its operands from, instead of moving them there per instruction.
        {
            const uint32_t idesc_qk = kFp8 ? make_idesc_e4m3(128, NP, 0, 0) : make_idesc_bf16(128, NP, 0, 0);
            // descriptors: everything but the start address is fixed, and the start
            // address field (address / 16) moves by compile-time steps
            const uint64_t kd0 = make_smem_desc(base + sm.k, 16, 1024, kSwizzle128B);
            uint64_t qd[8];
#pragma unroll
            for (int j = 0; j < 8; ++j)
                qd[j] = make_smem_desc(base + sm.q + (j >> 2) * (NP * 128) + (j & 3) * 32, 16, 1024,
                                       kSwizzle128B);
            Ring k_ring(cfg.ks), s_ring(cfg.sb), hand(kSoftmaxGroups), freed(kSoftmaxGroups);
            auto issue_qk = [&](int i) -> bool {
                const int ks = k_ring.idx, sb = s_ring.idx;
                LVSPEC_TILE_TS(tile_tr, 1, i, 0);     // starts waiting for the K tile
                bool there = mbar_wait(k_full(ks), k_ring.parity, abort_flag);
                LVSPEC_TILE_TS(tile_tr, 1, i, 1);     // K tile there
                // the tile that used this S^T buffer last (tile i - sb) has been read
                if (i >= cfg.sb) {
                    there = mbar_wait(bar1 + 8 * (kSoftmaxGroups + freed.idx), freed.parity, abort_flag) && there;
                    freed.next();
                }
                if (!__all_sync(0xffffffffu, there)) return false;
                LVSPEC_TILE_TS(tile_tr, 1, i, 2);     // S^T buffer free
                tc_fence_after();
                const uint64_t kd = kd0 + (uint64_t)(ks * (kSlot >> 4));
                const uint32_t d = tm_s0 + sb * NP;
                // bf16: 8 steps of 16 channels over the two 64-channel boxes (4 over the one box
                // of head_dim 64); fp8: 4 steps of 32 channels against q's leading bits, then the
                // same 4 against the rest
                if (elect_one()) {
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        if (kFp8) mma_f8_ss(d, kd + (uint64_t)((j & 3) * 2), qd[j], idesc_qk, j > 0);
                        else if (j < 4 || two_boxes)
                            mma_f16_ss(d, kd + (uint64_t)((j >> 2) * (kBoxBytes >> 4) + (j & 3) * 2), qd[j],
                                       idesc_qk, j > 0);
                    }
                    mma_commit(bar1 + 8 * hand.idx);      // s_full of tile i
                    mma_commit(k_empty(ks));
                }
                __syncwarp();
                LVSPEC_TILE_TS(tile_tr, 1, i, 3);     // K.Q^T issued
                k_ring.next();
                s_ring.next();
                hand.next();
                return true;
            };
            bool ok = __all_sync(0xffffffffu, mbar_wait(q_full, 0, abort_flag));
            for (int i = 0; ok && i < T; ++i) ok = issue_qk(i);
            // every MMA issued by the elected lane has finished before TMEM is released
            if (elect_one()) {
                mma_commit(drain_bar);
                wait_unconditional(drain_bar, 0);
            }
            __syncwarp();
        }
    } else if (warp == kPvWarp) {
        // ------------------------------------------------- P.V and sum MMA issuer
        // (whole warp in the loop, one elected lane issues: see the K.Q^T issuer)
        {
            const uint32_t idesc_pv = kFp8 ? make_idesc_e4m3(128, 2 * NP, 1, 1) : make_idesc_bf16(128, NP, 1, 1);
            const uint32_t idesc_sum = kFp8 ? make_idesc_e4m3(64, 2 * NP, 0, 1) : make_idesc_bf16(64, NP, 0, 1);
            // one MMA covers 16 positions of a bf16 tile, 32 of an fp8 tile
            constexpr int kSteps = kFp8 ? 4 : 8, kStepPos = kTilePos / kSteps;
            constexpr uint32_t kVStep = kStepPos * 128 >> 4, kPStep = kStepPos * 16 >> 4;   // descriptor units
            const uint64_t vd0 = make_smem_desc(base + sm.v, kBoxBytes, 1024, kSwizzle128B);
            const uint64_t pd0 = make_smem_desc(base + sm.p, 128, 2048, kSwizzleNone);
            const uint64_t a2d0 = make_smem_desc(base + sm.a2, 1024, 128, kSwizzleNone);
            Ring v_ring(cfg.vs), p_ring(cfg.pb), hand(kSoftmaxGroups);
            for (int i = 0; i < T; ++i, v_ring.next(), p_ring.next(), hand.next()) {
                const int pb = p_ring.idx, vsl = v_ring.idx;
                LVSPEC_TILE_TS(tile_tr, 2, i, 0);     // starts waiting for P^T
                bool there = mbar_wait(bar1 + 8 * (2 * kSoftmaxGroups + hand.idx), hand.parity, abort_flag);   // p_full of tile i
                LVSPEC_TILE_TS(tile_tr, 2, i, 1);     // P^T there
                there = mbar_wait(v_full(vsl), v_ring.parity, abort_flag) && there;
                if (!__all_sync(0xffffffffu, there)) break;
                LVSPEC_TILE_TS(tile_tr, 2, i, 2);     // V tile there
                tc_fence_after();
                // V^T: channels contiguous (M-major), 64-channel halves kBoxBytes apart,
                // groups of 8 positions 1024 bytes apart.  (At head_dim 64 the product still
                // has 128 rows: its upper half reads whatever follows the box in shared memory
                // and lands in TMEM lanes nobody reads.)  P^T: rows contiguous in
                // 16-byte chunks (N-major), chunk stride 2048, groups of 8 positions 128
                // bytes apart.
                const uint64_t vd = vd0 + (uint64_t)(vsl * (kSlot >> 4));
                const uint64_t pd = pd0 + (uint64_t)(pb * ((NP * 256) >> 4));
                const int pos0 = (t_begin + i) * kTilePos;
                // constant tile per block of 16 (fp8: 32) positions: 0 inside the span, 1
                // outside, 2 / 3 the blocks holding the span's start / end
                int uniform = -1;
                if (pos0 >= vs && pos0 + kTilePos <= ve) uniform = 0;
                else if (pos0 + kTilePos <= vs || pos0 >= ve) uniform = 1;
                const uint32_t first_acc = i > 0 ? 1u : 0u;
                if (!elect_one()) {
                    // the other lanes wait at the end of the turn
                } else if (uniform >= 0) {
                    const uint64_t d2 = a2d0 + (uint64_t)(uniform * (kA2Bytes >> 4));
#pragma unroll
                    for (int j = 0; j < kSteps; ++j)
                        mma_ss<kFp8>(tm_l, d2, pd + (uint64_t)(j * kPStep), idesc_sum, j > 0 ? 1u : first_acc);
#pragma unroll
                    for (int j = 0; j < kSteps; ++j)
                        mma_ss<kFp8>(tm_o, vd + (uint64_t)(j * kVStep), pd + (uint64_t)(j * kPStep), idesc_pv,
                                     j > 0 ? 1u : first_acc);
                } else {
#pragma unroll
                    for (int j = 0; j < kSteps; ++j) {
                        const uint32_t acc = j > 0 ? 1u : first_acc;
                        const int pblk = pos0 + kStepPos * j;
                        int tile;
                        if (pblk >= vs && pblk + kStepPos <= ve) tile = 0;
                        else if (pblk + kStepPos <= vs || pblk >= ve) tile = 1;
                        else if ((vs & ~(kStepPos - 1)) == pblk) tile = 2;
                        else tile = 3;
                        mma_ss<kFp8>(tm_o, vd + (uint64_t)(j * kVStep), pd + (uint64_t)(j * kPStep), idesc_pv, acc);
                        mma_ss<kFp8>(tm_l, a2d0 + (uint64_t)(tile * (kA2Bytes >> 4)),
                                     pd + (uint64_t)(j * kPStep), idesc_sum, acc);
                    }
                }
                if (elect_one()) {
                    mma_commit(v_empty(vsl));
                    mma_commit(bar1 + 8 * (3 * kSoftmaxGroups + hand.idx));     // p_free of tile i
                }
                __syncwarp();
                LVSPEC_TILE_TS(tile_tr, 2, i, 3);     // sums and P.V issued
            }
            // the elected lane's MMAs have finished: tell the softmax warps and the TMEM owner
            if (elect_one()) {
                mma_commit(pv_done);
                mma_commit(done_bar);
            }
            __syncwarp();
        }
    } else {
        // ------------------------------------------------------------ softmax warps
        const int grp = (warp - kSoftmaxWarp0) >> 2;    // tiles grp, grp + 3, ... are this group's
        const int bar_id = 1 + grp;
        const int wq = warp & 3;                        // TMEM lane quarter of this warp
        const int row = wq * 32 + lane;                 // TMEM lane = position inside the tile
        const int gtid = ((warp - kSoftmaxWarp0) & 3) * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(wq * 32) << 16;
        const float scale = scale_cta;
        constexpr float kLimit = kFp8 ? kGuard8 : kGuard;    // a score this far above m moves m
        constexpr float kLift = kFp8 ? kHead8 : 0.f;         // where the reference position sits above m
        // this group's share of the columns (all tiles without turns; the epilogue always):
        // chunks of 8 columns [c_lo, c_hi), equal shares, at most kMaxChunks
        const int c_base = n8 / kSoftmaxGroups, c_rem = n8 - c_base * kSoftmaxGroups;
        const int c_lo = grp * c_base + min(grp, c_rem), c_hi = c_lo + c_base + (grp < c_rem ? 1 : 0);
        if constexpr (kTurns) {
            // bounded wait for a shared-memory counter to reach a value (the groups' turns)
            auto wait_counter = [&](volatile uint32_t *ctr, uint32_t at_least) {
                if (*ctr >= at_least) return;
                uint64_t t0 = 0;
                for (uint32_t spin = 1;; ++spin) {
                    if (*ctr >= at_least || *abort_flag) return;
                    if ((spin & 1023u) == 0) {
                        const uint64_t now = global_timer_ns();
                        if (t0 == 0) t0 = now;
                        else if (now - t0 > 2000000000ull) {
                            *abort_flag = 1;
                            return;
                        }
                    }
                }
            };
            // buffers of this group's tile advance by counting, not by dividing
            int sbi = grp % cfg.sb, pb = grp % cfg.pb;
            auto advance = [](int &idx, int n) {
                idx += kSoftmaxGroups;
                while (idx >= n) idx -= n;
            };
            for (int i = grp; i < T; i += kSoftmaxGroups) {
                const int pos0 = (t_begin + i) * kTilePos;
                const int pos = pos0 + row;
                if (warp == kSoftmaxWarp0) LVSPEC_TILE_TS(tile_tr, 0, i, 0);     // starts waiting for S^T
                mbar_wait(s_full(i), hand_parity(i), abort_flag);
                if (warp == kSoftmaxWarp0) LVSPEC_TILE_TS(tile_tr, 0, i, 1);     // S^T there
                tc_fence_after();
                const uint32_t s_addr = tm_s0 + sbi * NP + lane_addr;
                // The oldest uncommitted tile is the one whose group may move m.  Tile 0 is that
                // from the start and sets m up; the others read m under an epoch and check it
                // when their turn comes.
                bool my_turn = i == 0;
                uint32_t e0 = 0;
                if (i == 0) {
                    if (!kFp8) {
                        // reference exponent of each row: its score at the split's first position
                        // (every warp reads the chunks c8 = its quarter, quarter + 4, ... from the TMEM
                        // lanes it can reach; only the first quarter holds position 0)
                        if (wq == 0) {
#pragma unroll 1
                            for (int cb = 0; cb < n8; cb += 2) {
                                uint32_t r[2][8];
#pragma unroll
                                for (int u = 0; u < 2; ++u)
                                    if (cb + u < n8) tmem_ld_x8(s_addr + (cb + u) * 8, r[u]);
                                tmem_wait_ld();
                                if (lane == 0) {
#pragma unroll
                                    for (int u = 0; u < 2; ++u)
                                        if (cb + u < n8) {
#pragma unroll
                                            for (int k = 0; k < 8; ++k)
                                                m_s[(cb + u) * 8 + k] = __uint_as_float(r[u][k]) * scale - kLift;
                                        }
                                }
                            }
                        }
                        group_sync(bar_id);
                        if (gtid == 0) {
                            __threadfence_block();
                            *epoch_s = 1;
                        }
                    }
                } else {
                    if (i < kSoftmaxGroups) wait_counter(epoch_s, 1);     // m comes from the first tile
                    e0 = *epoch_s;
                    __threadfence_block();
                }
                const bool tail = pos0 + kTilePos > L - gamma;
                const int gmin = pos - L + gamma;           // tail index of `pos`: queries below it do not see it
                // P^T goes straight to shared memory: the P.V product that read this buffer last is done
                // (tile i - pb; this group saw tile i - 3 - pb's product done a turn ago)
                if (i >= cfg.pb) mbar_wait(p_free(i - cfg.pb), hand_parity(i - cfg.pb), abort_flag);
                if (warp == kSoftmaxWarp0) LVSPEC_TILE_TS(tile_tr, 0, i, 2);     // P buffer free
                uint8_t *prow = gbase + sm.p + pb * (NP * 256) + row * 16;

                // fp8 cache: E4M3 has 17 binades, so the reference exponent of a row starts
                // from the largest score of the split's first tile (the path below), not
                // from whatever score its first position happens to have
                bool take_max = kFp8 && i == 0;
                for (int attempt = 0; attempt < 4; ++attempt) {
                    float gmax = -INFINITY;
                    if (!take_max)
                        gmax = !tail ? softmax_pass<0, kFp8>(s_addr, n8, m_s, scale, vis_s, G, gmin, prow,
                                                             warp == kSoftmaxWarp0 ? tile_tr : nullptr, i)
                                     : softmax_pass<kTree ? 2 : 1, kFp8>(s_addr, n8, m_s, scale, vis_s, G, gmin, prow, nullptr, i);
                    if (warp == kSoftmaxWarp0) LVSPEC_TILE_TS(tile_tr, 0, i, 3);     // exponentials done
                    if (!my_turn) {
                        wait_counter(committed_s, (uint32_t)i);
                        my_turn = true;
                        __threadfence_block();
                        const uint32_t e1 = *epoch_s;       // final: only this group can move m now
                        const bool stale = e1 != e0;
                        if (!group_any(bar_id, stale || gmax > kLimit)) break;
                        // m moved while some thread computed under the old one: once more
                        if (group_any(bar_id, stale)) continue;
                    } else if (!take_max && !group_any(bar_id, gmax > kLimit)) {
                        break;
                    }
                    take_max = false;

                    // ---- a score ran past the guard: move m up to the tile maximum ----
                    // (the masked form, with its divisions, only where the tile reaches the draft slots)
                    auto tile_max = [&](auto masked) {
#pragma unroll 1
                        for (int c8 = 0; c8 < n8; ++c8) {
                            uint32_t r[8];
                            tmem_ld_x8(s_addr + c8 * 8, r);
                            tmem_wait_ld();
                            // eight reductions in flight, then their results stored
                            float s2[8];
#pragma unroll
                            for (int k = 0; k < 8; ++k) {
                                s2[k] = __uint_as_float(r[k]) * scale;
                                if constexpr (decltype(masked)::value) {
                                    if (kTree ? !column_sees(vis_s[c8 * 8 + k], gmin) : (c8 * 8 + k) / G < gmin)
                                        s2[k] = -INFINITY;
                                }
                            }
#pragma unroll
                            for (int k = 0; k < 8; ++k) s2[k] = warp_max_f32(s2[k]);
                            if (lane == 0) {
                                float *dst = tmx_s + wq * NP + c8 * 8;
                                *reinterpret_cast<float4 *>(dst) = make_float4(s2[0], s2[1], s2[2], s2[3]);
                                *reinterpret_cast<float4 *>(dst + 4) = make_float4(s2[4], s2[5], s2[6], s2[7]);
                            }
                        }
                    };
                    if (tail) tile_max(std::true_type{});
                    else tile_max(std::false_type{});
                    group_sync(bar_id);
                    for (int n = gtid; n < n8 * 8; n += 128) {
                        const float mt = fmaxf(fmaxf(tmx_s[n], tmx_s[NP + n]),
                                               fmaxf(tmx_s[2 * NP + n], tmx_s[3 * NP + n])) - kLift;
                        const float mo = m_s[n];
                        const float mn = fmaxf(mo, mt);
                        dl_s[n] = mo - mn;              // <= 0
                        m_s[n] = mn;
                    }
                    group_sync(bar_id);
                    if (gtid == 0) {
                        __threadfence_block();
                        *epoch_s = *epoch_s + 1;
                    }
                    if (i > 0) {
                        // O^T and the sums were accumulated under the old m: rescale them once
                        // the P.V product of tile i - 1 has finished (tile i - 1 is committed, so
                        // its group has seen the product of tile i - 4 or a later one done)
                        mbar_wait(p_free(i - 1), hand_parity(i - 1), abort_flag);
                        tc_fence_after();
                        // (fp8 cache: accumulator columns 2n and 2n + 1 belong to row n)
                        for (int c = 0; c < n8 * kAccCols; ++c) {
                            uint32_t r[8];
                            tmem_ld_x8(tm_o + lane_addr + c * 8, r);
                            tmem_wait_ld();
#pragma unroll
                            for (int k = 0; k < 8; ++k)
                                r[k] = __float_as_uint(__uint_as_float(r[k]) * ex2(dl_s[(c * 8 + k) / kAccCols]));
                            tmem_st_x8(tm_o + lane_addr + c * 8, r);
                            if (wq == 0) {
                                tmem_ld_x8(tm_l + c * 8, r);
                                tmem_wait_ld();
#pragma unroll
                                for (int k = 0; k < 8; ++k)
                                    r[k] = __float_as_uint(__uint_as_float(r[k]) * ex2(dl_s[(c * 8 + k) / kAccCols]));
                                tmem_st_x8(tm_l + c * 8, r);
                            }
                        }
                        tmem_wait_st();
                        tc_fence_before();
                    }
                    group_sync(bar_id);
                }
                if (warp == kSoftmaxWarp0) LVSPEC_TILE_TS(tile_tr, 0, i, 4);     // this tile's turn came and m stood
                // m stands for this tile: the next tile's group may take its turn
                if (gtid == 0) {
                    __threadfence_block();
                    *committed_s = (uint32_t)i + 1;
                }
                if (pos0 + kTilePos > L) {
                    // slots at or beyond kv_len hold whatever the cache holds: zero their V
                    // rows so that 0 * junk cannot poison the accumulators.  Once the product of
                    // tile i - 1 is done, the V slot's barrier can only be in this tile's phase.
                    if (i > 0) mbar_wait(p_free(i - 1), hand_parity(i - 1), abort_flag);
                    const int vsl = i % cfg.vs;
                    mbar_wait(v_full(vsl), (i / cfg.vs) & 1, abort_flag);
                    if (pos >= L) {
                        uint8_t *vrow = gbase + sm.v + vsl * kSlot + row * 128;
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            *reinterpret_cast<uint4 *>(vrow + c * 16) = make_uint4(0, 0, 0, 0);
                            if (two_boxes) *reinterpret_cast<uint4 *>(vrow + kBoxBytes + c * 16) = make_uint4(0, 0, 0, 0);
                        }
                    }
                }
                // one arrival per warp: S^T has been read (the K.Q^T of a later tile may overwrite
                // it) and P^T, with any zeroed V rows, is in shared memory
                tc_fence_before();
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(s_free(i));
                    mbar_arrive(p_full(i));
                }
                if (warp == kSoftmaxWarp0) LVSPEC_TILE_TS(tile_tr, 0, i, 5);     // P^T handed over
                advance(sbi, cfg.sb);
                advance(pb, cfg.pb);
            }
        } else {
            // ring positions advance by counting, not by dividing
            int pb = 0, vsl = 0;                 // P buffer and V slot of tile i
            uint32_t pb_round = 0, vs_round = 0; // how often each ring has wrapped
            for (int i = 0; i < T; ++i) {
                const int pos0 = (t_begin + i) * kTilePos;
                const int pos = pos0 + row;
                const int sb = i & 1;
                if (warp == kSoftmaxWarp0) LVSPEC_TILE_TS(tile_tr, 0, i, 0);     // starts waiting for S^T
                mbar_wait(s_full(i), hand_parity(i), abort_flag);
                if (warp == kSoftmaxWarp0) LVSPEC_TILE_TS(tile_tr, 0, i, 1);     // S^T there
                tc_fence_after();
                const uint32_t s_addr = tm_s0 + sb * NP + lane_addr;
                if (!kFp8 && i == 0) {
                    // reference exponent of each row: its score at the split's first position
                    if (wq == 0) {
                        for (int c8 = c_lo; c8 < c_hi; ++c8) {
                            uint32_t r[8];
                            tmem_ld_x8(s_addr + c8 * 8, r);
                            tmem_wait_ld();
                            if (lane == 0) {
#pragma unroll
                                for (int k = 0; k < 8; ++k) m_s[c8 * 8 + k] = __uint_as_float(r[k]) * scale - kLift;
                            }
                        }
                    }
                    group_sync(bar_id);
                }
                const bool tail = pos0 + kTilePos > L - gamma;
                const int gmin = pos - L + gamma;           // tail index of `pos`: queries below it do not see it
                uint8_t *prow = gbase + sm.p + pb * (NP * 256) + row * 16;
                uint4 pk[kMaxChunks];   // this position's probabilities, 8 columns per entry

                for (int attempt = 0; attempt < 3; ++attempt) {
                    // fp8 cache: E4M3 has 17 binades, so the reference exponent of a row starts
                    // from the largest score of the split's first tile (the path below), not
                    // from whatever score its first position happens to have
                    const bool first_max = kFp8 && i == 0 && attempt == 0;
                    if (!first_max) {
                        const float gmax =
                            !tail ? softmax_pass_share<0, kFp8>(s_addr, c_lo, c_hi, m_s, scale, vis_s, G, gmin, pk)
                                  : softmax_pass_share<kTree ? 2 : 1, kFp8>(s_addr, c_lo, c_hi, m_s, scale, vis_s, G, gmin, pk);
                        if (warp == kSoftmaxWarp0) LVSPEC_TILE_TS(tile_tr, 0, i, 2);     // exponentials done
                        if (!group_any(bar_id, gmax > kLimit)) break;
                    }

                    // ---- a score ran past the guard: move m up to the tile maximum ----
                    for (int c8 = c_lo; c8 < c_hi; ++c8) {
                        uint32_t r[8];
                        tmem_ld_x8(s_addr + c8 * 8, r);
                        tmem_wait_ld();
#pragma unroll
                        for (int k = 0; k < 8; ++k) {
                            float s2 = __uint_as_float(r[k]) * scale;
                            if (tail && (kTree ? !column_sees(vis_s[c8 * 8 + k], gmin) : (c8 * 8 + k) / G < gmin))
                                s2 = -INFINITY;
                            s2 = warp_max_f32(s2);
                            if (lane == 0) tmx_s[wq * NP + c8 * 8 + k] = s2;
                        }
                    }
                    group_sync(bar_id);
                    for (int n = c_lo * 8 + gtid; n < c_hi * 8; n += 128) {
                        const float mt = fmaxf(fmaxf(tmx_s[n], tmx_s[NP + n]),
                                               fmaxf(tmx_s[2 * NP + n], tmx_s[3 * NP + n])) - kLift;
                        const float mo = m_s[n];
                        const float mn = fmaxf(mo, mt);
                        dl_s[n] = mo - mn;              // <= 0
                        m_s[n] = mn;
                    }
                    group_sync(bar_id);
                    if (i > 0) {
                        // O^T and the sums were accumulated under the old m: rescale this
                        // group's columns once PV(i-1) has finished
                        mbar_wait(p_free(i - 1), hand_parity(i - 1), abort_flag);
                        tc_fence_after();
                        // (fp8 cache: accumulator columns 2n and 2n + 1 belong to row n)
                        for (int c = c_lo * kAccCols; c < c_hi * kAccCols; ++c) {
                            uint32_t r[8];
                            tmem_ld_x8(tm_o + lane_addr + c * 8, r);
                            tmem_wait_ld();
#pragma unroll
                            for (int k = 0; k < 8; ++k)
                                r[k] = __float_as_uint(__uint_as_float(r[k]) * ex2(dl_s[(c * 8 + k) / kAccCols]));
                            tmem_st_x8(tm_o + lane_addr + c * 8, r);
                            if (wq == 0) {
                                tmem_ld_x8(tm_l + c * 8, r);
                                tmem_wait_ld();
#pragma unroll
                                for (int k = 0; k < 8; ++k)
                                    r[k] = __float_as_uint(__uint_as_float(r[k]) * ex2(dl_s[(c * 8 + k) / kAccCols]));
                                tmem_st_x8(tm_l + c * 8, r);
                            }
                        }
                        tmem_wait_st();
                        tc_fence_before();
                    }
                    group_sync(bar_id);
                }
                if (tail && grp == 0) {
                    // slots at or beyond kv_len hold whatever the cache holds: zero their V
                    // rows so that 0 * junk cannot poison the accumulators
                    mbar_wait(v_full(vsl), vs_round & 1, abort_flag);
                    if (pos >= L) {
                        uint8_t *vrow = gbase + sm.v + vsl * kSlot + row * 128;
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            *reinterpret_cast<uint4 *>(vrow + c * 16) = make_uint4(0, 0, 0, 0);
                            if (two_boxes) *reinterpret_cast<uint4 *>(vrow + kBoxBytes + c * 16) = make_uint4(0, 0, 0, 0);
                        }
                    }
                }
                if (warp == kSoftmaxWarp0) LVSPEC_TILE_TS(tile_tr, 0, i, 3);     // the group agrees: no rescale
                // P^T goes to shared memory once the P.V product that read this buffer is done
                if (i >= cfg.pb) mbar_wait(p_free(i - cfg.pb), hand_parity(i - cfg.pb), abort_flag);
                if (warp == kSoftmaxWarp0) LVSPEC_TILE_TS(tile_tr, 0, i, 4);     // P buffer free
#pragma unroll
                for (int j = 0; j < kMaxChunks; ++j)
                    if (c_lo + j < c_hi) *reinterpret_cast<uint4 *>(prow + (c_lo + j) * 2048) = pk[j];
                // one arrival per warp: S^T has been read (the next K.Q^T but one may overwrite
                // it) and P^T, with any zeroed V rows, is in shared memory
                tc_fence_before();
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(s_free(i));
                    mbar_arrive(p_full(i));
                }
                if (warp == kSoftmaxWarp0) LVSPEC_TILE_TS(tile_tr, 0, i, 5);     // P^T stored and handed over
                if (++pb == cfg.pb) { pb = 0; ++pb_round; }
                if (++vsl == cfg.vs) { vsl = 0; ++vs_round; }
            }
        }

        // ---------------------------------------------------------------- epilogue
        // (every group takes its share of the columns)
        // the last P.V product has finished (and with it all before)
        mbar_wait(pv_done, 0, abort_flag);
        tc_fence_after();
        if (p.n_split == 1) {
            // a single split: nothing to merge, normalise and write the results here
            if (wq == 0) {
                for (int c8 = c_lo; c8 < c_hi; ++c8) {
                    float lsum[8];
                    load_acc8<kFp8>(tm_l, c8, lsum);      // lane 0: l, lane 1: l_vis
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const int n = c8 * 8 + k;
                        const float lv = __shfl_sync(0xffffffffu, lsum[k], 1);
                        if (lane == 0 && n < M) {
                            const float inv = 1.f / lsum[k];
                            dl_s[n] = inv * v_scale;
                            const int g = n / G, hg = n - g * G;
                            p.mass[((size_t)b * gamma + g) * p.Hq + kvh * G + hg] = lv * inv;
                        }
                    }
                }
            }
            group_sync(bar_id);
            __nv_bfloat16 *out = reinterpret_cast<__nv_bfloat16 *>(p.out);
            for (int c8 = c_lo; c8 < c_hi; ++c8) {
                float o8[8];
                load_acc8<kFp8>(tm_o + lane_addr, c8, o8);
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const int n = c8 * 8 + k;
                    if (n < M && row < D) {
                        const int g = n / G, hg = n - g * G;
                        out[(((size_t)b * gamma + g) * p.Hq + kvh * G + hg) * D + row] =
                            __float2bfloat16_rn(o8[k] * dl_s[n]);
                    }
                }
            }
        } else {
            // This code runs once, on cold instruction caches, where every instruction
            // costs about ten cycles: short rolled loops, one chunk of 8 columns a turn;
            // only a last chunk that is not full takes the guarded path.
            // (TMEM lanes are channels: at head_dim 64 the upper half of the lanes holds nothing)
            float *po = part_o + (size_t)c_lo * 8 * D + row;
            const int m_store = row < D ? M : 0;
#pragma unroll 1
            for (int c8 = c_lo; c8 < c_hi; ++c8, po += 8 * D) {
                float o8[8];
                load_acc8<kFp8>(tm_o + lane_addr, c8, o8);
                if (kFp8) {
#pragma unroll
                    for (int k = 0; k < 8; ++k) o8[k] *= v_scale;
                }
                if (c8 * 8 + 8 <= m_store) {
#pragma unroll
                    for (int k = 0; k < 8; ++k) po[k * D] = o8[k];
                } else {
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        if (c8 * 8 + k < m_store) po[k * D] = o8[k];
                }
            }
            if (wq == 0) {
#pragma unroll 1
                for (int c8 = c_lo; c8 < c_hi; ++c8) {
                    float lsum[8];
                    load_acc8<kFp8>(tm_l, c8, lsum);      // lane 0: l, lane 1: l_vis
                    // lane k takes column k of the chunk: l from lane 0, l_vis from lane 1
                    float lk = 0.f, lvk = 0.f;
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const float a = __shfl_sync(0xffffffffu, lsum[k], 0);
                        const float c = __shfl_sync(0xffffffffu, lsum[k], 1);
                        if (lane == k) { lk = a; lvk = c; }
                    }
                    if (lane < 8 && c8 * 8 + lane < M)
                        *reinterpret_cast<float4 *>(part_stat + (c8 * 8 + lane) * 4) =
                            make_float4(m_s[c8 * 8 + lane], lk, lvk, 0.f);
                }
            }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(done_bar);
    }

    // ------------------------------------------------------------------ teardown
    // TMEM goes back once the MMAs have drained and every softmax warp is done
    if (warp == 1) {
        if (lane == 0) {
            bool all_done = false;
#ifdef LVSPEC_TRACE
            if (rec) rec[5] = lvspec_trace_now();
#endif
            for (int tries = 0; tries < 4 && !all_done; ++tries) all_done = wait_unconditional(done_bar, 0);
#ifdef LVSPEC_TRACE
            if (rec) rec[6] = lvspec_trace_now();
#endif
            if (*abort_flag || !all_done) atomicOr(p.status, LVSPEC_DEV_WAIT_EXPIRED);
            // this CTA is done but for freeing TMEM: a dependent launch may be scheduled
            // once every CTA has come this far (earlier, its CTAs would pile up on the
            // few SMs this grid leaves idle)
            grid_launch_dependents();
        }
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, (uint32_t)cfg.tmem_cols);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                  const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                  const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            return nullptr;
        fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

// A cache as a 4-D tensor [sequences or pages][heads][positions][128 channels] with the
// caller's strides (in elements; the channels are contiguous).  bf16: boxes of 64 channels
// x 128 positions; E4M3: boxes of 128 channels x 128 positions.
bool make_kv_map(CUtensorMap *map, const void *ptr, bool fp8, int D, int positions, int heads, int outer,
                 int64_t s_pos, int64_t s_head, int64_t s_outer)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t esz = fp8 ? 1 : 2;
    const cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)positions, (cuuint64_t)heads, (cuuint64_t)outer};
    const cuuint64_t strides[3] = {(cuuint64_t)s_pos * esz, (cuuint64_t)s_head * esz, (cuuint64_t)s_outer * esz};
    const cuuint32_t box[4] = {fp8 ? 128u : 64u, 128, 1, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(map, fp8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4,
              const_cast<void *>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// q [B][gamma][Hq][128] bf16 as a 4-D tensor; one box = 64 channels of the G heads of one
// KV head for all gamma queries: its rows land in shared memory in the order g * G + hg
bool make_q_map(CUtensorMap *map, const void *ptr, int B, int gamma, int Hq, int G, int D)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t row = (cuuint64_t)D * 2;
    const cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)Hq, (cuuint64_t)gamma, (cuuint64_t)B};
    const cuuint64_t strides[3] = {row, (cuuint64_t)Hq * row, (cuuint64_t)gamma * Hq * row};
    const cuuint32_t box[4] = {64, (cuuint32_t)G, (cuuint32_t)gamma, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(ptr), dims, strides, box,
              estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

constexpr uint32_t kMaxSmem = 232448 - 1024;   // 227 KB less the alignment slack

TcConfig pick_config(int M, int page_slots, bool fp8, bool turns, int D)
{
    TcConfig c;
    c.n_pad = (M + 15) & ~15;
    c.page_slots = page_slots;
    const bool small_tiles = fp8 || D == 64;     // one 16 KB box per tile: twice the slots
    c.slot_bytes = small_tiles ? kBoxBytes : kSlotBytes;
    const int acc = fp8 ? 4 : 2;     // TMEM columns per padded row of O^T and the sums
    if (!turns) {
        // All groups on every tile: S^T twice.  Six ring slots when they fit, also at the
        // price of the second P buffer (with 40 rows the stream is bound by HBM: bytes in
        // flight count, and the probabilities wait in registers for the buffer anyway).
        c.sb = 2;
        const int tries[6][3] = {{3, 3, 2}, {3, 3, 1}, {2, 3, 2}, {2, 2, 2}, {2, 3, 1}, {2, 2, 1}};
        const int tries8[6][3] = {{5, 6, 2}, {5, 5, 2}, {4, 5, 2}, {4, 4, 2}, {4, 4, 1}, {3, 3, 1}};
        for (int t = 0; t < 6; ++t) {
            const int *tr = small_tiles ? tries8[t] : tries[t];
            c.ks = tr[0]; c.vs = tr[1]; c.pb = tr[2];
            if (smem_map(c).total <= kMaxSmem) break;
        }
    } else {
        // Tiles in turn: an S^T buffer per softmax group when TMEM has the columns, else
        // two.  Shared memory: a P^T buffer per group before more ring slots (a group that
        // shares its buffer waits for the product of an earlier tile before it can store
        // anything); of the rings, V slots are held longer than K slots.  An fp8 tile is
        // half the bytes: twice the slots for the same bytes in flight.
        c.sb = (kSoftmaxGroups + acc) * c.n_pad <= 512 ? kSoftmaxGroups : 2;
        const int tries[8][3] = {{3, 3, 3}, {2, 3, 3}, {3, 2, 3}, {2, 2, 3}, {2, 2, 2}, {2, 2, 1}, {1, 2, 1}, {1, 1, 1}};
        const int tries8[8][3] = {{5, 6, 3}, {5, 5, 3}, {4, 5, 3}, {4, 4, 3}, {4, 4, 2}, {3, 3, 2}, {3, 3, 1}, {2, 2, 1}};
        for (int t = 0; t < 8; ++t) {
            const int *tr = small_tiles ? tries8[t] : tries[t];
            c.ks = tr[0]; c.vs = tr[1]; c.pb = tr[2];
            if (smem_map(c).total <= kMaxSmem) break;
        }
    }
    // LVSPEC_TC_RING="K slots,V slots,P buffers,S buffers" overrides the choice (for
    // measurements; a combination that does not fit is refused by the launch)
    if (const char *e = std::getenv("LVSPEC_TC_RING")) {
        int ks, vs, pb, sb;
        if (std::sscanf(e, "%d,%d,%d,%d", &ks, &vs, &pb, &sb) == 4 && ks >= 1 && ks <= 8 && vs >= 1 && vs <= 8 &&
            pb >= 1 && pb <= kSoftmaxGroups && sb >= 2 && sb <= kSoftmaxGroups && (turns || (sb == 2 && pb <= 2))) {
            c.ks = ks; c.vs = vs; c.pb = pb; c.sb = sb;
        }
    }
    int cols = 32;
    while (cols < (c.sb + acc) * c.n_pad) cols <<= 1;
    c.tmem_cols = cols;
    return c;
}

}  // namespace

bool attn_tc_supported(const AttnParams &p)
{
    if (p.fp8 && (p.M > kMaxRowsFp8 || p.page_size > 0 || p.branch_len != p.gamma)) return false;
    return (p.D == 128 || (p.D == 64 && !p.fp8)) && p.Lmax >= kTilePos && p.M <= LVSPEC_MAX_ROWS;
}

cudaError_t launch_attn_tc(const AttnParams &p, const SeqInfo &seq, cudaStream_t stream, int *launches)
{
    TcParams P;
    P.a = p;
    const bool paged = p.page_size > 0;
    // paged: one block-table entry per tile of the longest split, rounded up to 4
    const int tiles = (p.Lmax + kTilePos - 1) / kTilePos;
    const bool fp8 = p.fp8 != 0;
    // Tiles in turn where a CTA streams long enough for the throughput of the softmax stage
    // to outweigh its latency at the two ends of the stream (measured on the 40/8-head sweep:
    // 5 to 10 % faster from about a hundred tiles per CTA, slower below 32), and with an fp8
    // cache of up to 64 padded rows (half the bytes per tile for the same work; with more
    // rows TMEM holds only two S^T buffers and the shared columns win).
    // LVSPEC_TC_TURNS=0/1 overrides the choice (for measurements).
    bool turns = (tiles + p.n_split - 1) / p.n_split >= 96 || (fp8 && p.M <= 64);
    if (const char *e = std::getenv("LVSPEC_TC_TURNS"))
        if (e[0] == '0' || e[0] == '1') turns = e[0] == '1';
    P.cfg = pick_config(p.M, paged ? ((tiles + p.n_split - 1) / p.n_split + 4) & ~3 : 0, fp8, turns, p.D);
    if (smem_map(P.cfg).total > kMaxSmem || P.cfg.tmem_cols > 512) return cudaErrorInvalidConfiguration;
    CUtensorMap mk, mv, mq;
    const int map_len = paged ? p.page_size : p.Lmax;
    const int map_outer = paged ? p.n_pages : p.B;
    if (!make_kv_map(&mk, p.k, fp8, p.D, map_len, p.Hkv, map_outer, p.k_sp, p.k_sh, p.k_sb) ||
        !make_kv_map(&mv, p.v, fp8, p.D, map_len, p.Hkv, map_outer, p.v_sp, p.v_sh, p.v_sb))
        return cudaErrorInvalidValue;
    if (fp8) mq = mk;     // not used by the kernel
    else if (!make_q_map(&mq, p.q, p.B, p.gamma, p.Hq, p.G, p.D)) return cudaErrorInvalidValue;
    const size_t smem = smem_map(P.cfg).total + 1024;
    const bool tree = p.branch_len != p.gamma;
    if ((tree && paged) || (fp8 && (tree || paged))) return cudaErrorNotSupported;
    auto kernel = fp8 ? (turns ? attn_tc_kernel<false, false, true, true> : attn_tc_kernel<false, false, true, false>)
                  : turns ? (paged ? attn_tc_kernel<false, true, false, true>
                                   : (tree ? attn_tc_kernel<true, false, false, true>
                                           : attn_tc_kernel<false, false, false, true>))
                          : (paged ? attn_tc_kernel<false, true, false, false>
                                   : (tree ? attn_tc_kernel<true, false, false, false>
                                           : attn_tc_kernel<false, false, false, false>));
    cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(p.n_split, p.Hkv, p.B);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = p.pdl ? 1 : 0;
    err = cudaLaunchKernelEx(&cfg, kernel, P, seq, mk, mv, mq);
    ++*launches;
    return err != cudaSuccess ? err : cudaGetLastError();
}

}  // namespace lvspec
