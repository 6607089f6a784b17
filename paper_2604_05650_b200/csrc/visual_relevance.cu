// The paper's own visual-relevance score (Sec. 3.1, Eq. 4): for every draft
// token the mean of the N largest cosine similarities between its final-layer
// hidden state and the visual tokens' final-layer hidden states.
//
// Two kernels per call:
//   cos_tc_kernel       streams H_V once (the HBM-bound part): every CTA takes an
//                       equal share of the visual rows, in chunks of up to 256
//                       rows = two row blocks with one accumulator each;
//                       S[row, k] = H_V[row, :] . H_D[k, :] on the tensor core
//                       (tcgen05, MMA M = 128 rows, N = K padded to 16 by the TMA
//                       unit's zero fill, the hidden dimension in TMA stages of 64
//                       channels); its otherwise idle epilogue warps take H_D's
//                       reciprocal norms meanwhile; then
//                       cosine = S * inv_norm_v[row] * inv_norm_d[k].
//                       N <= 32: every warp keeps, per draft token, only the N largest
//                       cosines of its 32 rows (they hold every value the exact Top-N
//                       can contain) and appends them to the token's candidate list;
//                       N > 32: all cosines go to scratch.
//   topn_mean_kernel    exact Top-N mean per draft token over the candidates (or
//                       all cosines), summed in descending order of value
// The reciprocal norms of H_V's rows come from row_inv_norms_kernel, run once
// after prefill.
#include <cuda.h>
#include <cuda_bf16.h>

#include "lvspec_internal.h"
#include "sm100_ptx.cuh"

namespace lvspec {
namespace {

using namespace ptx;

// ------------------------------------------------------------------ row norms
constexpr int kNormWarps = 8;

__device__ __forceinline__ float sumsq_bf16x8(uint4 w, float acc)
{
    const uint32_t x[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float lo = __uint_as_float(x[i] << 16), hi = __uint_as_float(x[i] & 0xffff0000u);
        acc = fmaf(lo, lo, acc);
        acc = fmaf(hi, hi, acc);
    }
    return acc;
}

// one warp per row; dim a multiple of 8
__global__ void __launch_bounds__(32 * kNormWarps)
row_inv_norms_kernel(const uint16_t *x, long long rows, int dim, float *out)
{
    const long long r = (long long)blockIdx.x * kNormWarps + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (r >= rows) return;
    const uint4 *src = reinterpret_cast<const uint4 *>(x + r * dim);
    float acc = 0.f;
    for (int i = lane; i < dim / 8; i += 32) acc = sumsq_bf16x8(__ldg(src + i), acc);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) out[r] = acc > 0.f ? 1.f / sqrtf(acc) : 0.f;
}

// ------------------------------------------------------------- cosine kernel
constexpr int kCosThreads = 192;            // warp 0 producer, warp 1 MMA, warps 2-5 epilogue
constexpr uint32_t kGroupBytes = 2048;      // 16 rows x 64 channels bf16
constexpr uint32_t kBlockBytes = 8 * kGroupBytes;    // one row block: 128 rows
constexpr int kChunkGroups = 16;            // most groups of 16 rows per chunk
constexpr int kMaxStages = 24;
constexpr uint32_t kBarBytes = 1024;        // barriers and the TMEM slot, ahead of the stages

constexpr int kTopFused = 32;               // Top-N up to this is selected per warp in the cosine kernel
constexpr uint32_t kDinvOffset = 704;       // reciprocal norms of H_D's rows, inside the barrier block

struct CosParams {
    RelevanceParams r;
    int NP;                 // K padded to a multiple of 16 (MMA N)
    int smem_bytes;         // dynamic shared memory of the launch (after 1024-byte alignment)
    int tmem_cols;
    int tail_a, tail_b;     // row-group counts that have a one-box tensor map of their own (0 = none)
    int n_grp;              // groups of 16 rows per batch element
    int total_groups;       // B * n_grp
    int chunk_groups;       // groups of 16 rows per chunk (<= kChunkGroups)
};

// The chunks (up to 16 groups of 16 rows of one batch element) of one CTA's share
// of the row groups; producer, MMA issuer and epilogue walk them in step.
struct ChunkWalk {
    int gg, end, n_grp, chunk_groups;
    int b, row0, n_groups;   // the current chunk
    __device__ bool next()
    {
        if (gg >= end) return false;
        b = gg / n_grp;
        const int g0 = gg - b * n_grp;
        n_groups = min(chunk_groups, min(n_grp - g0, end - gg));
        row0 = g0 * 16;
        gg += n_groups;
        return true;
    }
};

// order-preserving map float -> unsigned (larger float, larger key)
__device__ __forceinline__ uint32_t float_key(float v)
{
    const uint32_t u = __float_as_uint(v);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_float(uint32_t k)
{
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

__device__ __forceinline__ bool wait_teardown(uint32_t bar, uint32_t parity)
{
    const uint64_t t0 = global_timer_ns();
    while (!mbar_try_wait(bar, parity))
        if (global_timer_ns() - t0 > 1000000000ull) return false;
    return true;
}

__global__ void __launch_bounds__(kCosThreads, 1)
cos_tc_kernel(const CosParams P, const __grid_constant__ CUtensorMap tmap_v,
              const __grid_constant__ CUtensorMap tmap_v128, const __grid_constant__ CUtensorMap tmap_va,
              const __grid_constant__ CUtensorMap tmap_vb, const __grid_constant__ CUtensorMap tmap_d)
{
    extern __shared__ uint8_t smem_raw[];
    const RelevanceParams &p = P.r;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int NP = P.NP, KC = p.d / 64;

    // this CTA's share of the row groups: equal shares, sizes differ by at most one
    ChunkWalk walk;
    {
        const int n_cta = gridDim.x, c = blockIdx.x;
        const int per = P.total_groups / n_cta, rem = P.total_groups - per * n_cta;
        walk.gg = c * per + min(c, rem);
        walk.end = walk.gg + per + (c < rem ? 1 : 0);
        walk.n_grp = P.n_grp;
        walk.chunk_groups = P.chunk_groups;
    }
    // A stage holds 64 channels of the tallest chunk this CTA can meet (row block 0,
    // then row block 1, then the draft tile); the fewer rows, the more stages fit,
    // and bytes in flight, not stages, are what covers the memory latency.
    const int cap = max(1, min(P.chunk_groups, walk.end - walk.gg));
    const uint32_t d_off = cap <= 8 ? (uint32_t)cap * kGroupBytes : kBlockBytes + (uint32_t)(cap - 8) * kGroupBytes;
    const uint32_t stage_bytes = (d_off + (uint32_t)NP * 128u + 1023u) & ~1023u;
    // An MMA always reads whole row blocks of 128 rows (rows a chunk does not have are
    // junk lanes nobody looks at), so from the last stage's start one or two full
    // blocks must still lie inside the allocation.
    const uint32_t read_extent = cap > 8 ? 2 * kBlockBytes : kBlockBytes;
    const int S = min(kMaxStages,
                      1 + (int)(((uint32_t)P.smem_bytes - kBarBytes - max(read_extent, stage_bytes)) / stage_bytes));

    const uint32_t base0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gbase = smem_raw + (base0 - smem_u32(smem_raw));
    const uint32_t bar0 = base0;
    const uint32_t base = base0 + kBarBytes;          // first stage
    auto full = [&](int s) { return bar0 + 8 * s; };
    auto empty = [&](int s) { return bar0 + 8 * (S + s); };
    auto acc_full = [&](int s) { return bar0 + 8 * (2 * S + s); };
    auto acc_free = [&](int s) { return bar0 + 8 * (2 * S + 2 + s); };
    const uint32_t done_bar = bar0 + 8 * (2 * S + 4);
    const uint32_t drain_bar = bar0 + 8 * (2 * S + 5);
    const uint32_t misc = bar0 + 8 * (2 * S + 6);
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(gbase + (misc - base0));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(gbase + (misc - base0) + 4);

    if (warp == 0) {
        if (lane == 0) prefetch_tensormap(&tmap_v);
        if (lane == 1) prefetch_tensormap(&tmap_d);
        if (lane == 2) prefetch_tensormap(&tmap_v128);
        if (lane == 3) prefetch_tensormap(&tmap_va);
        if (lane == 4) prefetch_tensormap(&tmap_vb);
        const int n_bars = 2 * S + 6;
        for (int j = lane; j < n_bars; j += 32) {
            uint32_t count = 1;
            if (j >= 2 * S + 2 && j < 2 * S + 4) count = 4;   // acc_free: the epilogue warps
            else if (j == 2 * S + 4) count = 4;               // done
            mbar_init(bar0 + 8 * j, count);
        }
        if (lane == 0) *abort_flag = 0;
        mbar_fence_init();
        fence_proxy_async_smem();
    } else if (warp == 1) {
        tmem_alloc(misc, (uint32_t)P.tmem_cols);
        tmem_relinquish();
    }
    // the padded draft tile comes from the kernel before this one
    grid_dependency_wait();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            const uint64_t stream_policy = l2_evict_first_policy();
            int n = 0;                       // stages filled so far
            bool ok = true;
            // Every CTA walks the channels from a different slab on (and around): at a row
            // pitch like 10 KB the same slab of all rows shares its low address bits, and
            // with all CTAs on the same slab the requests crowd on few memory channels.
            const int kc0 = (int)((blockIdx.x * 37u) % (unsigned)KC);
            while (ok && walk.next()) {
                for (int kci = 0; kci < KC; ++kci, ++n) {
                    const int kc = kci + kc0 < KC ? kci + kc0 : kci + kc0 - KC;
                    const int s = n % S;
                    if (n >= S && !mbar_wait(empty(s), ((n / S) - 1) & 1, abort_flag)) { ok = false; break; }
                    const uint32_t dst = base + s * stage_bytes;
                    mbar_arrive_expect_tx(full(s), (uint32_t)walk.n_groups * kGroupBytes + (uint32_t)NP * 128u);
                    // a full row block in one box of 128 rows, the rest in boxes of 16
                    int g = 0;
                    if (walk.n_groups >= 8) {
                        tma_load_3d_hint(dst, &tmap_v128, full(s), kc * 64, walk.row0, walk.b, stream_policy);
                        g = 8;
                    }
                    if (walk.n_groups == 16) {
                        tma_load_3d_hint(dst + kBlockBytes, &tmap_v128, full(s), kc * 64, walk.row0 + 128,
                                         walk.b, stream_policy);
                        g = 16;
                    }
                    // what is left of the chunk: in one box when its height is one of the
                    // two the launch made maps for (issuing a TMA costs the producer
                    // more than a hundred cycles), else in boxes of 16 rows
                    const int left = walk.n_groups - g;
                    if (left > 0 && left == P.tail_a) {
                        tma_load_3d_hint(dst + g * kGroupBytes, &tmap_va, full(s), kc * 64,
                                         walk.row0 + g * 16, walk.b, stream_policy);
                    } else if (left > 0 && left == P.tail_b) {
                        tma_load_3d_hint(dst + g * kGroupBytes, &tmap_vb, full(s), kc * 64,
                                         walk.row0 + g * 16, walk.b, stream_policy);
                    } else {
                        for (; g < walk.n_groups; ++g)
                            tma_load_3d_hint(dst + g * kGroupBytes, &tmap_v, full(s), kc * 64,
                                             walk.row0 + g * 16, walk.b, stream_policy);
                    }
                    tma_load_3d(dst + d_off, &tmap_d, full(s), kc * 64, 0, walk.b);
                }
            }
            if (*abort_flag) {
                // wait (bounded) for the copies still in flight before the CTA leaves
                for (int j = max(0, n - S); j < n; ++j) wait_teardown(full(j % S), (j / S) & 1);
            }
        }
    } else if (warp == 1) {
        // -------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            const uint32_t idesc = make_idesc_bf16(128, NP, 0, 0);
            int s = 0, chunk = 0;
            uint32_t round = 0;
            bool ok = true;
            while (ok && walk.next()) {
                const int buf = chunk & 1;
                if (chunk >= 2 && !mbar_wait(acc_free(buf), ((chunk >> 1) - 1) & 1, abort_flag)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * 2 * NP;
                const bool two_blocks = walk.n_groups > 8;
                for (int kc = 0; kc < KC; ++kc) {
                    if (!mbar_wait(full(s), round & 1, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a0 = base + s * stage_bytes;
                    const uint64_t da = make_smem_desc(a0, 16, 1024, kSwizzle128B);
                    const uint64_t db = make_smem_desc(a0 + d_off, 16, 1024, kSwizzle128B);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        mma_f16_ss(d_tmem, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), idesc,
                                   (kc | kk) != 0 ? 1u : 0u);
                    if (two_blocks) {
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)
                            mma_f16_ss(d_tmem + NP, da + (uint64_t)((kBlockBytes >> 4) + kk * 2),
                                       db + (uint64_t)(kk * 2), idesc, (kc | kk) != 0 ? 1u : 0u);
                    }
                    mma_commit(empty(s));
                    if (++s == S) { s = 0; ++round; }
                }
                if (!ok) break;
                mma_commit(acc_full(buf));
                ++chunk;
            }
            mma_commit(drain_bar);         // this thread's MMAs have drained
            wait_teardown(drain_bar, 0);
        }
    } else {
        // ---------------------------------------------------------- epilogue warps
        const int wq = warp & 3;
        const int row = wq * 32 + lane;                    // TMEM lane = row inside the chunk
        const uint32_t lane_addr = (uint32_t)(wq * 32) << 16;
        float *dinv_s = reinterpret_cast<float *>(gbase + kDinvOffset);
        const bool fused = p.top_n <= kTopFused;
        const int n_it = min(p.top_n, 32);
        int chunk = 0, cur_b = -1;
        while (walk.next()) {
            if (walk.b != cur_b) {
                // reciprocal norms of this batch element's draft rows: a warp per row,
                // while the rows of H_V stream in (fixed summation order)
                if (cur_b >= 0) asm volatile("bar.sync 1, 128;" ::: "memory");   // the old ones are no longer read
                cur_b = walk.b;
                for (int k = wq; k < NP; k += 4) {
                    float acc = 0.f;
                    if (k < p.K) {
                        const uint4 *src = reinterpret_cast<const uint4 *>(p.h_draft + ((size_t)cur_b * p.K + k) * p.d);
                        for (int i = lane; i < p.d / 8; i += 32) acc = sumsq_bf16x8(__ldg(src + i), acc);
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
                    }
                    if (lane == 0) dinv_s[k] = acc > 0.f ? 1.f / sqrtf(acc) : 0.f;
                }
                asm volatile("bar.sync 1, 128;" ::: "memory");
            }
            const int buf = chunk & 1;
            mbar_wait(acc_full(buf), (chunk >> 1) & 1, abort_flag);
            tc_fence_after();
            const int n_blocks = walk.n_groups > 8 ? 2 : 1;
            for (int blk = 0; blk < n_blocks; ++blk) {
                const int rc = blk * 128 + row;                // row inside the chunk
                const int j = walk.row0 + rc;                  // visual row of this thread
                const bool valid = rc < walk.n_groups * 16 && j < p.lv;
                const float vin = valid ? __ldg(p.v_inv_norm + (size_t)walk.b * p.lv + j) : 0.f;
                float *dst = p.cos_t + (size_t)walk.b * p.K * p.lv_pad;
                if (fused && __ballot_sync(0xffffffffu, valid) == 0u) continue;     // no row of this warp in the chunk
                for (int c8 = 0; c8 < NP / 8 && c8 * 8 < p.K; ++c8) {
                    uint32_t r[8];
                    tmem_ld_x8(tmem_base + (buf * 2 + blk) * NP + lane_addr + c8 * 8, r);
                    tmem_wait_ld();
                    if (!fused) {
#pragma unroll
                        for (int k = 0; k < 8; ++k) {
                            const int kk = c8 * 8 + k;
                            if (valid && kk < p.K)
                                dst[(size_t)kk * p.lv_pad + j] = __uint_as_float(r[k]) * vin * dinv_s[kk];
                        }
                        continue;
                    }
                    // the N largest of this warp's 32 rows, per draft token: the warp sorts
                    // the 32 keys of a column with shuffles (descending; the eight columns
                    // side by side), lane t then holds the t-th largest.  Key 0 = no value.
                    uint32_t top[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const int kk = c8 * 8 + k;
                        top[k] = (valid && kk < p.K) ? float_key(__uint_as_float(r[k]) * vin * dinv_s[kk]) : 0u;
                    }
#pragma unroll
                    for (int size = 2; size <= 32; size <<= 1) {
#pragma unroll
                        for (int stride = size >> 1; stride > 0; stride >>= 1) {
                            const bool upper = (lane & stride) != 0;          // holds the second of the pair
                            const bool descending = (lane & size) == 0;
                            const bool take_max = (upper != descending);      // first of a descending pair keeps the max
#pragma unroll
                            for (int k = 0; k < 8; ++k) {
                                const uint32_t y = __shfl_xor_sync(0xffffffffu, top[k], stride);
                                top[k] = take_max ? max(top[k], y) : min(top[k], y);
                            }
                        }
                    }
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        if (lane >= n_it) top[k] = 0u;
                    // lane k reserves the places of column k: the eight requests travel together
                    uint32_t my_cnt = 0u;
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const uint32_t cnt = __popc(__ballot_sync(0xffffffffu, top[k] != 0u));
                        if (lane == k) my_cnt = cnt;
                    }
                    uint32_t my_off = 0u;
                    if (lane < 8 && c8 * 8 + lane < p.K && my_cnt > 0u)
                        my_off = atomicAdd(p.counters + (size_t)walk.b * p.K + c8 * 8 + lane, my_cnt);
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const int kk = c8 * 8 + k;
                        const uint32_t off = __shfl_sync(0xffffffffu, my_off, k);
                        if (kk < p.K && top[k] != 0u) dst[(size_t)kk * p.lv_pad + off + lane] = key_float(top[k]);
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_free(buf));
            ++chunk;
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(done_bar);
    }

    __syncwarp();
    if (warp == 1) {
        if (lane == 0) {
            bool all_done = false;
            for (int tries = 0; tries < 4 && !all_done; ++tries) all_done = wait_teardown(done_bar, 0);
            if (*abort_flag || !all_done) atomicOr(p.status, LVSPEC_DEV_WAIT_EXPIRED);
            grid_launch_dependents();
        }
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, (uint32_t)P.tmem_cols);
    }
}

// ------------------------------------------------------------- Top-N mean
constexpr int kTopThreads = 1024;

constexpr int kTopPerThread = 32;      // fast path: lv <= 32 * 1024
constexpr int kTopCandidates = 2048;
constexpr int kRankCandidates = 256;    // up to here the candidates are ranked by counting, not sorted

// descending bitonic sort of a power-of-two array of keys in shared memory
__device__ void bitonic_sort_desc(uint32_t *a, int n, int tid)
{
    for (int size = 2; size <= n; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            __syncthreads();
            for (int i = tid; i < n / 2; i += kTopThreads) {
                const int lo = 2 * i - (i & (stride - 1));      // index with the `stride` bit clear
                const int hi = lo + stride;
                const bool descending = (lo & size) == 0;
                const uint32_t x = a[lo], y = a[hi];
                if ((x < y) == descending) { a[lo] = y; a[hi] = x; }
            }
        }
    }
    __syncthreads();
}

// One CTA per (draft token, batch element): the exact mean of the n = min(N, lv)
// largest of lv cosines, summed in descending order of value (reproducible).
//
// Fast path (lv <= 32768, n <= 1024): every thread keeps its strided elements in
// registers and reports its largest; the n-th largest of these 1024 maxima is
// a lower bound of the n-th largest element, so only the few elements at or
// above it are collected and sorted.  If the candidates do not fit (the large
// values all sit in few threads' strides) or the row is longer, the general
// path finds the n-th largest key by radix selection, 8 bits per pass.
__global__ void __launch_bounds__(kTopThreads) topn_mean_kernel(const RelevanceParams p)
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
    __shared__ uint32_t keys[kTopCandidates];
    __shared__ uint32_t hist[256];
    __shared__ uint32_t ranked[kRankCandidates];
    __shared__ uint32_t sel_prefix, sel_need, n_cand;
    __shared__ float warp_sum[kTopThreads / 32];
    __shared__ int n_values;
    const int k = blockIdx.x, b = blockIdx.y, tid = threadIdx.x;
    const float *row = p.cos_t + ((size_t)b * p.K + k) * p.lv_pad;
    // with N <= kTopFused the row holds the candidates the cosine kernel appended (at
    // least min(N, lv) of them, every value of the exact Top-N among them) and the
    // counter says how many; the counter goes back to zero for the next call
    if (tid == 0) {
        n_values = p.lv;
        if (p.top_n <= kTopFused) {
            uint32_t *cnt = p.counters + (size_t)b * p.K + k;
            n_values = (int)min(__ldcg(cnt), (uint32_t)p.lv);
            *cnt = 0u;
        }
    }
    __syncthreads();
    const int lv = n_values;
    const uint32_t n = (uint32_t)min(p.top_n, p.lv);
    float *out = p.relevance + (size_t)b * p.K + k;
    if ((uint32_t)lv < n) {       // cannot happen unless the cosine kernel gave up on a wait
        if (tid == 0) *out = __int_as_float(0x7fc00000);
        return;
    }

    if (lv <= kTopPerThread * kTopThreads && n <= (uint32_t)kTopThreads) {
        uint32_t mine[kTopPerThread];
        uint32_t best = 0;                                  // below every real key
#pragma unroll
        for (int i = 0; i < kTopPerThread; ++i) {
            const int j = tid + i * kTopThreads;
            mine[i] = j < lv ? float_key(__ldcg(row + j)) : 0u;
            best = max(best, mine[i]);
        }
        if (tid == 0) n_cand = 0;
        uint32_t bound;
        if (n <= 32u) {
            // the n-th largest of the 32 warp maxima: a looser bound, but one warp sorts
            // 32 keys with shuffles alone
            uint32_t wbest = best;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) wbest = max(wbest, __shfl_xor_sync(0xffffffffu, wbest, o));
            if ((tid & 31) == 0) keys[tid >> 5] = wbest;
            __syncthreads();
            if (tid < 32) {
                uint32_t x = keys[tid];
#pragma unroll
                for (int size = 2; size <= 32; size <<= 1) {
#pragma unroll
                    for (int stride = size >> 1; stride > 0; stride >>= 1) {
                        const uint32_t y = __shfl_xor_sync(0xffffffffu, x, stride);
                        const bool upper = (tid & stride) != 0;          // holds the second of the pair
                        const bool descending = (tid & size) == 0;
                        const bool take_max = (upper != descending);     // first of a descending pair keeps the max
                        x = take_max ? max(x, y) : min(x, y);
                    }
                }
                keys[tid] = x;                                           // descending
            }
            __syncthreads();
            bound = keys[n - 1];
        } else {
            keys[tid] = best;
            bitonic_sort_desc(keys, kTopThreads, tid);
            bound = keys[n - 1];                            // >= n elements are at or above it
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < kTopPerThread; ++i) {
            if (mine[i] >= bound && mine[i] != 0u) {
                const uint32_t slot = atomicAdd(&n_cand, 1u);
                if (slot < (uint32_t)kTopCandidates) keys[slot] = mine[i];
            }
        }
        __syncthreads();
        const uint32_t c = n_cand;
        if (c <= (uint32_t)kRankCandidates) {
            // few candidates (the usual case): every candidate counts those ahead of it
            // (larger key, or equal key and lower index) and the first n go to their places;
            // one pass and one barrier where a block-wide sort takes dozens
            for (uint32_t i = tid; i < c; i += kTopThreads) {
                const uint32_t key = keys[i];
                uint32_t rank = 0;
                for (uint32_t j = 0; j < c; ++j) {
                    const uint32_t kj = keys[j];
                    rank += (kj > key || (kj == key && j < i)) ? 1u : 0u;
                }
                if (rank < n) ranked[rank] = key;
            }
            __syncthreads();
            if (tid == 0) {
                float sum = 0.f;
                for (uint32_t i = 0; i < n; ++i) sum += key_float(ranked[i]);
                *out = sum / (float)n;
            }
            return;
        }
        if (c <= (uint32_t)kTopCandidates) {
            int pow2 = 32;
            while ((uint32_t)pow2 < c) pow2 <<= 1;
            for (int i = c + tid; i < pow2; i += kTopThreads) keys[i] = 0u;
            bitonic_sort_desc(keys, pow2, tid);
            if (tid == 0) {
                float sum = 0.f;
                for (uint32_t i = 0; i < n; ++i) sum += key_float(keys[i]);
                *out = sum / (float)n;
            }
            return;
        }
        __syncthreads();
    }

    uint32_t prefix = 0, mask = 0, need = n;
    for (int shift = 24; shift >= 0; shift -= 8) {
        for (int i = tid; i < 256; i += kTopThreads) hist[i] = 0;
        __syncthreads();
        for (int j = tid; j < lv; j += kTopThreads) {
            const uint32_t key = float_key(__ldcg(row + j));
            if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
        }
        __syncthreads();
        if (tid == 0) {
            uint32_t above = 0;
            int bin = 255;
            for (; bin > 0; --bin) {
                if (above + hist[bin] >= need) break;
                above += hist[bin];
            }
            sel_prefix = prefix | ((uint32_t)bin << shift);
            sel_need = need - above;       // how many of this bin still belong to the top n
        }
        __syncthreads();
        prefix = sel_prefix;
        need = sel_need;
        mask |= 255u << shift;
        __syncthreads();
    }
    // prefix = key of the n-th largest value; `need` copies of it are inside the top n
    float acc = 0.f;
    for (int j = tid; j < lv; j += kTopThreads) {
        const float v = __ldcg(row + j);
        if (float_key(v) > prefix) acc += v;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if ((tid & 31) == 0) warp_sum[tid >> 5] = acc;
    __syncthreads();
    if (tid < 32) {
        float s2 = tid < kTopThreads / 32 ? warp_sum[tid] : 0.f;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s2 += __shfl_xor_sync(0xffffffffu, s2, o);
        if (tid == 0) *out = (s2 + (float)need * key_float(prefix)) / (float)n;
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

// [B][rows][d] bf16 as a 3-D tensor; boxes of 64 channels x box_rows rows, 128-byte swizzle
bool make_rows_map(CUtensorMap *map, const void *ptr, int d, int rows, int B, int box_rows)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)rows, (cuuint64_t)B};
    const cuuint64_t strides[2] = {(cuuint64_t)d * 2, (cuuint64_t)rows * d * 2};
    const cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(ptr), dims, strides, box,
              estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

cudaError_t launch_row_inv_norms(const uint16_t *x, long long rows, int dim, float *out,
                                 cudaStream_t stream, int *launches)
{
    const long long blocks = (rows + kNormWarps - 1) / kNormWarps;
    row_inv_norms_kernel<<<(unsigned)blocks, 32 * kNormWarps, 0, stream>>>(x, rows, dim, out);
    ++*launches;
    return cudaGetLastError();
}

// Scratch behind p.cos_t: per (sequence, draft token) a row of lv_pad fp32 values (the
// Top-N candidates, or all cosines when N is large).
size_t relevance_scratch_bytes(int B, int K, int lv, int d)
{
    (void)d;
    const int lv_pad = (lv + 3) & ~3;
    return (size_t)B * K * lv_pad * sizeof(float);
}

cudaError_t launch_visual_relevance(const RelevanceParams &p, cudaStream_t stream, int *launches)
{
    const int NP = (p.K + 15) & ~15;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;

    CosParams P;
    P.r = p;
    P.NP = NP;
    P.smem_bytes = 232448 - 1024;      // everything an SM offers, less the alignment slack
    int cols = 32;
    while (cols < 4 * NP) cols <<= 1;
    P.tmem_cols = cols;
    P.n_grp = (p.lv + 15) / 16;
    P.total_groups = p.B * P.n_grp;
    // The shares are `per` or `per + 1` groups; what a share leaves after its full chunks
    // and its full row block is the tail that gets a map of its own.  (Chunks as tall as
    // possible: every stage of a chunk costs the producer the same two or three TMA
    // requests whatever its height; shares cut into three chunks of 64 rows, so that
    // epilogues could run beside the stream, took twice the time.)
    const int n_cta = P.total_groups < p.n_sm ? P.total_groups : p.n_sm;
    P.chunk_groups = kChunkGroups;
    auto tail_of = [](int groups) {
        const int t = groups % kChunkGroups;
        return t > 8 ? t - 8 : t;       // 0..8 groups
    };
    P.tail_a = tail_of(P.total_groups / n_cta);
    P.tail_b = tail_of(P.total_groups / n_cta + 1);
    if (P.tail_a * 16 > p.lv) P.tail_a = 0;
    if (P.tail_b * 16 > p.lv) P.tail_b = 0;
    CUtensorMap mv, mv128, mva, mvb, md;
    if (!make_rows_map(&mv, p.h_visual, p.d, p.lv, p.B, 16) ||
        // (fewer than 128 rows never make a full row block: the wide map is then not used)
        !make_rows_map(&mv128, p.h_visual, p.d, p.lv, p.B, p.lv >= 128 ? 128 : 16) ||
        !make_rows_map(&mva, p.h_visual, p.d, p.lv, p.B, P.tail_a > 0 ? P.tail_a * 16 : 16) ||
        !make_rows_map(&mvb, p.h_visual, p.d, p.lv, p.B, P.tail_b > 0 ? P.tail_b * 16 : 16) ||
        // the draft rows as they are: the box is NP rows high, the rows beyond K read as zeros
        !make_rows_map(&md, p.h_draft, p.d, p.K, p.B, NP))
        return cudaErrorInvalidValue;
    const size_t smem = (size_t)P.smem_bytes + 1024;
    cudaError_t err = cudaFuncSetAttribute(cos_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)n_cta, 1, 1);
    cfg.blockDim = dim3(kCosThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    err = cudaLaunchKernelEx(&cfg, cos_tc_kernel, P, mv, mv128, mva, mvb, md);
    ++*launches;
    if (err != cudaSuccess) return err;

    cudaLaunchConfig_t cfg2 = {};
    cfg2.gridDim = dim3((unsigned)p.K, (unsigned)p.B, 1);
    cfg2.blockDim = dim3(kTopThreads, 1, 1);
    cfg2.stream = stream;
    cfg2.attrs = attr;
    cfg2.numAttrs = 1;
    err = cudaLaunchKernelEx(&cfg2, topn_mean_kernel, p);
    ++*launches;
    return err != cudaSuccess ? err : cudaGetLastError();
}

}  // namespace lvspec
