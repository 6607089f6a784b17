// Verification attention with fused visual mass: TMA + tcgen05 kernel (D = 128).
//
// One CTA owns one KV split of one (sequence, KV head) and the M = gamma * G
// query rows that read this head.  The GQA-grouped queries are the small side
// of the problem, so the products are taken transposed: per tile of 128 cache
// positions
//     S^T[pos, n] = K_tile[pos, :] . Q[n, :]          (MMA M = 128 positions, N = rows)
//     O^T[d, n]  += V_tile[:, d]^T . P^T[:, n]        (MMA M = 128 channels,  N = rows)
//     L[0..1, n] += [1; in_span]   . P^T[:, n]        (MMA M = 64: row 0 = l, row 1 = l_vis)
// so every TMEM lane of S^T is one cache position (all 128 softmax threads do
// useful exponentials) and the padded dimension is N (granularity 16), not M.
// The softmax denominators l and the visual-span numerators l_vis come out of
// the tensor core as two extra accumulator rows fed by a constant 0/1 tile.
//
// The running maximum m[n] is kept fixed while scores stay within 2^60 of it:
// the tile's own maximum (a cross-lane reduction in this layout) is only taken
// when a score exceeds the guard, in which case the accumulators are rescaled.
// fp32 and bf16 share the exponent range, so nothing is lost in between.
//
// Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer (and TMEM owner),
// warps 2-3 = prologue helpers, warps 4-7 = softmax (TMEM lane quarter = warp
// % 4).  K and V tiles sit in separate shared-memory rings, each slot two
// 128-position x 64-channel boxes with the 128-byte swizzle.  Every mbarrier
// wait is bounded; a wait that gives up raises LVSPEC_DEV_WAIT_EXPIRED.
#include <cuda.h>
#include <cuda_bf16.h>

#include "lvspec_internal.h"
#include "sm100_ptx.cuh"

namespace lvspec {
namespace {

using namespace ptx;

constexpr int kTilePos = 128;
constexpr int kThreads = 256;
constexpr uint32_t kBoxBytes = 16384;       // 128 positions x 64 channels bf16
constexpr uint32_t kSlotBytes = 2 * kBoxBytes;
constexpr uint32_t kA2Bytes = 2048;         // one 64 x 16 constant tile
constexpr float kGuard = 60.f;              // log2 units above m before a rescale
constexpr float kMFloor = -1.0e30f;

struct TcConfig {
    int n_pad;   // MMA N: rows padded to a multiple of 16
    int ks, vs, pb;   // K slots, V slots, P buffers
    int tmem_cols;
};

// Byte offsets of the shared-memory regions (relative to a 1024-aligned base).
struct SmemMap {
    uint32_t k, v, q, p, a2, m, dl, tmx, bars, misc, total;
};
__host__ __device__ inline SmemMap smem_map(const TcConfig &c)
{
    SmemMap s;
    uint32_t o = 0;
    s.k = o;    o += c.ks * kSlotBytes;
    s.v = o;    o += c.vs * kSlotBytes;
    s.q = o;    o += c.n_pad * 256;
    s.p = o;    o += c.pb * c.n_pad * 256;
    s.a2 = o;   o += 4 * kA2Bytes;
    s.m = o;    o += c.n_pad * 4;
    s.dl = o;   o += c.n_pad * 4;
    s.tmx = o;  o += 4 * c.n_pad * 4;
    s.bars = o; o += 8 * (2 * c.ks + 2 * c.vs + 4 + 2 * c.pb + 1);
    s.misc = o; o += 16;
    s.total = o;
    return s;
}

struct TcParams {
    AttnParams a;
    TcConfig cfg;
};

__device__ __forceinline__ bool wait_unconditional(uint32_t bar, uint32_t parity)
{
    // used only while tearing down after an abort: time-bounded, ignores the flag
    const uint64_t t0 = global_timer_ns();
    while (!mbar_try_wait(bar, parity))
        if (global_timer_ns() - t0 > 1000000000ull) return false;
    return true;
}

__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(const TcParams P, const SeqInfo seq, const __grid_constant__ CUtensorMap tmap_k,
               const __grid_constant__ CUtensorMap tmap_v)
{
    extern __shared__ uint8_t smem_raw[];
    const AttnParams &p = P.a;
    const TcConfig cfg = P.cfg;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int split = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
    const int L = seq.kv_len[b], vs = seq.span_start[b], ve = seq.span_end[b];
    const int M = p.M, G = p.G, gamma = p.gamma, NP = cfg.n_pad;
    const int n8 = (M + 7) >> 3;

    const int n_tiles = (L + kTilePos - 1) / kTilePos;
    const int tiles_per_split = (n_tiles + p.n_split - 1) / p.n_split;
    const int t_begin = split * tiles_per_split;
    const int T = min(n_tiles, t_begin + tiles_per_split) - t_begin;

    const size_t unit = ((size_t)b * p.Hkv + kvh) * p.n_split + split;
    float *part_o = p.part_o + unit * (size_t)M * 128;
    float *part_stat = p.part_stat + unit * (size_t)M * 4;
    if (T <= 0) {   // a split with no tile: contributes nothing
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
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(gbase + sm.misc);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(gbase + sm.misc + 4);

    // barrier addresses
    const uint32_t bar0 = base + sm.bars;
    auto k_full = [&](int s) { return bar0 + 8 * s; };
    auto k_empty = [&](int s) { return bar0 + 8 * (cfg.ks + s); };
    auto v_full = [&](int s) { return bar0 + 8 * (2 * cfg.ks + s); };
    auto v_empty = [&](int s) { return bar0 + 8 * (2 * cfg.ks + cfg.vs + s); };
    const uint32_t bar1 = bar0 + 8 * (2 * cfg.ks + 2 * cfg.vs);
    auto s_full = [&](int s) { return bar1 + 8 * s; };
    auto s_free = [&](int s) { return bar1 + 8 * (2 + s); };
    auto p_full = [&](int s) { return bar1 + 8 * (4 + s); };
    auto p_free = [&](int s) { return bar1 + 8 * (4 + cfg.pb + s); };
    const uint32_t drain_bar = bar1 + 8 * (4 + 2 * cfg.pb);

    // ------------------------------------------------------------------ prologue
    if (tid == 0) {
        for (int s = 0; s < cfg.ks; ++s) { mbar_init(k_full(s), 1); mbar_init(k_empty(s), 1); }
        for (int s = 0; s < cfg.vs; ++s) { mbar_init(v_full(s), 1); mbar_init(v_empty(s), 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(s_full(s), 1); mbar_init(s_free(s), 128); }
        for (int s = 0; s < cfg.pb; ++s) { mbar_init(p_full(s), 128); mbar_init(p_free(s), 1); }
        mbar_init(drain_bar, 1);
        *abort_flag = 0;
        mbar_fence_init();
        prefetch_tensormap(&tmap_k);
        prefetch_tensormap(&tmap_v);
    }
    if (warp == 1) {
        tmem_alloc(base + sm.misc, (uint32_t)cfg.tmem_cols);
        tmem_relinquish();
    }
    if (warp == 2 || warp == 3) {
        const int idx = tid - 64;
        // Q rows of this KV head, K-major with the 128-byte swizzle: two halves of
        // 64 channels, rows of 128 bytes, 16-byte chunk c of row r stored at c ^ (r % 8)
        for (int i = idx; i < NP * 16; i += 64) {
            const int r = i >> 4, c = i & 15, h = c >> 3, cc = c & 7;
            uint4 val = make_uint4(0, 0, 0, 0);
            if (r < M) {
                const int g = r / G, hg = r - g * G;
                const size_t off = (((size_t)b * gamma + g) * p.Hq + kvh * G + hg) * 128 + c * 8;
                val = *reinterpret_cast<const uint4 *>(p.q + off);
            }
            uint8_t *dst = gbase + sm.q + h * (NP * 128) + (r >> 3) * 1024 + (r & 7) * 128 +
                           ((cc ^ (r & 7)) << 4);
            *reinterpret_cast<uint4 *>(dst) = val;
        }
        // P buffers and the constant tiles start as zeros
        for (uint32_t i = idx * 16; i < (uint32_t)(cfg.pb * NP * 256) + 4 * kA2Bytes; i += 64 * 16)
            *reinterpret_cast<uint4 *>(gbase + sm.p + i) = make_uint4(0, 0, 0, 0);
        for (int n = idx; n < NP; n += 64) m_s[n] = kMFloor;
        asm volatile("bar.sync 2, 64;" ::: "memory");
        // constant 64 x 16 tiles (K-major, no swizzle: chunk c of 8 positions at
        // c * 1024, row r at (r / 8) * 128 + (r % 8) * 16).  Row 0 = ones (sums l),
        // row 1 = 1 inside the visual span (sums l_vis).
        // tile 0: inside the span, 1: outside, 2: the 16-block holding span start,
        // 3: the 16-block holding span end
        if (idx < 64) {
            const int tile = idx >> 4, kpos = idx & 15, c = kpos >> 3, e = kpos & 7;
            uint16_t *t16 = reinterpret_cast<uint16_t *>(gbase + sm.a2 + tile * kA2Bytes + c * 1024);
            int ind;
            if (tile == 0) ind = 1;
            else if (tile == 1) ind = 0;
            else {
                const int pos = ((tile == 2 ? vs : ve) & ~15) + kpos;
                ind = (pos >= vs && pos < ve) ? 1 : 0;
            }
            t16[e] = 0x3F80;                    // row 0
            t16[8 + e] = ind ? 0x3F80 : 0;      // row 1
        }
        fence_proxy_async_smem();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tm_s0 = tmem_base, tm_o = tmem_base + 2 * NP, tm_l = tmem_base + 3 * NP;
    const int bh = b * p.Hkv + kvh;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int i = 0;
            for (; i < T; ++i) {
                const int pos0 = (t_begin + i) * kTilePos;
                const int ks = i % cfg.ks;
                if (i >= cfg.ks && !mbar_wait(k_empty(ks), ((i / cfg.ks) - 1) & 1, abort_flag)) break;
                mbar_arrive_expect_tx(k_full(ks), kSlotBytes);
                tma_load_3d(base + sm.k + ks * kSlotBytes, &tmap_k, k_full(ks), 0, pos0, bh);
                tma_load_3d(base + sm.k + ks * kSlotBytes + kBoxBytes, &tmap_k, k_full(ks), 64, pos0, bh);
                const int vsl = i % cfg.vs;
                if (i >= cfg.vs && !mbar_wait(v_empty(vsl), ((i / cfg.vs) - 1) & 1, abort_flag)) {
                    // the K load of this tile is already in flight: wait for it here
                    wait_unconditional(k_full(ks), (i / cfg.ks) & 1);
                    break;
                }
                mbar_arrive_expect_tx(v_full(vsl), kSlotBytes);
                tma_load_3d(base + sm.v + vsl * kSlotBytes, &tmap_v, v_full(vsl), 0, pos0, bh);
                tma_load_3d(base + sm.v + vsl * kSlotBytes + kBoxBytes, &tmap_v, v_full(vsl), 64, pos0, bh);
            }
            if (*abort_flag) {
                // wait (bounded) for the copies still in flight before the CTA leaves
                for (int j = max(0, i - cfg.ks); j < i; ++j)
                    wait_unconditional(k_full(j % cfg.ks), (j / cfg.ks) & 1);
                for (int j = max(0, i - cfg.vs); j < i; ++j)
                    wait_unconditional(v_full(j % cfg.vs), (j / cfg.vs) & 1);
            }
        }
    } else if (warp == 1) {
        // -------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            const uint32_t idesc_qk = make_idesc_bf16(128, NP, 0, 0);
            const uint32_t idesc_pv = make_idesc_bf16(128, NP, 1, 1);
            const uint32_t idesc_sum = make_idesc_bf16(64, NP, 0, 1);
            auto issue_qk = [&](int i) -> bool {
                const int ks = i % cfg.ks, sb = i & 1;
                if (!mbar_wait(k_full(ks), (i / cfg.ks) & 1, abort_flag)) return false;
                if (i >= 2 && !mbar_wait(s_free(sb), ((i >> 1) - 1) & 1, abort_flag)) return false;
                tc_fence_after();
                const uint32_t kslot = base + sm.k + ks * kSlotBytes;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const uint64_t da = make_smem_desc(kslot + (j >> 2) * kBoxBytes + (j & 3) * 32, 16,
                                                       1024, kSwizzle128B);
                    const uint64_t db = make_smem_desc(base + sm.q + (j >> 2) * (NP * 128) + (j & 3) * 32,
                                                       16, 1024, kSwizzle128B);
                    mma_f16_ss(tm_s0 + sb * NP, da, db, idesc_qk, j > 0);
                }
                mma_commit(s_full(sb));
                mma_commit(k_empty(ks));
                return true;
            };
            bool ok = issue_qk(0);
            for (int i = 0; ok && i < T; ++i) {
                if (i + 1 < T && !issue_qk(i + 1)) break;
                const int pb = i % cfg.pb, vsl = i % cfg.vs;
                if (!mbar_wait(p_full(pb), (i / cfg.pb) & 1, abort_flag)) break;
                if (!mbar_wait(v_full(vsl), (i / cfg.vs) & 1, abort_flag)) break;
                tc_fence_after();
                const uint32_t vslot = base + sm.v + vsl * kSlotBytes;
                const uint32_t pbuf = base + sm.p + pb * (NP * 256);
                const int pos0 = (t_begin + i) * kTilePos;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    // V^T: channels contiguous (M-major), 64-channel halves kBoxBytes apart,
                    // groups of 8 positions 1024 bytes apart
                    const uint64_t da = make_smem_desc(vslot + j * 2048, kBoxBytes, 1024, kSwizzle128B);
                    // P^T: rows contiguous in 16-byte chunks (N-major), chunk stride 2048,
                    // groups of 8 positions 128 bytes apart
                    const uint64_t db = make_smem_desc(pbuf + j * 256, 128, 2048, kSwizzleNone);
                    const uint32_t acc = (i > 0 || j > 0) ? 1u : 0u;
                    mma_f16_ss(tm_o, da, db, idesc_pv, acc);
                    const int pblk = pos0 + 16 * j;
                    int tile;
                    if (pblk >= vs && pblk + 16 <= ve) tile = 0;
                    else if (pblk + 16 <= vs || pblk >= ve) tile = 1;
                    else if ((vs & ~15) == pblk) tile = 2;
                    else tile = 3;
                    const uint64_t d2 = make_smem_desc(base + sm.a2 + tile * kA2Bytes, 1024, 128,
                                                       kSwizzleNone);
                    mma_f16_ss(tm_l, d2, db, idesc_sum, acc);
                }
                mma_commit(v_empty(vsl));
                mma_commit(p_free(pb));
            }
            // every MMA issued by this thread has finished before TMEM is released
            mma_commit(drain_bar);
            wait_unconditional(drain_bar, 0);
        }
    } else if (warp >= 4) {
        // ------------------------------------------------------------ softmax warps
        const int wq = warp & 3;
        const int row = wq * 32 + lane;                 // TMEM lane = position inside the tile
        const uint32_t lane_addr = (uint32_t)(wq * 32) << 16;
        const int wtid = tid - 128;
        const float scale = p.scale_log2;
        for (int i = 0; i < T; ++i) {
            const int pos0 = (t_begin + i) * kTilePos;
            const int pos = pos0 + row;
            const int sb = i & 1, pb = i % cfg.pb;
            mbar_wait(s_full(sb), (i >> 1) & 1, abort_flag);
            tc_fence_after();
            if (i >= cfg.pb) mbar_wait(p_free(pb), ((i / cfg.pb) - 1) & 1, abort_flag);
            const bool tail = pos0 + kTilePos > L - gamma;
            const int gmin = pos - L + gamma;           // queries g < gmin do not see `pos`
            if (tail) {
                // slots at or beyond kv_len hold whatever the cache holds: zero their V
                // rows so that 0 * junk cannot poison the accumulators
                mbar_wait(v_full(i % cfg.vs), (i / cfg.vs) & 1, abort_flag);
                if (pos >= L) {
                    uint8_t *vrow = gbase + sm.v + (i % cfg.vs) * kSlotBytes + row * 128;
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        *reinterpret_cast<uint4 *>(vrow + c * 16) = make_uint4(0, 0, 0, 0);
                        *reinterpret_cast<uint4 *>(vrow + kBoxBytes + c * 16) = make_uint4(0, 0, 0, 0);
                    }
                }
            }
            uint8_t *prow = gbase + sm.p + pb * (NP * 256) + row * 16;
            const uint32_t s_addr = tm_s0 + sb * NP + lane_addr;

            for (int attempt = 0; attempt < 3; ++attempt) {
                float gmax = -INFINITY;
                for (int c8 = 0; c8 < n8; ++c8) {
                    uint32_t r[8];
                    tmem_ld_x8(s_addr + c8 * 8, r);
                    const float4 ma = *reinterpret_cast<const float4 *>(m_s + c8 * 8);
                    const float4 mb = *reinterpret_cast<const float4 *>(m_s + c8 * 8 + 4);
                    const float mm[8] = {ma.x, ma.y, ma.z, ma.w, mb.x, mb.y, mb.z, mb.w};
                    tmem_wait_ld();
                    float x[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k) x[k] = fmaf(__uint_as_float(r[k]), scale, -mm[k]);
                    if (tail) {
#pragma unroll
                        for (int k = 0; k < 8; ++k)
                            x[k] = ((c8 * 8 + k) / G >= gmin) ? x[k] : -INFINITY;
                    }
#pragma unroll
                    for (int k = 0; k < 8; ++k) gmax = fmaxf(gmax, x[k]);
                    uint4 pk;
                    pk.x = pack_bf16x2(ex2(x[0]), ex2(x[1]));
                    pk.y = pack_bf16x2(ex2(x[2]), ex2(x[3]));
                    pk.z = pack_bf16x2(ex2(x[4]), ex2(x[5]));
                    pk.w = pack_bf16x2(ex2(x[6]), ex2(x[7]));
                    *reinterpret_cast<uint4 *>(prow + c8 * 2048) = pk;
                }
                if (!wg_any(gmax > kGuard)) break;

                // ---- a score ran past the guard: move m up to the tile maximum ----
                for (int c8 = 0; c8 < n8; ++c8) {
                    uint32_t r[8];
                    tmem_ld_x8(s_addr + c8 * 8, r);
                    tmem_wait_ld();
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        float s2 = __uint_as_float(r[k]) * scale;
                        if (tail && (c8 * 8 + k) / G < gmin) s2 = -INFINITY;
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1)
                            s2 = fmaxf(s2, __shfl_xor_sync(0xffffffffu, s2, o));
                        if (lane == 0) tmx_s[wq * NP + c8 * 8 + k] = s2;
                    }
                }
                wg_sync();
                for (int n = wtid; n < n8 * 8; n += 128) {
                    const float mt = fmaxf(fmaxf(tmx_s[n], tmx_s[NP + n]),
                                           fmaxf(tmx_s[2 * NP + n], tmx_s[3 * NP + n]));
                    const float mo = m_s[n];
                    const float mn = fmaxf(mo, mt);
                    dl_s[n] = mo - mn;              // <= 0
                    m_s[n] = mn;
                }
                wg_sync();
                if (i > 0) {
                    // O^T and the sums were accumulated under the old m: rescale them
                    // once PV(i-1) has finished
                    mbar_wait(p_free((i - 1) % cfg.pb), ((i - 1) / cfg.pb) & 1, abort_flag);
                    tc_fence_after();
                    for (int c8 = 0; c8 < n8; ++c8) {
                        uint32_t r[8];
                        tmem_ld_x8(tm_o + lane_addr + c8 * 8, r);
                        tmem_wait_ld();
#pragma unroll
                        for (int k = 0; k < 8; ++k)
                            r[k] = __float_as_uint(__uint_as_float(r[k]) * ex2(dl_s[c8 * 8 + k]));
                        tmem_st_x8(tm_o + lane_addr + c8 * 8, r);
                        if (wq == 0) {
                            tmem_ld_x8(tm_l + c8 * 8, r);
                            tmem_wait_ld();
#pragma unroll
                            for (int k = 0; k < 8; ++k)
                                r[k] = __float_as_uint(__uint_as_float(r[k]) * ex2(dl_s[c8 * 8 + k]));
                            tmem_st_x8(tm_l + c8 * 8, r);
                        }
                    }
                    tmem_wait_st();
                    tc_fence_before();
                }
                wg_sync();
            }
            // S^T has been read: the MMA warp may overwrite this buffer
            tc_fence_before();
            mbar_arrive(s_free(sb));
            // P^T (and zeroed V rows) are in shared memory: visible to the tensor core
            fence_proxy_async_smem();
            mbar_arrive(p_full(pb));
        }

        // ---------------------------------------------------------------- epilogue
        mbar_wait(p_free((T - 1) % cfg.pb), ((T - 1) / cfg.pb) & 1, abort_flag);
        tc_fence_after();
        for (int c8 = 0; c8 < n8; ++c8) {
            uint32_t r[8];
            tmem_ld_x8(tm_o + lane_addr + c8 * 8, r);
            tmem_wait_ld();
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int n = c8 * 8 + k;
                if (n < M) part_o[(size_t)n * 128 + row] = __uint_as_float(r[k]);
            }
            if (wq == 0) {
                tmem_ld_x8(tm_l + c8 * 8, r);     // lane 0: l, lane 1: l_vis
                tmem_wait_ld();
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const int n = c8 * 8 + k;
                    const float lv = __shfl_sync(0xffffffffu, __uint_as_float(r[k]), 1);
                    if (lane == 0 && n < M)
                        *reinterpret_cast<float4 *>(part_stat + n * 4) =
                            make_float4(m_s[n], __uint_as_float(r[k]), lv, 0.f);
                }
            }
        }
        tc_fence_before();
    }

    // ------------------------------------------------------------------ teardown
    __syncthreads();
    if (tid == 0 && *abort_flag) atomicOr(p.status, LVSPEC_DEV_WAIT_EXPIRED);
    if (warp == 1) {
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

// [B*Hkv][Lmax][128] bf16 viewed as a 3-D tensor; boxes of 64 channels x 128 positions
bool make_kv_map(CUtensorMap *map, const void *ptr, int Lmax, int BH)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {128, (cuuint64_t)Lmax, (cuuint64_t)BH};
    const cuuint64_t strides[2] = {256, (cuuint64_t)Lmax * 256};
    const cuuint32_t box[3] = {64, 128, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(ptr), dims, strides, box,
              estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

TcConfig pick_config(int M)
{
    TcConfig c;
    c.n_pad = (M + 15) & ~15;
    if (c.n_pad <= 64) { c.ks = 2; c.vs = 3; c.pb = 2; }
    else if (c.n_pad <= 96) { c.ks = 2; c.vs = 2; c.pb = 2; }
    else { c.ks = 2; c.vs = 2; c.pb = 1; }
    int cols = 32;
    while (cols < 4 * c.n_pad) cols <<= 1;
    c.tmem_cols = cols;
    return c;
}

}  // namespace

bool attn_tc_supported(const AttnParams &p)
{
    return p.D == 128 && p.Lmax >= kTilePos && p.M <= LVSPEC_MAX_ROWS;
}

cudaError_t launch_attn_tc(const AttnParams &p, const SeqInfo &seq, cudaStream_t stream, int *launches)
{
    TcParams P;
    P.a = p;
    P.cfg = pick_config(p.M);
    CUtensorMap mk, mv;
    if (!make_kv_map(&mk, p.k, p.Lmax, p.B * p.Hkv) || !make_kv_map(&mv, p.v, p.Lmax, p.B * p.Hkv))
        return cudaErrorInvalidValue;
    const size_t smem = smem_map(P.cfg).total + 1024;
    cudaError_t err = cudaFuncSetAttribute(attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           (int)smem);
    if (err != cudaSuccess) return err;
    dim3 grid(p.n_split, p.Hkv, p.B);
    attn_tc_kernel<<<grid, kThreads, smem, stream>>>(P, seq, mk, mv);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace lvspec
