// Verification attention with fused visual mass, CUDA-core (SIMT) kernel, and
// the split-KV combine kernel.  Covers every supported shape; it is the plain
// device implementation the tensor-core kernel is cross-checked with.
//
// One CTA owns one KV split of one (sequence, KV head) and all M = gamma * G
// query rows that read that head (row r = g * G + hg).  Per tile of 32 cache
// positions: scores by fp32 FMA from shared memory, an online softmax per row
// (fp32, base-2 exponent), the running sums l and l_vis (probability mass
// inside the visual span) and the P.V update.  The unnormalised partials go to
// scratch memory; `attn_combine_kernel` merges the splits.
#include <cuda_bf16.h>

#include "lvspec_internal.h"

#ifdef LVSPEC_TRACE
cudaError_t lvspec::trace_set_buffer_merge(unsigned long long *device_words)
{
    return cudaMemcpyToSymbol(g_lvspec_trace, &device_words, sizeof device_words);
}
#endif

namespace lvspec {
namespace {

constexpr int kTile = 32;      // cache positions per tile
constexpr int kThreads = 256;

__device__ __forceinline__ float bf16_bits_to_float(uint16_t b)
{
    return __uint_as_float(((uint32_t)b) << 16);
}

__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int D>
__global__ void __launch_bounds__(kThreads)
attn_simt_kernel(const AttnParams p, const SeqInfo seq)
{
    constexpr int DP = D + 4;                 // padded row: conflict-free float4 reads
    constexpr int D4 = D / 4;
    constexpr int kRowGroups = kThreads / D4; // thread (rg, d4) accumulates rows rg, rg+kRowGroups, ...
    constexpr int kMaxRowsPerThread = (LVSPEC_MAX_ROWS + kRowGroups - 1) / kRowGroups;

    extern __shared__ __align__(16) float smem[];
    const int M = p.M;
    float *q_s = smem;                        // [M][DP]
    float *k_s = q_s + (size_t)M * DP;        // [kTile][DP]
    float *v_s = k_s + kTile * DP;            // [kTile][DP]
    float *s_s = v_s + kTile * DP;            // [M][kTile]  scores, then probabilities
    float *m_s = s_s + (size_t)M * kTile;     // [M]
    float *l_s = m_s + M;
    float *lv_s = l_s + M;
    float *corr_s = lv_s + M;

    const int split = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int L = seq.kv_len[b];
    const int vs = seq.span_start[b], ve = seq.span_end[b];
    const int G = p.G, gamma = p.gamma;

    // split ranges are whole tiles
    const int n_tiles = (L + kTile - 1) / kTile;
    const int tiles_per_split = (n_tiles + p.n_split - 1) / p.n_split;
    const int t_begin = split * tiles_per_split;
    const int t_end = min(n_tiles, t_begin + tiles_per_split);

    // Q rows of this KV head -> shared memory as fp32
    for (int i = tid; i < M * D; i += kThreads) {
        const int r = i / D, d = i - r * D;
        const int g = r / G, hg = r - g * G;
        const size_t off = (((size_t)b * gamma + g) * p.Hq + kvh * G + hg) * D + d;
        q_s[r * DP + d] = bf16_bits_to_float(p.q[off]);
    }
    for (int r = tid; r < M; r += kThreads) {
        m_s[r] = -INFINITY;
        l_s[r] = 0.f;
        lv_s[r] = 0.f;
    }

    const int d4 = tid % D4, rg = tid / D4;
    float4 acc[kMaxRowsPerThread];
#pragma unroll
    for (int i = 0; i < kMaxRowsPerThread; ++i) acc[i] = make_float4(0.f, 0.f, 0.f, 0.f);

    const uint16_t *kbase = p.k + (size_t)b * p.k_sb + (size_t)kvh * p.k_sh;
    const uint16_t *vbase = p.v + (size_t)b * p.v_sb + (size_t)kvh * p.v_sh;
    __syncthreads();

    for (int t = t_begin; t < t_end; ++t) {
        const int pos0 = t * kTile;
        // K and V tile -> shared memory (8 bf16 per 16-byte load)
        for (int i = tid; i < kTile * (D / 8); i += kThreads) {
            const int j = i / (D / 8), c = i - j * (D / 8);
            const int pos = pos0 + j;
            uint4 kk = make_uint4(0, 0, 0, 0), vv = make_uint4(0, 0, 0, 0);
            if (pos < L) {
                kk = *reinterpret_cast<const uint4 *>(kbase + (size_t)pos * p.k_sp + c * 8);
                vv = *reinterpret_cast<const uint4 *>(vbase + (size_t)pos * p.v_sp + c * 8);
            }
            const uint32_t kw[4] = {kk.x, kk.y, kk.z, kk.w}, vw[4] = {vv.x, vv.y, vv.z, vv.w};
            float *kd = k_s + j * DP + c * 8, *vd = v_s + j * DP + c * 8;
#pragma unroll
            for (int w = 0; w < 4; ++w) {
                kd[2 * w] = __uint_as_float(kw[w] << 16);
                kd[2 * w + 1] = __uint_as_float(kw[w] & 0xffff0000u);
                vd[2 * w] = __uint_as_float(vw[w] << 16);
                vd[2 * w + 1] = __uint_as_float(vw[w] & 0xffff0000u);
            }
        }
        __syncthreads();

        // scores: s[r][j], one (r, j) pair per thread per pass
        for (int i = tid; i < M * kTile; i += kThreads) {
            const int r = i / kTile, j = i - r * kTile;
            const float4 *qr = reinterpret_cast<const float4 *>(q_s + r * DP);
            const float4 *kr = reinterpret_cast<const float4 *>(k_s + j * DP);
            float s = 0.f;
#pragma unroll 8
            for (int c = 0; c < D4; ++c) {
                const float4 a = qr[c], k4 = kr[c];
                s = fmaf(a.x, k4.x, s);
                s = fmaf(a.y, k4.y, s);
                s = fmaf(a.z, k4.z, s);
                s = fmaf(a.w, k4.w, s);
            }
            s_s[i] = s * p.scale_log2;
        }
        __syncthreads();

        // online softmax, one warp per row, lane = position inside the tile
        for (int r = warp; r < M; r += kThreads / 32) {
            const int g = r / G;
            const int pos = pos0 + lane;
            const bool visible = pos < L && draft_query_sees(g, pos - (L - gamma), p.branch_len);
            const float s = visible ? s_s[r * kTile + lane] : -INFINITY;
            float mx = s;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            const float m_old = m_s[r];
            const float m_new = fmaxf(m_old, mx);
            float pr = 0.f, corr = 1.f;
            if (m_new > -INFINITY) {
                pr = visible ? fast_exp2(s - m_new) : 0.f;
                corr = fast_exp2(m_old - m_new);  // m_old = -inf gives 0
            }
            float sum = pr, sumv = (pos >= vs && pos < ve) ? pr : 0.f;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                sum += __shfl_xor_sync(0xffffffffu, sum, o);
                sumv += __shfl_xor_sync(0xffffffffu, sumv, o);
            }
            s_s[r * kTile + lane] = pr;
            if (lane == 0) {
                m_s[r] = m_new;
                l_s[r] = l_s[r] * corr + sum;
                lv_s[r] = lv_s[r] * corr + sumv;
                corr_s[r] = corr;
            }
        }
        __syncthreads();

        // O[r][:] = O[r][:] * corr + sum_j p[r][j] * V[j][:]
#pragma unroll
        for (int i = 0; i < kMaxRowsPerThread; ++i) {
            const int r = rg + i * kRowGroups;
            if (r < M) {
                const float c = corr_s[r];
                float4 a = acc[i];
                a.x *= c; a.y *= c; a.z *= c; a.w *= c;
                const float *pr = s_s + r * kTile;
#pragma unroll 8
                for (int j = 0; j < kTile; ++j) {
                    const float pj = pr[j];
                    const float4 v4 = *reinterpret_cast<const float4 *>(v_s + j * DP + d4 * 4);
                    a.x = fmaf(pj, v4.x, a.x);
                    a.y = fmaf(pj, v4.y, a.y);
                    a.z = fmaf(pj, v4.z, a.z);
                    a.w = fmaf(pj, v4.w, a.w);
                }
                acc[i] = a;
            }
        }
        __syncthreads();
    }

    // partials of this split
    const size_t unit = ((size_t)b * p.Hkv + kvh) * p.n_split + split;
    float *po = p.part_o + unit * (size_t)M * D;
#pragma unroll
    for (int i = 0; i < kMaxRowsPerThread; ++i) {
        const int r = rg + i * kRowGroups;
        if (r < M) *reinterpret_cast<float4 *>(po + (size_t)r * D + d4 * 4) = acc[i];
    }
    float *ps = p.part_stat + unit * (size_t)M * 4;
    for (int r = tid; r < M; r += kThreads)
        *reinterpret_cast<float4 *>(ps + r * 4) = make_float4(m_s[r], l_s[r], lv_s[r], 0.f);
}

// Merge of the KV splits: one warp per (sequence, KV head, row), each lane four
// output channels.  The result does not depend on scheduling (every sum has a fixed
// order).  The kernel may be launched programmatically dependent on the attention
// kernel: it lets the next launch be scheduled, then waits for the partials.
//
// The kernel runs once per layer on cold instruction caches, where straight-line code
// costs about ten cycles per instruction: so the splits' rows come in by cp.async in a
// short rolled loop (a batch of up to 32 splits per round trip to L2, landing in shared
// memory), lane u meanwhile turns the statistics of split u into its weight, and a second
// rolled loop accumulates from shared memory.  The running reference exponent moves up
// between batches like an online softmax.
constexpr int kCombineBatch = 32;
constexpr int kCombineWarps = 2;

__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gmem_src)
{
    const uint32_t dst = (uint32_t)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(gmem_src) : "memory");
}

// dynamic shared memory per warp: `batch` rows of 32 float4, then `batch` weights
__global__ void __launch_bounds__(32 * kCombineWarps) attn_combine_kernel(const AttnParams p, const int batch)
{
    extern __shared__ float4 combine_smem[];
#ifdef LVSPEC_TRACE
    const unsigned long long trace_t0 = lvspec_trace_now();
#endif
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // every address is worked out before the wait for the attention grid: the CTA is
    // resident by then, and the cold parameter loads and index arithmetic cost it nothing
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int r = blockIdx.x * kCombineWarps + w, kvh = blockIdx.y, b = blockIdx.z;
    const int M = p.M, D = p.D, ns = p.n_split;
    if (r >= M) return;
    const bool active = lane * 4 < D;                   // D = 64 uses half the lanes
    float4 *rows = combine_smem + (size_t)w * (batch * 32 + (batch + 3) / 4);
    float *weights = reinterpret_cast<float *>(rows + batch * 32);
    const size_t unit0 = ((size_t)b * p.Hkv + kvh) * ns;
    const float4 *ps = reinterpret_cast<const float4 *>(p.part_stat) + unit0 * (size_t)M + r;
    const float4 *po = reinterpret_cast<const float4 *>(p.part_o + (unit0 * (size_t)M + r) * D) +
                       (active ? lane : 0);
    const size_t o_stride = (size_t)M * D / 4;          // float4 units between splits
    const int g = r / p.G, hg = r - g * p.G;
    const size_t row = ((size_t)b * p.gamma + g) * p.Hq + kvh * p.G + hg;
    uint16_t *out_row = p.out + row * D + lane * 4;
    float *mass_row = p.mass + row;
    float *lse_row = p.lse2 ? p.lse2 + row : nullptr;
    asm volatile("griddepcontrol.wait;" ::: "memory");
#ifdef LVSPEC_TRACE
    unsigned long long *rec = nullptr;
    if (g_lvspec_trace && threadIdx.x == 0) {
        const unsigned long long idx = atomicAdd(g_lvspec_trace, 1ull);
        if (idx < (unsigned long long)kTraceCtaRecords) {
            rec = g_lvspec_trace + 8 + idx * 8;
            rec[0] = 2;
            rec[1] = (unsigned long long)p.q;
            rec[2] = blockIdx.x + 1000 * blockIdx.y + 1000000 * blockIdx.z;
            rec[3] = trace_t0;
            rec[4] = lvspec_trace_now();
        }
    }
#endif

    float m_run = -INFINITY, l = 0.f, lv = 0.f;
    float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s0 = 0; s0 < ns; s0 += batch) {
        const int n = min(batch, ns - s0);
        // the statistics first: the weights hang on them, the rows are only needed after
        float4 st = make_float4(-INFINITY, 0.f, 0.f, 0.f);
        if (lane < n) st = __ldcg(ps + (size_t)(s0 + lane) * M);
        if (active) {
            const float4 *src = po + (size_t)s0 * o_stride;
            float4 *dst = rows + lane;
            for (int u = 0; u < n; ++u, src += o_stride, dst += 32) cp_async16(dst, src);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        float m_b = st.y > 0.f ? st.x : -INFINITY;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) m_b = fmaxf(m_b, __shfl_xor_sync(0xffffffffu, m_b, off));
        if (m_b > m_run) {
            const float c = exp2f(m_run - m_b);         // 0 on the first batch
            l *= c; lv *= c;
            o.x *= c; o.y *= c; o.z *= c; o.w *= c;
            m_run = m_b;
        }
        const float w_mine = st.y > 0.f ? exp2f(st.x - m_run) : 0.f;
        float sl = w_mine * st.y, slv = w_mine * st.z;   // two sums, one butterfly
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            sl += __shfl_xor_sync(0xffffffffu, sl, off);
            slv += __shfl_xor_sync(0xffffffffu, slv, off);
        }
        l += sl;
        lv += slv;
        if (lane < n) weights[lane] = w_mine;           // batch <= 32: one weight per lane
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncwarp();
        if (active) {
            const float4 *v = rows + lane;
#pragma unroll 3
            for (int u = 0; u < n; ++u, v += 32) {
                // a split without weight (no tile of its own, or all of it masked) may
                // have left its rows unwritten: whatever the scratch holds there, NaN
                // bit patterns included, must not reach the sum
                const float wu = weights[u];
                if (wu == 0.f) continue;
                const float4 x = *v;
                o.x = fmaf(wu, x.x, o.x);
                o.y = fmaf(wu, x.y, o.y);
                o.z = fmaf(wu, x.z, o.z);
                o.w = fmaf(wu, x.w, o.w);
            }
        }
        __syncwarp();
    }
    const float inv = 1.f / l;
    if (active) {
        __nv_bfloat162 lo = __floats2bfloat162_rn(o.x * inv, o.y * inv);
        __nv_bfloat162 hi = __floats2bfloat162_rn(o.z * inv, o.w * inv);
        uint2 pk;
        pk.x = *reinterpret_cast<uint32_t *>(&lo);
        pk.y = *reinterpret_cast<uint32_t *>(&hi);
        *reinterpret_cast<uint2 *>(out_row) = pk;
    }
    if (lane == 0) {
        *mass_row = lv * inv;
        if (lse_row) *lse_row = m_run + log2f(l);
    }
#ifdef LVSPEC_TRACE
    if (rec) rec[6] = lvspec_trace_now();
#endif
}

}  // namespace

cudaError_t launch_attn_simt(const AttnParams &p, const SeqInfo &seq, cudaStream_t stream,
                             int *launches)
{
    const int DP = p.D + 4;
    const size_t smem = sizeof(float) * ((size_t)p.M * DP + 2 * kTile * DP + (size_t)p.M * kTile +
                                         4 * (size_t)p.M);
    dim3 grid(p.n_split, p.Hkv, p.B);
    cudaError_t err;
    if (p.D == 128) {
        err = cudaFuncSetAttribute(attn_simt_kernel<128>,
                                   cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err != cudaSuccess) return err;
        attn_simt_kernel<128><<<grid, kThreads, smem, stream>>>(p, seq);
    } else {
        err = cudaFuncSetAttribute(attn_simt_kernel<64>,
                                   cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err != cudaSuccess) return err;
        attn_simt_kernel<64><<<grid, kThreads, smem, stream>>>(p, seq);
    }
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_attn_combine(const AttnParams &p, cudaStream_t stream, int *launches)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((p.M + kCombineWarps - 1) / kCombineWarps, p.Hkv, p.B);
    cfg.blockDim = dim3(32 * kCombineWarps, 1, 1);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = p.pdl ? 1 : 0;
    const int batch = p.n_split < kCombineBatch ? p.n_split : kCombineBatch;
    cfg.dynamicSmemBytes = (size_t)kCombineWarps * (batch * 32 + (batch + 3) / 4) * sizeof(float4);
    cudaError_t err = cudaLaunchKernelEx(&cfg, attn_combine_kernel, p, batch);
    ++*launches;
    return err != cudaSuccess ? err : cudaGetLastError();
}

}  // namespace lvspec
