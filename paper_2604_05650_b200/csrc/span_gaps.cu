// Visual mass over several spans (video frames with text between them).
//
// The attention kernels fuse the mass of ONE span into their softmax.  For several
// spans they run on the hull [first start, last end), and this kernel takes off
// what the positions between the spans hold: for every gap position j and query
// row, p_j = exp2(scale * <q, k_j> - lse2), with lse2 the log2 of the row's softmax
// denominator that the combine kernel leaves behind.  Gap positions are few (a few
// text tokens per frame), only the layer whose mass feeds the rule needs it, and
// all of them lie before the draft slots, so every draft query sees them.
//
// One CTA per KV head and group of eight query rows of one sequence: warp w owns row
// 8 * blockIdx.y + w, lane l owns positions l, l + 32, l + 64, l + 96 of every tile of 128
// gap positions (few, long rounds: a round costs a trip to memory for the keys); a row's
// sum over the lanes is a fixed butterfly, so the result does not depend on scheduling.
#include "lvspec_internal.h"

namespace lvspec {
namespace {

constexpr int kGapThreads = 256;
constexpr int kGapTile = 128;
constexpr int kKeyStride = 65;   // 32-bit words per staged key row (64 + 1: no bank conflicts)

__device__ __forceinline__ float2 bf16x2_to_float2(uint32_t w)
{
    return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}

__global__ void __launch_bounds__(kGapThreads) gap_mass_kernel(const GapParams p)
{
    __shared__ __align__(16) uint32_t q_s[8 * 64];      // this CTA's rows, bf16 pairs
    __shared__ uint32_t k_s[kGapTile * kKeyStride];
    __shared__ int first_s[kMaxGaps + 1];               // flat index of each gap's first position
    __shared__ int start_s[kMaxGaps];                   // cache position of each gap's first position
    __shared__ int pos_s[kGapTile];                     // cache position of each slot of the tile
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int kvh = blockIdx.x, b = p.b;
    const int M = p.M, G = p.G, words = p.D / 2;        // 32-bit words per row
    const int r = blockIdx.y * 8 + warp;                // row g * G + hg of this head: query g, head kvh * G + hg
    const bool row_ok = r < M;
    const int g = row_ok ? r / G : 0, hg = row_ok ? r - g * G : 0;
    const size_t out_idx = ((size_t)b * p.gamma + g) * p.Hq + kvh * G + hg;

    for (int i = tid; i <= p.n_gaps; i += kGapThreads) {
        first_s[i] = p.gap_first[i];
        if (i < p.n_gaps) start_s[i] = p.gap_start[i];
    }
    {
        const uint32_t *src = reinterpret_cast<const uint32_t *>(p.q + out_idx * p.D);
        for (int w = lane; w < 64; w += 32) q_s[warp * 64 + w] = (row_ok && w < words) ? src[w] : 0u;
    }
    __syncthreads();
    const int total = first_s[p.n_gaps];
    const uint16_t *k_head = p.k + ((size_t)b * p.Hkv + kvh) * (size_t)p.Lmax * p.D;
    const float lse = row_ok ? p.lse2[out_idx] : 0.f;

    float corr = 0.f;
    for (int f0 = 0; f0 < total; f0 += kGapTile) {
        if (tid < kGapTile) {
            const int f = f0 + tid;
            int pos = -1;
            if (f < total) {
                int lo = 0, hi = p.n_gaps - 1;      // the last gap whose first index is <= f
                while (lo < hi) {
                    const int mid = (lo + hi + 1) >> 1;
                    if (first_s[mid] <= f) lo = mid;
                    else hi = mid - 1;
                }
                pos = start_s[lo] + (f - first_s[lo]);
            }
            pos_s[tid] = pos;
        }
        __syncthreads();
        // warp w stages the keys w, w + 8, ...: all loads of a batch of eight keys are
        // issued before any is stored (one trip to memory per batch, not per key)
#pragma unroll 1
        for (int j0 = warp; j0 < kGapTile; j0 += 64) {
            uint32_t lo[8], hi[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int j = j0 + 8 * u;
                const int pos = j < kGapTile ? pos_s[j] : -1;
                const uint32_t *src = reinterpret_cast<const uint32_t *>(k_head + (size_t)(pos >= 0 ? pos : 0) * p.D);
                lo[u] = pos >= 0 ? __ldg(src + lane) : 0u;
                hi[u] = (pos >= 0 && words > 32) ? __ldg(src + 32 + lane) : 0u;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int j = j0 + 8 * u;
                if (j < kGapTile) {
                    k_s[j * kKeyStride + lane] = lo[u];
                    k_s[j * kKeyStride + 32 + lane] = hi[u];
                }
            }
        }
        __syncthreads();
        if (row_ok) {
            const uint4 *qr = reinterpret_cast<const uint4 *>(q_s + warp * 64);
            float dot[kGapTile / 32];
#pragma unroll
            for (int t = 0; t < kGapTile / 32; ++t) dot[t] = 0.f;
            for (int w4 = 0; w4 < words / 4; ++w4) {
                const uint4 qq = qr[w4];
                const uint32_t qw[4] = {qq.x, qq.y, qq.z, qq.w};
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const float2 a = bf16x2_to_float2(qw[u]);
#pragma unroll
                    for (int t = 0; t < kGapTile / 32; ++t) {
                        const float2 c = bf16x2_to_float2(k_s[(lane + 32 * t) * kKeyStride + w4 * 4 + u]);
                        dot[t] = fmaf(a.x, c.x, dot[t]);
                        dot[t] = fmaf(a.y, c.y, dot[t]);
                    }
                }
            }
#pragma unroll
            for (int t = 0; t < kGapTile / 32; ++t)
                if (pos_s[lane + 32 * t] >= 0) corr += exp2f(dot[t] * p.scale_log2 - lse);
        }
        __syncthreads();
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) corr += __shfl_xor_sync(0xffffffffu, corr, o);
    if (lane == 0 && row_ok) p.mass[out_idx] = fmaxf(p.mass[out_idx] - corr, 0.f);
}

}  // namespace

cudaError_t launch_gap_mass(const GapParams &p, cudaStream_t stream, int *launches)
{
    gap_mass_kernel<<<dim3(p.Hkv, (p.M + 7) / 8), kGapThreads, 0, stream>>>(p);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace lvspec
