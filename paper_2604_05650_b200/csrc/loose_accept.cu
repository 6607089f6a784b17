// Loose acceptance pass (Sec. 3.2 / 3.3): vocabulary-wide argmax of every
// target-logits row, then the rule and the accepted length, in one launch.
//
// Grid = (vocab slices, gamma, B).  Each CTA scans one slice of one row with
// 16-byte loads and reduces (value, index) pairs under the order "larger
// value first, then lower index" at every level (thread, warp, CTA, slice), so
// the result is the first occurrence of the row maximum whatever the
// partitioning.  The last CTA to finish for a sequence (an atomic ticket; no
// CTA ever waits on another) merges the slices and evaluates the rule.
#include "lvspec_internal.h"

namespace lvspec {
namespace {

constexpr int kThreads = 256;
constexpr int kNoIndex = 0x7fffffff;

struct Best {
    float v;
    int i;
};

__device__ __forceinline__ Best better(Best a, Best b)
{
    return (b.v > a.v || (b.v == a.v && b.i < a.i)) ? b : a;
}

__device__ __forceinline__ void take(Best &best, float x, int idx, bool &nan_seen)
{
    if (x != x) {                 // NaN ranks as -inf
        nan_seen = true;
        return;
    }
    if (x > best.v) {             // indices arrive in increasing order per thread
        best.v = x;
        best.i = idx;
    }
}

__global__ void __launch_bounds__(kThreads) loose_accept_kernel(const AcceptParams p)
{
    const int slice = blockIdx.x, i_pos = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int V = p.V, gamma = p.gamma;
    const size_t row_id = (size_t)b * gamma + i_pos;
    const float *row = p.logits + row_id * (size_t)V;

    // slice [c0, c1): equal shares rounded up to a multiple of 4 elements
    const int per = (((V + p.n_vsplit - 1) / p.n_vsplit) + 3) & ~3;
    const int c0 = min(V, slice * per), c1 = min(V, c0 + per);

    Best best = {-INFINITY, kNoIndex};
    bool nan_seen = false;
    // elements up to the first 16-byte boundary, vector body, tail
    const uintptr_t addr = reinterpret_cast<uintptr_t>(row + c0);
    int head = (int)(((16 - (addr & 15)) & 15) >> 2);
    head = min(head, c1 - c0);
    if (tid < head) take(best, row[c0 + tid], c0 + tid, nan_seen);
    const int body0 = c0 + head;
    const int n_vec = (c1 - body0) >> 2;
    const float4 *vec = reinterpret_cast<const float4 *>(row + body0);
    for (int j = tid; j < n_vec; j += kThreads) {
        const float4 x = __ldg(vec + j);
        const int idx = body0 + 4 * j;
        take(best, x.x, idx, nan_seen);
        take(best, x.y, idx + 1, nan_seen);
        take(best, x.z, idx + 2, nan_seen);
        take(best, x.w, idx + 3, nan_seen);
    }
    const int tail0 = body0 + 4 * n_vec;
    if (tail0 + tid < c1) take(best, row[tail0 + tid], tail0 + tid, nan_seen);
    // per thread the indices came in increasing order (head < body < tail), so a
    // strict ">" kept the first occurrence of the thread's maximum

#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        Best other;
        other.v = __shfl_xor_sync(0xffffffffu, best.v, o);
        other.i = __shfl_xor_sync(0xffffffffu, best.i, o);
        best = better(best, other);
    }
    __shared__ Best warp_best[kThreads / 32];
    __shared__ int s_nan;
    __shared__ bool s_last;
    if (tid == 0) s_nan = 0;
    __syncthreads();
    if (nan_seen) s_nan = 1;
    if (lane == 0) warp_best[warp] = best;
    __syncthreads();
    if (tid == 0) {
        Best bb = warp_best[0];
        for (int w = 1; w < kThreads / 32; ++w) bb = better(bb, warp_best[w]);
        p.part_val[row_id * p.n_vsplit + slice] = bb.v;
        p.part_idx[row_id * p.n_vsplit + slice] = bb.i;
        if (s_nan) atomicOr(p.status, LVSPEC_DEV_NAN_LOGIT);
        __threadfence();
        const unsigned total = (unsigned)(p.n_vsplit * gamma);
        const unsigned ticket = atomicAdd(p.counters + b, 1u);
        s_last = (ticket == total - 1);
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();

    // ---- last CTA of sequence b: merge slices, apply the rule ----
    __shared__ int y_s[LVSPEC_MAX_GAMMA];
    __shared__ int draft_s[LVSPEC_MAX_GAMMA];
    __shared__ double score_s[LVSPEC_MAX_GAMMA];
    __shared__ unsigned char acc_s[LVSPEC_MAX_GAMMA];
    // One warp per position (round robin): the lanes fetch the slices' partials and the
    // heads' masses side by side, so a position costs one round trip to L2, not one per
    // partial.  "Greater value, then lower index" is a total order: any reduction tree
    // gives the same winner.  The masses are added in index order, in double, as the rule
    // is defined: lane order restored by shuffles.
    for (int i = warp; i < gamma; i += kThreads / 32) {
        const size_t rid = (size_t)b * gamma + i;
        Best bb = {-INFINITY, kNoIndex};
        for (int s = lane; s < p.n_vsplit; s += 32) {
            Best o = {__ldcg(p.part_val + rid * p.n_vsplit + s), __ldcg(p.part_idx + rid * p.n_vsplit + s)};
            bb = better(bb, o);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            Best other;
            other.v = __shfl_xor_sync(0xffffffffu, bb.v, o);
            other.i = __shfl_xor_sync(0xffffffffu, bb.i, o);
            bb = better(bb, other);
        }
        double sc = 0.0;
        const float *mrow = p.mass + rid * p.Hm;
        for (int h0 = 0; h0 < p.Hm; h0 += 32) {
            const float mine = h0 + lane < p.Hm ? mrow[h0 + lane] : 0.f;
            const int n = min(32, p.Hm - h0);
            for (int h = 0; h < n; ++h) sc += (double)__shfl_sync(0xffffffffu, mine, h);
        }
        if (lane == 0) {
            y_s[i] = (bb.i == kNoIndex) ? 0 : bb.i;   // nothing above -inf: token 0
            draft_s[i] = p.draft[rid];
            score_s[i] = sc;
        }
    }
    __syncthreads();
    if (tid < gamma) {
        const double sc = score_s[tid];
        int rank = 0;                              // position in the ascending stable order
        for (int j = 0; j < gamma; ++j) {
            const double sj = score_s[j];
            rank += (sj < sc || (sj == sc && j < tid)) ? 1 : 0;
        }
        const int y = y_s[tid];
        bool ok = (draft_s[tid] == y) || (rank < p.n_loose);
        if (!ok) {
            const int lo = max(0, tid - p.window), hi = min(gamma - 1, tid + p.window);
            for (int k = lo; k <= hi; ++k) ok = ok || (draft_s[k] == y);
        }
        acc_s[tid] = ok ? 1 : 0;
        const size_t rid = (size_t)b * gamma + tid;
        if (p.target) p.target[rid] = y;
        if (p.accepted) p.accepted[rid] = ok ? 1 : 0;
    }
    __syncthreads();
    __shared__ int tau_s;
    if (tid == 0) {
        int tau = 0;
        while (tau < gamma && acc_s[tau]) ++tau;
        p.accept_len[b] = tau;
        tau_s = tau;
        p.counters[b] = 0;                         // ready for the next call
        // emit step: how many tokens go back to the decoding loop and how long the
        // cache is afterwards (the accepted draft slots stay, the rest is dropped)
        if (p.n_emitted) p.n_emitted[b] = min(tau + 1, gamma);
        if (p.new_kv_len && p.kv_len) p.new_kv_len[b] = p.kv_len[b] - gamma + tau;
    }
    if (p.emitted) {
        __syncthreads();
        // accepted draft tokens as they are, then the target's own token at the
        // rejected position, then -1
        if (tid < gamma) {
            const int tau = tau_s;
            const int tok = tid < tau ? draft_s[tid] : (tid == tau ? y_s[tid] : -1);
            p.emitted[(size_t)b * gamma + tid] = tok;
        }
    }
}

// Draft-token trees: one accepted length per branch goes in, the branch with the
// longest one (the first among equals) comes out.  One thread per sequence.
__global__ void select_branch_kernel(const int32_t *accept_len, int B, int R, int32_t *best_branch,
                                     int32_t *best_len)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    int best = 0, len = accept_len[(size_t)b * R];
    for (int r = 1; r < R; ++r) {
        const int l = accept_len[(size_t)b * R + r];
        if (l > len) { len = l; best = r; }
    }
    best_branch[b] = best;
    best_len[b] = len;
}

}  // namespace

cudaError_t launch_select_branch(const int32_t *accept_len, int B, int R, int32_t *best_branch,
                                 int32_t *best_len, cudaStream_t stream, int *launches)
{
    select_branch_kernel<<<(B + 127) / 128, 128, 0, stream>>>(accept_len, B, R, best_branch, best_len);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_loose_accept(const AcceptParams &p, cudaStream_t stream, int *launches)
{
    dim3 grid(p.n_vsplit, p.gamma, p.B);
    loose_accept_kernel<<<grid, kThreads, 0, stream>>>(p);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace lvspec
