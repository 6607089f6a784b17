// Instruction costs the kernels of this library are designed around, measured in isolation:
// back-to-back tcgen05.mma of the shapes the attention kernel issues (one and two issuing
// warps), and the per-warp-instruction throughput of ex2, the bf16 / E4M3 conversions, fma
// and the warp maximum (redux.sync against a shuffle butterfly).  One CTA, a few
// microseconds; every wait is bounded.  Built and run by
//     python -m paper_2604_05650_b200.instr_cost
#include <cstdio>
#include <cstdlib>
#include <cuda_runtime.h>
#include <stdint.h>

#include "sm100_ptx.cuh"
using namespace lvspec::ptx;

// ------------------------------------------------------------------ tcgen05.mma
struct Case {
    int fp8, M, N, a_mn, b_mn, swz;   // swz: 0 none, 2 = 128B
    int n_issue;                      // MMAs per issuer
    int two;                          // second issuer concurrently (same shape, other TMEM columns)
    int vary;                         // descriptor start address varies per MMA
};

__global__ void __launch_bounds__(128, 1) mma_cost_kernel(Case c, long long *out)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *g = smem_raw + (base - smem_u32(smem_raw));
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // zero 128 KB of operand space
    for (int i = tid * 16; i < 128 * 1024; i += 128 * 16) *reinterpret_cast<uint4 *>(g + i) = make_uint4(0, 0, 0, 0);
    const uint32_t bars = base + 128 * 1024;
    volatile uint32_t *slot = reinterpret_cast<volatile uint32_t *>(g + 128 * 1024 + 64);
    if (tid == 0) {
        mbar_init(bars, 1);
        mbar_init(bars + 8, 1);
        mbar_fence_init();
    }
    fence_proxy_async_smem();
    if (warp == 1) {
        tmem_alloc(base + 128 * 1024 + 64, 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tm = *slot;
    const uint32_t idesc = c.fp8 ? make_idesc_e4m3(c.M, c.N, c.a_mn, c.b_mn) : make_idesc_bf16(c.M, c.N, c.a_mn, c.b_mn);
    if ((warp == 0 || (warp == 2 && c.two)) ) {
        const int w = warp == 0 ? 0 : 1;
        const uint64_t ad0 = (!c.a_mn && c.swz == 0) ? make_smem_desc(base + w * 65536, 1024, 128, 0)
                                                    : make_smem_desc(base + w * 65536, c.a_mn ? 16384 : 16, 1024, c.swz);
        const uint64_t bd0 = make_smem_desc(base + w * 65536 + 32768, c.b_mn ? 128 : 16, c.b_mn ? 2048 : 1024, c.b_mn ? 0 : c.swz);
        const uint32_t d = tm + w * 256;
        __syncwarp();
        long long t0 = clock64();
        if (elect_one()) {
            for (int i = 0; i < c.n_issue; ++i) {
                const uint64_t off = c.vary ? (uint64_t)((i & 7) * 2) : 0;
                if (c.fp8) mma_f8_ss(d, ad0 + off, bd0 + off, idesc, i > 0);
                else mma_f16_ss(d, ad0 + off, bd0 + off, idesc, i > 0);
            }
            mma_commit(bars + 8 * w);
        }
        __syncwarp();
        long long t1 = clock64();
        for (int spin = 0; spin < (1 << 22) && !mbar_try_wait(bars + 8 * w, 0); ++spin) {}
        long long t2 = clock64();
        if (lane == 0 && blockIdx.x == 0) {
            out[w * 2 + 0] = t1 - t0;
            out[w * 2 + 1] = t2 - t0;
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 1) tmem_dealloc(tm, 512);
}

// ------------------------------------------------------- plain and special-function ops
__device__ __forceinline__ float ex2v(float x) { float y; asm volatile("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }
__device__ __forceinline__ uint32_t pk16(float lo, float hi) { uint32_t r; asm volatile("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo)); return r; }
__device__ __forceinline__ uint32_t pk8(float lo, float hi) { uint16_t r; asm volatile("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo)); return r; }
__device__ __forceinline__ float rmax(float x) { float r; asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(x)); return r; }
// kOp: 0 ex2, 1 cvt to bf16x2, 2 cvt to e4m3x2, 3 fma, 4 redux.sync.max.f32, 5 shuffle butterfly maximum
template <int kOp>
__global__ void op_cost_kernel(float *out, long long *cyc, int iters)
{
    float a[8];
    for (int j = 0; j < 8; ++j) a[j] = threadIdx.x * 0.001f + j;
    uint32_t acc = 0;
    __syncthreads();
    const long long t0 = clock64();
    for (int i = 0; i < iters; ++i) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            if (kOp == 0) a[j] = ex2v(a[j]);
            else if (kOp == 1) acc ^= pk16(a[j], a[(j + 1) & 7] + i);
            else if (kOp == 2) acc ^= pk8(a[j], a[(j + 1) & 7] + i);
            else if (kOp == 3) a[j] = fmaf(a[j], 1.0001f, 0.5f);
            else if (kOp == 4) a[j] = rmax(a[j] + i);
            else {
                float v = a[j] + i;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
                a[j] = v;
            }
        }
    }
    const long long t1 = clock64();
    float s = 0;
    for (int j = 0; j < 8; ++j) s += a[j];
    out[blockIdx.x * blockDim.x + threadIdx.x] = s + acc;
    if (threadIdx.x == 0) cyc[blockIdx.x] = t1 - t0;
}

template <int kOp>
static void run_op(const char *name, float *o, long long *c)
{
    const int iters = 2048;
    for (int threads : {128, 384}) {
        long long h = 0;
        for (int rep = 0; rep < 2; ++rep) {
            op_cost_kernel<kOp><<<1, threads>>>(o, c, iters);
            if (cudaDeviceSynchronize() != cudaSuccess) { printf("error in %s\n", name); exit(1); }
        }
        cudaMemcpy(&h, c, 8, cudaMemcpyDeviceToHost);
        printf("%-22s %d warp(s) per scheduler: %.2f cycles per warp instruction and scheduler\n", name, threads / 128,
               (double)h / (iters * 8.0 * (threads / 128)));
    }
}

int main()
{
    long long *d_out, h[4];
    cudaMalloc(&d_out, 32);
    const size_t smem = 128 * 1024 + 1024 + 256;
    cudaFuncSetAttribute(mma_cost_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    const int n = 256;
    Case cases[] = {
        // fp8 M N a_mn b_mn swz n two vary
        {0, 128, 48, 0, 0, 2, n, 0, 1},     // QK bf16
        {0, 128, 80, 0, 0, 2, n, 0, 1},
        {0, 128, 128, 0, 0, 2, n, 0, 1},
        {0, 128, 256, 0, 0, 2, n, 0, 1},
        {0, 128, 48, 1, 1, 2, n, 0, 1},     // PV bf16
        {0, 128, 80, 1, 1, 2, n, 0, 1},
        {0, 64, 48, 0, 1, 0, n, 0, 1},      // sum bf16
        {0, 64, 80, 0, 1, 0, n, 0, 1},
        {0, 128, 48, 0, 0, 2, n, 1, 1},     // two issuers
        {0, 128, 48, 1, 1, 2, n, 1, 1},
        {1, 128, 48, 0, 0, 2, n, 0, 1},     // QK fp8
        {1, 128, 80, 0, 0, 2, n, 0, 1},
        {1, 128, 128, 0, 0, 2, n, 0, 1},
        {1, 128, 256, 0, 0, 2, n, 0, 1},
        {1, 128, 96, 1, 1, 2, n, 0, 1},     // PV fp8
        {1, 128, 160, 1, 1, 2, n, 0, 1},
        {1, 64, 96, 0, 1, 0, n, 0, 1},      // sum fp8
        {1, 64, 160, 0, 1, 0, n, 0, 1},
        {1, 128, 48, 0, 0, 2, n, 1, 1},
        {1, 128, 96, 1, 1, 2, n, 1, 1},
        {0, 128, 48, 0, 0, 2, n, 0, 0},     // same descriptor every time
        {0, 128, 16, 0, 0, 2, n, 0, 1},
        {0, 128, 32, 0, 0, 2, n, 0, 1},
        {0, 128, 64, 0, 0, 2, n, 0, 1},
        {0, 64, 64, 0, 0, 2, n, 0, 1},
        {0, 128, 144, 0, 1, 2, n, 0, 1},    // PV not transposed: A = P K-major, B = V MN-major, N = 144
        {0, 64, 144, 0, 1, 2, n, 0, 1},
    };
    for (const Case &c : cases) {
        for (int rep = 0; rep < 2; ++rep) {
            cudaMemset(d_out, 0, 32);
            mma_cost_kernel<<<1, 128, smem>>>(c, d_out);
            cudaError_t e = cudaDeviceSynchronize();
            if (e != cudaSuccess) {
                printf("error %s\n", cudaGetErrorString(e));
                return 1;
            }
        }
        cudaMemcpy(h, d_out, 32, cudaMemcpyDeviceToHost);
        printf("fp8 %d M %3d N %3d a_mn %d b_mn %d swz %d two %d vary %d | issue %.1f total %.1f cycles/MMA", c.fp8, c.M, c.N,
               c.a_mn, c.b_mn, c.swz, c.two, c.vary, (double)h[0] / c.n_issue, (double)h[1] / c.n_issue);
        if (c.two) printf(" | second: issue %.1f total %.1f", (double)h[2] / c.n_issue, (double)h[3] / c.n_issue);
        printf("\n");
    }
    float *o;
    long long *c;
    cudaMalloc(&o, 4 * 1024 * 16);
    cudaMalloc(&c, 64);
    run_op<0>("ex2.approx.f32", o, c);
    run_op<1>("cvt.rn.bf16x2.f32", o, c);
    run_op<2>("cvt e4m3x2.f32", o, c);
    run_op<3>("fma.rn.f32", o, c);
    run_op<4>("redux.sync.max.f32", o, c);
    run_op<5>("shuffle maximum", o, c);
    return 0;
}
