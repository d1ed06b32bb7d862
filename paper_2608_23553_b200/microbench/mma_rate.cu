// Microbenchmark behind the shape of the stage-1 MMA schedule: how long one tcgen05.mma kind::i8 instruction
// (M = 128, K = 32) takes as a function of N, with the A operand in shared memory or in tensor memory.  One CTA of one
// issuing thread per SM, 20,000 back-to-back instructions on zero operands, every wait bounded.  Build and run:
//   nvcc -gencode arch=compute_100a,code=sm_100a -O3 -std=c++17 -I paper_2608_23553_b200/csrc -I include \
//        -o mma_rate paper_2608_23553_b200/microbench/mma_rate.cu && ./mma_rate
// It is not part of the library.
#include <cstdio>
#include <cstdint>
#include <cuda_runtime.h>
#include "umma.cuh"
using namespace chimera;

__device__ __forceinline__ void mma_ts(uint32_t d, uint32_t a, uint64_t b, uint32_t idesc, uint32_t acc)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, p;\n\t}"
                 ::"r"(d), "r"(a), "l"(b), "r"(idesc), "r"(acc) : "memory");
}

template <int N, bool TS>
__global__ void __launch_bounds__(128) rate_kernel(int iters, long long *out, int *err)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint32_t s_tmem;
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sA = base, sB = base + 16384, bar = sB + 256 * 128;
    const int tid = threadIdx.x, warp = tid >> 5;
    for (uint32_t e = tid; e < (16384 + 256 * 128) / 16; e += 128)
        asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(base + e * 16), "r"(0u) : "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    if (tid == 0) { mbar_init(bar, 1); asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
    if (warp == 0) { __syncwarp(); tmem_alloc(&s_tmem, 512); }
    tc_fence_before(); __syncthreads(); tc_fence_after();
    const uint32_t tmem = s_tmem;
    constexpr uint32_t IDESC = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
    long long t_issue = 0, t_done = 0;
    if (tid == 0) {
        const uint64_t da = umma_desc(sA), db = umma_desc(sB);
        const long long t0 = clock64();
        for (int i = 0; i < iters; i += 4) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                if (TS) mma_ts(tmem, tmem + 256 + 8 * k, db + 2 * k, IDESC, 1u);
                else umma_i8(tmem, da + 2 * k, db + 2 * k, IDESC, 1u);
            }
        }
        umma_commit(bar);
        t_issue = clock64() - t0;
        const bool ok = mbar_wait(bar, 0, 2000000000LL);
        t_done = clock64() - t0;
        if (!ok) *err = 1;
        if (blockIdx.x == 0) { out[0] = t_issue; out[1] = t_done; }
    }
    tc_fence_before(); __syncthreads();
    if (warp == 0) { tc_fence_after(); tmem_dealloc(tmem, 512); }
}

template <int N, bool TS> void run(int iters, long long *d_out, int *d_err)
{
    const int smem = 16384 + 256 * 128 + 1024 + 64;
    cudaFuncSetAttribute(rate_kernel<N, TS>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    cudaEvent_t e0, e1; cudaEventCreate(&e0); cudaEventCreate(&e1);
    rate_kernel<N, TS><<<148, 128, smem>>>(iters, d_out, d_err);       // warm-up
    cudaEventRecord(e0);
    rate_kernel<N, TS><<<148, 128, smem>>>(iters, d_out, d_err);
    cudaEventRecord(e1);
    cudaError_t rc = cudaDeviceSynchronize();
    float ms = 0; cudaEventElapsedTime(&ms, e0, e1);
    long long h[2]; int herr = 0;
    cudaMemcpy(h, d_out, sizeof(h), cudaMemcpyDeviceToHost); cudaMemcpy(&herr, d_err, sizeof(int), cudaMemcpyDeviceToHost);
    const double ops = 2.0 * 128 * N * 32 * (double)iters * 148;
    printf("N=%3d %s: %s err=%d  issue %.1f clk/MMA, done %.1f clk/MMA (%.2f clk/column), %.3f ms, %.0f TOP/s\n", N,
           TS ? "A in TMEM" : "A in smem", cudaGetErrorString(rc), herr, (double)h[0] / iters, (double)h[1] / iters,
           (double)h[1] / iters / N, ms, ops / (ms * 1e-3) / 1e12);
}

int main()
{
    long long *d_out; int *d_err;
    cudaMalloc(&d_out, 16); cudaMalloc(&d_err, 4); cudaMemset(d_err, 0, 4);
    const int iters = 20000;
    run<32, false>(iters, d_out, d_err);  run<32, true>(iters, d_out, d_err);
    run<96, false>(iters, d_out, d_err);  run<96, true>(iters, d_out, d_err);
    run<128, true>(iters, d_out, d_err);  run<192, true>(iters, d_out, d_err);
    run<256, false>(iters, d_out, d_err); run<256, true>(iters, d_out, d_err);
    return 0;
}
