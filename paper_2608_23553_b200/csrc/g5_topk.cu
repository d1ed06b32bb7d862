// Stage 5: batched top-k (Definition 2, Eq. 1): per query the k survivors with the largest stage-4 score, best
// first, ties towards the smaller document id; missing entries are (-1, -inf).
//
// One block per query.  Each (score, id) becomes a 64-bit key whose unsigned order is (score desc, id asc); the keys
// are sorted descending with a bitonic network in shared memory (n_prune <= 16384 keys = 128 KB) and the first k are
// decoded back.
#include <math.h>

#include "common.cuh"

namespace chimera {

constexpr int TOPK_THREADS = 1024;

__device__ __forceinline__ uint32_t float_order(float f)
{
    uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float float_unorder(uint32_t o)
{
    uint32_t u = (o & 0x80000000u) ? (o & 0x7fffffffu) : ~o;
    return __uint_as_float(u);
}

__global__ void __launch_bounds__(TOPK_THREADS)
topk_kernel(const int32_t *__restrict__ pruned, const float *__restrict__ score4, int n_prune, int n_pow2, int k,
            int32_t *__restrict__ out_ids, float *__restrict__ out_scores)
{
    extern __shared__ unsigned long long keys[];
    const int b = blockIdx.x;
    for (int j = threadIdx.x; j < n_pow2; j += TOPK_THREADS) {
        unsigned long long key = 0ull;
        if (j < n_prune) {
            int32_t id = pruned[(int64_t)b * n_prune + j];
            if (id >= 0)
                key = ((unsigned long long)float_order(score4[(int64_t)b * n_prune + j]) << 32) |
                      (uint32_t)(0xFFFFFFFFu - (uint32_t)id);
        }
        keys[j] = key;
    }
    __syncthreads();
    for (int size = 2; size <= n_pow2; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            for (int t = threadIdx.x; t < (n_pow2 >> 1); t += TOPK_THREADS) {
                int lo = 2 * t - (t & (stride - 1));      // index with the stride bit clear
                int hi = lo + stride;
                bool descending = (lo & size) == 0;
                unsigned long long a = keys[lo], c = keys[hi];
                if ((a < c) == descending) { keys[lo] = c; keys[hi] = a; }
            }
            __syncthreads();
        }
    }
    for (int r = threadIdx.x; r < k; r += TOPK_THREADS) {
        unsigned long long key = r < n_pow2 ? keys[r] : 0ull;
        if (key == 0ull) {
            out_ids[(int64_t)b * k + r] = -1;
            out_scores[(int64_t)b * k + r] = -INFINITY;
        } else {
            out_ids[(int64_t)b * k + r] = (int32_t)(0xFFFFFFFFu - (uint32_t)key);
            out_scores[(int64_t)b * k + r] = float_unorder((uint32_t)(key >> 32));
        }
    }
}

int launch_topk(const Index &ix, const Params &p, const int32_t *pruned, const float *score4, int32_t *out_ids,
                float *out_scores, cudaStream_t st)
{
    (void)ix;
    int n_pow2 = 2;
    while (n_pow2 < p.n_prune) n_pow2 <<= 1;
    const size_t smem = sizeof(unsigned long long) * (size_t)n_pow2;
    if (smem > 48 * 1024)
        CHIMERA_CUDA(cudaFuncSetAttribute(topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    topk_kernel<<<(unsigned)p.B, TOPK_THREADS, smem, st>>>(pruned, score4, p.n_prune, n_pow2, p.k, out_ids,
                                                           out_scores);
    CHIMERA_CUDA(cudaGetLastError());
    count_launch(SLOT_TOPK);
    return CHIMERA_OK;
}

}  // namespace chimera
