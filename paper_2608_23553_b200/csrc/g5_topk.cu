// Stage 5: batched top-k (Definition 2, Eq. 1): per query the k survivors with the largest stage-4 score, best
// first, ties towards the smaller document id; missing entries are (-1, -inf).
//
// One block per query.  Each (score, id) becomes a 64-bit key whose unsigned order is (score desc, id asc); the keys
// are sorted descending with a bitonic network in shared memory (n_prune <= 16384 keys = 128 KB) and the first k are
// decoded back.  For k <= 16 the keys stay in registers instead and the block extracts its maximum k times (two
// barriers per result instead of the network's log^2 stages), and for k <= 128 over at most 4096 entries the warps sort
// 128-key runs in registers and merge them pairwise, keeping the better half each time: the shorter chains matter
// when one query is served at a time.
#include <math.h>

#include "common.cuh"

namespace chimera {

constexpr int TOPK_THREADS = 1024;

__device__ __forceinline__ uint32_t float_order(float f)
{
    uint32_t u = __float_as_uint(f);
    if (u == 0x80000000u) u = 0u;        // -0 and +0 are the same score (the tie goes to the smaller id)
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float float_unorder(uint32_t o)
{
    uint32_t u = (o & 0x80000000u) ? (o & 0x7fffffffu) : ~o;
    return __uint_as_float(u);
}

// Entry j of query b.  A query's entries are one run of n_prune (seg_len = n_prune) or, for the merge of several
// shards' lists laid out [shard][query][seg_len], one run of seg_len per shard, seg_stride apart.
__device__ __forceinline__ int64_t entry_index(int j, int b, int seg_len, long long seg_stride)
{
    return (int64_t)(j / seg_len) * seg_stride + (int64_t)b * seg_len + j % seg_len;
}

__global__ void __launch_bounds__(TOPK_THREADS)
topk_kernel(const int32_t *__restrict__ pruned, const float *__restrict__ score4, int n_prune, int n_pow2, int k,
            int seg_len, long long seg_stride, int32_t *__restrict__ out_ids, float *__restrict__ out_scores)
{
    extern __shared__ unsigned long long keys[];
    const int b = blockIdx.x;
    for (int j = threadIdx.x; j < n_pow2; j += TOPK_THREADS) {
        unsigned long long key = 0ull;
        if (j < n_prune) {
            const int64_t at = entry_index(j, b, seg_len, seg_stride);
            int32_t id = pruned[at];
            if (id >= 0)
                key = ((unsigned long long)float_order(score4[at]) << 32) | (uint32_t)(0xFFFFFFFFu - (uint32_t)id);
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

template <int KPT>      // keys per thread: n_prune <= KPT * TOPK_THREADS
__global__ void __launch_bounds__(TOPK_THREADS)
topk_small_kernel(const int32_t *__restrict__ pruned, const float *__restrict__ score4, int n_prune, int k,
                  int seg_len, long long seg_stride, int32_t *__restrict__ out_ids, float *__restrict__ out_scores)
{
    __shared__ unsigned long long warp_max[32];
    __shared__ unsigned long long s_win;
    const int b = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned long long keys[KPT];
#pragma unroll
    for (int e = 0; e < KPT; ++e) {
        const int j = e * TOPK_THREADS + threadIdx.x;
        keys[e] = 0ull;
        if (j < n_prune) {
            const int64_t at = entry_index(j, b, seg_len, seg_stride);
            const int32_t id = pruned[at];
            if (id >= 0)
                keys[e] = ((unsigned long long)float_order(score4[at]) << 32) | (uint32_t)(0xFFFFFFFFu - (uint32_t)id);
        }
    }
    for (int r = 0; r < k; ++r) {
        unsigned long long m = keys[0];
#pragma unroll
        for (int e = 1; e < KPT; ++e) m = keys[e] > m ? keys[e] : m;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const unsigned long long t = __shfl_xor_sync(0xffffffffu, m, o);
            m = t > m ? t : m;
        }
        if (lane == 0) warp_max[warp] = m;
        __syncthreads();
        if (warp == 0) {
            unsigned long long v = warp_max[lane];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const unsigned long long t = __shfl_xor_sync(0xffffffffu, v, o);
                v = t > v ? t : v;
            }
            if (lane == 0) {
                s_win = v;
                out_ids[(int64_t)b * k + r] = v ? (int32_t)(0xFFFFFFFFu - (uint32_t)v) : -1;
                out_scores[(int64_t)b * k + r] = v ? float_unorder((uint32_t)(v >> 32)) : -INFINITY;
            }
        }
        __syncthreads();
        const unsigned long long win = s_win;       // keys are distinct (the id is part of the key): one owner
#pragma unroll
        for (int e = 0; e < KPT; ++e)
            if (keys[e] == win) keys[e] = 0ull;
    }
}

// 16 < k <= 128 and at most 4096 entries: the full network's ~80 block barriers are what a single query waits for, so
// here every warp sorts its own 128 keys in registers (element e * 32 + lane in register e; strides below 32 are
// shuffles, 32 and 64 are register pairs), and the 32 sorted runs are then merged pairwise in five rounds through
// shared memory, each merge keeping only the 128 best of its 256 keys: max(A[i], B[127 - i]) of two descending runs is
// a bitonic sequence holding exactly those, and one bitonic merge sorts it again.  Six block barriers in all.
constexpr int RUN = 128;                 // keys per warp and per run

__device__ __forceinline__ unsigned long long shfl_xor_u64(unsigned long long v, int o)
{
    return __shfl_xor_sync(0xffffffffu, v, o);
}
// one compare-exchange stage with partner index i ^ stride over the warp's 128 keys; desc[e] = the direction of the
// block that element e * 32 + lane lies in
__device__ __forceinline__ void run_stage(unsigned long long (&key)[4], int stride, const bool (&desc)[4], int lane)
{
    if (stride < 32) {
        const bool lower = (lane & stride) == 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const unsigned long long other = shfl_xor_u64(key[e], stride);
            const bool take_max = lower == desc[e];
            const unsigned long long hi = key[e] > other ? key[e] : other, lo = key[e] > other ? other : key[e];
            key[e] = take_max ? hi : lo;
        }
    } else {
        const int d = stride >> 5;       // 1: pairs (0,1), (2,3); 2: pairs (0,2), (1,3)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if ((e & d) == 0) {
                unsigned long long &a = key[e], &b = key[e | d];
                const unsigned long long hi = a > b ? a : b, lo = a > b ? b : a;
                a = desc[e] ? hi : lo;
                b = desc[e] ? lo : hi;
            }
        }
    }
}
// bitonic merge of a bitonic 128-key sequence into descending order
__device__ __forceinline__ void run_merge_desc(unsigned long long (&key)[4], int lane)
{
    const bool desc[4] = {true, true, true, true};
#pragma unroll
    for (int stride = 64; stride > 0; stride >>= 1) run_stage(key, stride, desc, lane);
}

__global__ void __launch_bounds__(TOPK_THREADS)
topk_runs_kernel(const int32_t *__restrict__ pruned, const float *__restrict__ score4, int n_prune, int k, int seg_len,
                 long long seg_stride, int32_t *__restrict__ out_ids, float *__restrict__ out_scores)
{
    extern __shared__ unsigned long long runs[];           // [32][RUN] then [16][RUN]
    unsigned long long *buf0 = runs, *buf1 = runs + 32 * RUN;
    const int b = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned long long key[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const int j = warp * RUN + e * 32 + lane;
        key[e] = 0ull;
        if (j < n_prune) {
            const int64_t at = entry_index(j, b, seg_len, seg_stride);
            const int32_t id = pruned[at];
            if (id >= 0)
                key[e] = ((unsigned long long)float_order(score4[at]) << 32) | (uint32_t)(0xFFFFFFFFu - (uint32_t)id);
        }
    }
    // the warp's 128 keys, descending
#pragma unroll
    for (int size = 2; size <= RUN; size <<= 1) {
        bool desc[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) desc[e] = ((e * 32 + lane) & size) == 0;
#pragma unroll
        for (int stride = size >> 1; stride > 0; stride >>= 1) run_stage(key, stride, desc, lane);
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) buf0[warp * RUN + e * 32 + lane] = key[e];
    __syncthreads();
    unsigned long long *src = buf0, *dst = buf1;
    for (int n_runs = 32; n_runs > 1; n_runs >>= 1) {
        if (warp < (n_runs >> 1)) {
            const unsigned long long *A = src + (2 * warp) * RUN, *B = src + (2 * warp + 1) * RUN;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int i = e * 32 + lane;
                const unsigned long long a = A[i], c = B[RUN - 1 - i];
                key[e] = a > c ? a : c;
            }
            run_merge_desc(key, lane);
#pragma unroll
            for (int e = 0; e < 4; ++e) dst[warp * RUN + e * 32 + lane] = key[e];
        }
        __syncthreads();
        unsigned long long *t = src; src = dst; dst = t;
    }
    for (int r = threadIdx.x; r < k; r += TOPK_THREADS) {
        const unsigned long long v = src[r];
        out_ids[(int64_t)b * k + r] = v ? (int32_t)(0xFFFFFFFFu - (uint32_t)v) : -1;
        out_scores[(int64_t)b * k + r] = v ? float_unorder((uint32_t)(v >> 32)) : -INFINITY;
    }
}

// n entries per query (laid out by entry_index) -> the best k.
static int launch_topk_entries(const int32_t *ids, const float *scores, int B, int n, int k, int seg_len,
                               long long seg_stride, int32_t *out_ids, float *out_scores, cudaStream_t st)
{
    if (k <= 16 && n <= 16 * TOPK_THREADS) {
        if (n <= TOPK_THREADS)
            topk_small_kernel<1><<<(unsigned)B, TOPK_THREADS, 0, st>>>(ids, scores, n, k, seg_len, seg_stride, out_ids,
                                                                       out_scores);
        else if (n <= 4 * TOPK_THREADS)
            topk_small_kernel<4><<<(unsigned)B, TOPK_THREADS, 0, st>>>(ids, scores, n, k, seg_len, seg_stride, out_ids,
                                                                       out_scores);
        else
            topk_small_kernel<16><<<(unsigned)B, TOPK_THREADS, 0, st>>>(ids, scores, n, k, seg_len, seg_stride, out_ids,
                                                                        out_scores);
        CHIMERA_CUDA(cudaGetLastError());
        return CHIMERA_OK;
    }
    if (k <= RUN && n <= 32 * RUN) {
        topk_runs_kernel<<<(unsigned)B, TOPK_THREADS, sizeof(unsigned long long) * 48 * RUN, st>>>(
            ids, scores, n, k, seg_len, seg_stride, out_ids, out_scores);
        CHIMERA_CUDA(cudaGetLastError());
        return CHIMERA_OK;
    }
    int n_pow2 = 2;
    while (n_pow2 < n) n_pow2 <<= 1;
    const size_t smem = sizeof(unsigned long long) * (size_t)n_pow2;
    if (smem > 128 * 1024) return fail(CHIMERA_UNSUPPORTED, "top-k over %d entries per query does not fit shared memory", n);
    if (smem > 48 * 1024)
        CHIMERA_CUDA(cudaFuncSetAttribute(topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    topk_kernel<<<(unsigned)B, TOPK_THREADS, smem, st>>>(ids, scores, n, n_pow2, k, seg_len, seg_stride, out_ids,
                                                         out_scores);
    CHIMERA_CUDA(cudaGetLastError());
    return CHIMERA_OK;
}

int launch_topk(const Index &ix, const Params &p, const int32_t *pruned, const float *score4, int32_t *out_ids,
                float *out_scores, cudaStream_t st)
{
    (void)ix;
    const int rc = launch_topk_entries(pruned, score4, p.B, p.n_prune, p.k, p.n_prune, 0, out_ids, out_scores, st);
    if (rc) return rc;
    count_launch(SLOT_TOPK);
    return CHIMERA_OK;
}

// Final merge of a document-sharded search: all_ids / all_scores are the shards' top-k lists, [world][B][k] (global
// ids, -1 / -inf padded); out = the best k of their union per query, (score desc, id asc).
int launch_shard_merge_topk(const int32_t *all_ids, const float *all_scores, int world, int B, int k, int32_t *out_ids,
                            float *out_scores, cudaStream_t st)
{
    const int rc = launch_topk_entries(all_ids, all_scores, B, world * k, k, k, (long long)B * k, out_ids, out_scores, st);
    if (rc) return rc;
    count_launch(SLOT_TOPK);
    return CHIMERA_OK;
}

}  // namespace chimera
