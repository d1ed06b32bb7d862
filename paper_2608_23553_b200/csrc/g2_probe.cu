// Stage 2a: for each query token the nprobe centroids with the largest score (Sec. 3.2 step 1: the top-n_probe
// centroids of a query token), ordered by (score descending, centroid id ascending).
//
// The table is centroid-major [K][nq], so a warp reads one 128-byte row per step with lane = query token.  Every
// thread keeps a sorted list of its best P keys in shared memory (column layout list[j][thread], conflict-free); a
// key is a 64-bit integer whose order is (score desc, id asc).  Pass 1 turns slices of the table into partial lists,
// pass 2 folds the partial lists of a query into the final P per token.
#include "common.cuh"

namespace chimera {

constexpr int PROBE_THREADS = PROBE_WARPS * 32;

__device__ __forceinline__ void list_insert(unsigned long long *list, int P, unsigned long long key)
{
    // list[j * PROBE_THREADS] is entry j of this thread's list, descending.
    if (key <= list[(P - 1) * PROBE_THREADS]) return;
    int j = P - 1;
    while (j > 0) {
        unsigned long long up = list[(j - 1) * PROBE_THREADS];
        if (up >= key) break;
        list[j * PROBE_THREADS] = up;
        --j;
    }
    list[j * PROBE_THREADS] = key;
}

// grid (probe_blocks, B, ceil(nq / 32)).  part: [B][n_part][P][nq], n_part = probe_blocks * PROBE_WARPS.
__global__ void __launch_bounds__(PROBE_THREADS)
probe_partial(const int32_t *__restrict__ table, int64_t K, int nq, int P, int rows_per_block, int n_part,
              unsigned long long *__restrict__ part)
{
    extern __shared__ unsigned long long lists[];    // [P][PROBE_THREADS]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int col = blockIdx.z * 32 + lane;
    const int b = blockIdx.y;
    unsigned long long *mine = lists + threadIdx.x;
    for (int j = 0; j < P; ++j) mine[j * PROBE_THREADS] = 0ull;
    const int64_t r0 = (int64_t)blockIdx.x * rows_per_block;
    int64_t r1 = r0 + rows_per_block;
    if (r1 > K) r1 = K;
    if (col < nq) {
        const int32_t *tb = table + (int64_t)b * K * nq + col;
        int64_t r = r0 + warp;
        // four independent loads in flight per thread
        for (; r + 3 * PROBE_WARPS < r1; r += 4 * PROBE_WARPS) {
            int32_t s0 = tb[r * nq], s1 = tb[(r + PROBE_WARPS) * nq], s2 = tb[(r + 2 * PROBE_WARPS) * nq],
                    s3 = tb[(r + 3 * PROBE_WARPS) * nq];
            list_insert(mine, P, key_int(s0, (int32_t)r));
            list_insert(mine, P, key_int(s1, (int32_t)(r + PROBE_WARPS)));
            list_insert(mine, P, key_int(s2, (int32_t)(r + 2 * PROBE_WARPS)));
            list_insert(mine, P, key_int(s3, (int32_t)(r + 3 * PROBE_WARPS)));
        }
        for (; r < r1; r += PROBE_WARPS) list_insert(mine, P, key_int(tb[r * nq], (int32_t)r));
        unsigned long long *dst = part + (((int64_t)b * n_part + (int64_t)blockIdx.x * PROBE_WARPS + warp) * P) * nq + col;
        for (int j = 0; j < P; ++j) dst[(int64_t)j * nq] = mine[j * PROBE_THREADS];
    }
}

// grid (1, B, ceil(nq / 32)).  Folds n_part sorted lists per column into one; writes probes[b][col][0..P).
__global__ void __launch_bounds__(PROBE_THREADS)
probe_final(const unsigned long long *__restrict__ part, int nq, int P, int n_part, int32_t *__restrict__ probes)
{
    extern __shared__ unsigned long long lists[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int col = blockIdx.z * 32 + lane;
    const int b = blockIdx.y;
    unsigned long long *mine = lists + threadIdx.x;
    for (int j = 0; j < P; ++j) mine[j * PROBE_THREADS] = 0ull;
    if (col < nq) {
        for (int l = warp; l < n_part; l += PROBE_WARPS) {
            const unsigned long long *src = part + (((int64_t)b * n_part + l) * P) * nq + col;
            for (int j = 0; j < P; ++j) {
                unsigned long long key = src[(int64_t)j * nq];
                if (key <= mine[(P - 1) * PROBE_THREADS]) break;      // source list is descending
                list_insert(mine, P, key);
            }
        }
    }
    __syncthreads();
    if (warp == 0 && col < nq) {
        for (int w = 1; w < PROBE_WARPS; ++w) {
            const unsigned long long *src = lists + w * 32 + lane;
            for (int j = 0; j < P; ++j) {
                unsigned long long key = src[j * PROBE_THREADS];
                if (key <= mine[(P - 1) * PROBE_THREADS]) break;
                list_insert(mine, P, key);
            }
        }
        int32_t *dst = probes + ((int64_t)b * nq + col) * P;
        for (int j = 0; j < P; ++j) dst[j] = key_id(mine[j * PROBE_THREADS]);
    }
}

int launch_probes(const Index &ix, const Params &p, const Layout &L, const int32_t *table, unsigned long long *part,
                  int32_t *probes, cudaStream_t st)
{
    const size_t smem = sizeof(unsigned long long) * (size_t)p.P * PROBE_THREADS;
    if (smem > 48 * 1024) {
        CHIMERA_CUDA(cudaFuncSetAttribute(probe_partial, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        CHIMERA_CUDA(cudaFuncSetAttribute(probe_final, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    }
    const int rows_per_block = (int)((ix.K + L.probe_blocks - 1) / L.probe_blocks);
    const unsigned col_groups = (unsigned)((p.nq + 31) / 32);
    dim3 g1((unsigned)L.probe_blocks, (unsigned)p.B, col_groups);
    probe_partial<<<g1, PROBE_THREADS, smem, st>>>(table, ix.K, p.nq, p.P, rows_per_block, L.n_part, part);
    CHIMERA_CUDA(cudaGetLastError());
    dim3 g2(1, (unsigned)p.B, col_groups);
    probe_final<<<g2, PROBE_THREADS, smem, st>>>(part, p.nq, p.P, L.n_part, probes);
    CHIMERA_CUDA(cudaGetLastError());
    count_launch(SLOT_PROBE, 2);
    return CHIMERA_OK;
}

}  // namespace chimera
