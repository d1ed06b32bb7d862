// Stage 1: score table S[c, i] = <q_i, centroid_c> for every query token and every centroid (Definition 1's inner
// product), evaluated exactly in integers:
//     Xq = rint(q * 2^22), Xc = rint(c * 2^22),  T = sum_d Xq[d] * Xc[d],  S = floor((T + 2^19) / 2^20)   (Q.24).
// Each 23-bit integer is split into three balanced base-256 digits, so T = sum_{a,b} 256^(a+b) P_ab with the nine
// digit-plane products P_ab = sum_d qa[d] * cb[d] being int8 x int8 -> int32 contractions (exact in any order).
// Products of equal weight a+b share an accumulator (five accumulators, each |.| < 2^23); the epilogue recombines
// them with shifts in int64 and rounds.
//
// This file: digit split of the queries + the contraction on CUDA cores with dp4a (exact int32 accumulation).
#include "common.cuh"

namespace chimera {

constexpr int G1_CT = 64;        // centroids per block
constexpr int G1_THREADS = 256;

// grid (ceil(K / G1_CT), B).  smem: query digits transposed [3][D/4][nq] and centroid digits [3][G1_CT][D/4].
__global__ void __launch_bounds__(G1_THREADS)
score_table_dp4a(const int8_t *__restrict__ qdig, const int8_t *__restrict__ cdig, int64_t K, int D, int nq,
                 int64_t q_rows_total, int32_t *__restrict__ table)
{
    extern __shared__ int smem_i[];
    const int G = D >> 2;                       // 4-dim groups
    int *qs = smem_i;                           // [3][G][nq]
    int *cs = smem_i + 3 * G * nq;              // [3][G1_CT][G]
    const int b = blockIdx.y;
    const int64_t c0 = (int64_t)blockIdx.x * G1_CT;
    const int n_c = (int)((K - c0) < G1_CT ? (K - c0) : G1_CT);

    const int *q32 = reinterpret_cast<const int *>(qdig);
    const int *c32 = reinterpret_cast<const int *>(cdig);
    for (int e = threadIdx.x; e < 3 * nq * G; e += G1_THREADS) {
        int p = e / (nq * G), r = e % (nq * G), i = r / G, g = r % G;
        qs[(p * G + g) * nq + i] = q32[((int64_t)p * q_rows_total + (int64_t)b * nq + i) * G + g];
    }
    for (int e = threadIdx.x; e < 3 * n_c * G; e += G1_THREADS) {
        int p = e / (n_c * G), r = e % (n_c * G), c = r / G, g = r % G;
        cs[(p * G1_CT + c) * G + g] = c32[((int64_t)p * K + c0 + c) * G + g];
    }
    __syncthreads();

    int32_t *out = table + ((int64_t)b * K + c0) * nq;
    for (int o = threadIdx.x; o < n_c * nq; o += G1_THREADS) {
        const int c = o / nq, i = o % nq;
        int a0 = 0, a1 = 0, a2 = 0, a3 = 0, a4 = 0;
        for (int g = 0; g < G; ++g) {
            int q0 = qs[(0 * G + g) * nq + i], q1 = qs[(1 * G + g) * nq + i], q2 = qs[(2 * G + g) * nq + i];
            int x0 = cs[(0 * G1_CT + c) * G + g], x1 = cs[(1 * G1_CT + c) * G + g], x2 = cs[(2 * G1_CT + c) * G + g];
            a0 = __dp4a(q0, x0, a0);
            a1 = __dp4a(q0, x1, a1);
            a1 = __dp4a(q1, x0, a1);
            a2 = __dp4a(q0, x2, a2);
            a2 = __dp4a(q1, x1, a2);
            a2 = __dp4a(q2, x0, a2);
            a3 = __dp4a(q1, x2, a3);
            a3 = __dp4a(q2, x1, a3);
            a4 = __dp4a(q2, x2, a4);
        }
        long long T = (long long)a0 + (long long)a1 * 256LL + (long long)a2 * 65536LL + (long long)a3 * 16777216LL +
                      (long long)a4 * 4294967296LL;
        out[o] = (int32_t)((T + (1LL << 19)) >> 20);
    }
}

int launch_score_table(const Index &ix, const Params &p, const float *queries, int8_t *qdig, int32_t *table,
                       uint32_t *status, cudaStream_t st)
{
    const int64_t rows = (int64_t)p.B * p.nq;
    int rc = launch_digits(queries, rows, ix.D, qdig, status, st);
    if (rc) return rc;
    count_launch(SLOT_G1);
    const int G = ix.D / 4;
    size_t smem = sizeof(int) * (size_t)(3 * G * p.nq + 3 * G1_CT * G);
    if (smem > 48 * 1024)
        CHIMERA_CUDA(cudaFuncSetAttribute(score_table_dp4a, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    dim3 grid((unsigned)((ix.K + G1_CT - 1) / G1_CT), (unsigned)p.B);
    score_table_dp4a<<<grid, G1_THREADS, smem, st>>>(qdig, ix.cdig, ix.K, ix.D, p.nq, rows, table);
    CHIMERA_CUDA(cudaGetLastError());
    count_launch(SLOT_G1);
    return CHIMERA_OK;
}

}  // namespace chimera
