// Stage 4: residual-decode MaxSim of the surviving documents (Definition 1 on decoded tokens):
//   score(d) = sum_i max_{t in d} <q_i, c_{cid_t} + r^(code_t)>,   r^(u) = lo + (u + 0.5) * delta per dimension.
// By linearity  <q_i, c + r^> = S[cid_t, i] + delta * sum_x q_i[x] u_t[x] + (lo + delta/2) * sum_x q_i[x],
// so the centroid part comes from the stage-1 table (S * 2^-24) and only the code part is contracted here, in fp32.
//
// One block per (surviving document, query).  The query is staged transposed in shared memory ([D][nq], lane = query
// token, conflict-free); each warp takes every 4th token of the document, loads its packed code words once, and every
// lane accumulates the code contraction for its own query token(s).  Maxima are combined across the warps through
// shared memory and summed over query tokens with warp shuffles.
#include <math.h>

#include "common.cuh"

namespace chimera {

constexpr int G4_THREADS = 128;
constexpr int G4_WARPS = G4_THREADS / 32;

template <int NQW, int NBITS>
__global__ void __launch_bounds__(G4_THREADS)
residual_maxsim_kernel(const float *__restrict__ queries, const int32_t *__restrict__ table, int64_t K, int nq, int D,
                       int CB, float delta, float kappa, const int32_t *__restrict__ pruned, int n_prune,
                       const int32_t *__restrict__ cids, const uint8_t *__restrict__ codes,
                       const int64_t *__restrict__ doc_off, float *__restrict__ score4)
{
    extern __shared__ float smem_f[];
    float *qT = smem_f;                        // [D][nq]
    float *wmax = smem_f + D * nq;             // [G4_WARPS][nq]
    const int b = blockIdx.y, j = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int32_t d = pruned[(int64_t)b * n_prune + j];
    if (d < 0) {
        if (threadIdx.x == 0) score4[(int64_t)b * n_prune + j] = -INFINITY;
        return;
    }
    const float *q = queries + (int64_t)b * nq * D;
    for (int e = threadIdx.x; e < nq * D; e += G4_THREADS) {
        int i = e / D, x = e % D;
        qT[x * nq + i] = q[e];
    }
    __syncthreads();

    const int32_t *tb = table + (int64_t)b * K * nq;
    const int64_t t0 = doc_off[d], t1 = doc_off[d + 1];
    const int CW = CB >> 2;                    // 32-bit code words per token
    constexpr int DIMS_PER_WORD = 32 / NBITS;
    constexpr uint32_t MASK = (1u << NBITS) - 1u;
    const uint32_t *cw = reinterpret_cast<const uint32_t *>(codes);

    float best[NQW];
#pragma unroll
    for (int w = 0; w < NQW; ++w) best[w] = -INFINITY;

    for (int64_t t = t0 + warp; t < t1; t += G4_WARPS) {
        const int32_t c = cids[t];
        uint32_t myword = lane < CW ? cw[t * CW + lane] : 0u;
        float acc[NQW];
#pragma unroll
        for (int w = 0; w < NQW; ++w) acc[w] = 0.f;
        for (int wi = 0; wi < CW; ++wi) {
            const uint32_t word = __shfl_sync(0xffffffffu, myword, wi);
            const float *qrow = qT + (wi * DIMS_PER_WORD) * nq;
#pragma unroll
            for (int s = 0; s < DIMS_PER_WORD; ++s) {
                const float u = (float)((word >> (s * NBITS)) & MASK);
#pragma unroll
                for (int w = 0; w < NQW; ++w) {
                    int col = lane + 32 * w;
                    if (col < nq) acc[w] = fmaf(u, qrow[s * nq + col], acc[w]);
                }
            }
        }
#pragma unroll
        for (int w = 0; w < NQW; ++w) {
            int col = lane + 32 * w;
            if (col < nq) {
                float s = (float)tb[(int64_t)c * nq + col] * (1.0f / 16777216.0f) + delta * acc[w];
                best[w] = fmaxf(best[w], s);
            }
        }
    }
#pragma unroll
    for (int w = 0; w < NQW; ++w) {
        int col = lane + 32 * w;
        if (col < nq) wmax[warp * nq + col] = best[w];
    }
    __syncthreads();
    if (warp == 0) {
        float total = 0.f;
#pragma unroll
        for (int w = 0; w < NQW; ++w) {
            int col = lane + 32 * w;
            if (col < nq) {
                float m = wmax[col];
                for (int ww = 1; ww < G4_WARPS; ++ww) m = fmaxf(m, wmax[ww * nq + col]);
                // kappa * sum_x q[x]: the constant part of the residual term for this query token
                float sq = 0.f;
                for (int x = 0; x < D; ++x) sq += qT[x * nq + col];
                total += m + kappa * sq;
            }
        }
        total = warp_sum(total);
        if (lane == 0) score4[(int64_t)b * n_prune + j] = total;
    }
}

int launch_residual_scores(const Index &ix, const Params &p, const float *queries, const int32_t *table,
                           const int32_t *pruned, float *score4, cudaStream_t st)
{
    const float delta = (ix.res_hi - ix.res_lo) / (float)(1 << ix.nbits);
    const float kappa = ix.res_lo + 0.5f * delta;
    const size_t smem = sizeof(float) * ((size_t)ix.D * p.nq + (size_t)G4_WARPS * p.nq);
    dim3 grid((unsigned)p.n_prune, (unsigned)p.B);
    const int nqw = (p.nq + 31) / 32;
#define G4_LAUNCH(NQW_, NB_)                                                                                          \
    do {                                                                                                              \
        if (smem > 48 * 1024)                                                                                         \
            CHIMERA_CUDA(cudaFuncSetAttribute(residual_maxsim_kernel<NQW_, NB_>,                                      \
                                              cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));               \
        residual_maxsim_kernel<NQW_, NB_><<<grid, G4_THREADS, smem, st>>>(queries, table, ix.K, p.nq, ix.D, ix.CB,    \
                                                                          delta, kappa, pruned, p.n_prune, ix.cids,   \
                                                                          ix.codes, ix.doc_off, score4);              \
    } while (0)
    if (ix.nbits == 2) {
        if (nqw == 1) G4_LAUNCH(1, 2);
        else if (nqw == 2) G4_LAUNCH(2, 2);
        else G4_LAUNCH(4, 2);
    } else {
        if (nqw == 1) G4_LAUNCH(1, 1);
        else if (nqw == 2) G4_LAUNCH(2, 1);
        else G4_LAUNCH(4, 1);
    }
#undef G4_LAUNCH
    CHIMERA_CUDA(cudaGetLastError());
    count_launch(SLOT_G4);
    return CHIMERA_OK;
}

}  // namespace chimera
