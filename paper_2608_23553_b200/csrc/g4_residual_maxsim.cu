// Stage 4: residual-decode MaxSim of the surviving documents (Definition 1 on decoded tokens):
//   score(d) = sum_i max_{t in d} <q_i, c_{cid_t} + r^(code_t)>,   r^(u) = lo + (u + 0.5) * delta per dimension.
// By linearity  <q_i, c + r^> = S[cid_t, i] + delta * sum_x q_i[x] u_t[x] + (lo + delta/2) * sum_x q_i[x],
// so the centroid part comes from the stage-1 table (S * 2^-24) and only the code part is contracted here, in fp32
// on the FMA pipe.
//
// A block owns one query and walks over several of its surviving documents.  The query is staged once, transposed
// and zero-padded, in shared memory ([D][NQP]).  Per tile of TT document tokens the packed codes are expanded once to
// fp32 bucket indices in shared memory ([D][TT]); then every thread accumulates a 4-token x 4-query-token register
// tile over the D dimensions (two 16-byte shared loads per 16 FMAs), adds the centroid term from the table and keeps
// a running maximum over tokens.  Maxima are merged across the token rows through shared memory, the per-query-token
// constant is added and the query-token sum is taken with warp shuffles.
#include <math.h>

#include "common.cuh"

namespace chimera {

constexpr int G4_THREADS = 128;

template <int CT, int NBITS>      // CT = 4-column groups (padded q_len NQP = 4 * CT)
__global__ void __launch_bounds__(G4_THREADS)
residual_maxsim_kernel(const float *__restrict__ queries, const int32_t *__restrict__ table, int64_t K, int nq, int D,
                       int CW, float delta, float kappa, const int32_t *__restrict__ pruned, int n_prune,
                       const int32_t *__restrict__ cids, const uint32_t *__restrict__ codes,
                       const int64_t *__restrict__ doc_off, float *__restrict__ score4)
{
    constexpr int NQP = 4 * CT;
    constexpr int TY = G4_THREADS / CT;       // token rows of the thread grid
    constexpr int TT = 4 * TY;                // document tokens per tile
    constexpr int DPW = 32 / NBITS;           // dimensions per 32-bit code word
    constexpr uint32_t MASK = (1u << NBITS) - 1u;

    extern __shared__ __align__(16) float smem_f[];
    float *qT = smem_f;                        // [D][NQP]
    float *U = qT + D * NQP;                   // [D][TT]
    float *red = U + D * TT;                   // [TY][NQP]
    float *sumq = red + TY * NQP;              // [NQP]
    int32_t *tok_cid = reinterpret_cast<int32_t *>(sumq + NQP);   // [TT]
    __shared__ float warp_part[G4_THREADS / 32];

    const int b = blockIdx.y;
    const int tid = threadIdx.x;
    const int tx = tid % CT, ty = tid / CT;
    const float *q = queries + (int64_t)b * nq * D;
    for (int e = tid; e < NQP * D; e += G4_THREADS) {
        int i = e / D, x = e % D;
        qT[x * NQP + i] = i < nq ? q[e] : 0.f;
    }
    __syncthreads();
    for (int i = tid; i < NQP; i += G4_THREADS) {
        float s = 0.f;
        for (int x = 0; x < D; ++x) s += qT[x * NQP + i];
        sumq[i] = s;
    }

    const int32_t *tb = table + (int64_t)b * K * nq;
    const bool vec_rows = (nq == NQP);         // table rows are 16-byte aligned and complete
    const float4 *q4 = reinterpret_cast<const float4 *>(qT) + tx;
    const float4 *u4 = reinterpret_cast<const float4 *>(U) + ty;

    for (int j = blockIdx.x; j < n_prune; j += gridDim.x) {
        const int32_t d = pruned[(int64_t)b * n_prune + j];
        if (d < 0) {                            // uniform over the block
            if (tid == 0) score4[(int64_t)b * n_prune + j] = -INFINITY;
            continue;
        }
        const int64_t t0 = doc_off[DBG_DOC(d)], t1 = doc_off[DBG_DOC(d) + 1];
        float best[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
        for (int64_t base = t0; base < t1; base += TT) {
            const int cnt = (int)((t1 - base) < TT ? (t1 - base) : TT);
            __syncthreads();                    // previous tile (and red / sumq) fully consumed
            for (int w = tid; w < TT * CW; w += G4_THREADS) {
                const int tok = w % TT, wi = w / TT;
                const uint32_t word = tok < cnt ? __ldg(codes + (base + tok) * CW + wi) : 0u;
                float *dst = U + (wi * DPW) * TT + tok;
#pragma unroll
                for (int s = 0; s < DPW; ++s) dst[s * TT] = (float)((word >> (s * NBITS)) & MASK);
            }
            if (tid < TT) tok_cid[tid] = tid < cnt ? cids[base + tid] : -1;
            __syncthreads();

            float acc[4][4];
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int c = 0; c < 4; ++c) acc[r][c] = 0.f;
#pragma unroll 4
            for (int x = 0; x < D; ++x) {
                const float4 a = u4[x * TY];
                const float4 w = q4[x * CT];
                acc[0][0] = fmaf(a.x, w.x, acc[0][0]); acc[0][1] = fmaf(a.x, w.y, acc[0][1]);
                acc[0][2] = fmaf(a.x, w.z, acc[0][2]); acc[0][3] = fmaf(a.x, w.w, acc[0][3]);
                acc[1][0] = fmaf(a.y, w.x, acc[1][0]); acc[1][1] = fmaf(a.y, w.y, acc[1][1]);
                acc[1][2] = fmaf(a.y, w.z, acc[1][2]); acc[1][3] = fmaf(a.y, w.w, acc[1][3]);
                acc[2][0] = fmaf(a.z, w.x, acc[2][0]); acc[2][1] = fmaf(a.z, w.y, acc[2][1]);
                acc[2][2] = fmaf(a.z, w.z, acc[2][2]); acc[2][3] = fmaf(a.z, w.w, acc[2][3]);
                acc[3][0] = fmaf(a.w, w.x, acc[3][0]); acc[3][1] = fmaf(a.w, w.y, acc[3][1]);
                acc[3][2] = fmaf(a.w, w.z, acc[3][2]); acc[3][3] = fmaf(a.w, w.w, acc[3][3]);
            }
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const int32_t c = tok_cid[4 * ty + r];
                if (c < 0) continue;
                const int32_t *row = tb + (int64_t)DBG_CID(c) * nq + 4 * tx;
                int4 s;
                if (vec_rows) {
                    s = __ldg(reinterpret_cast<const int4 *>(row));
                } else {
                    s.x = 4 * tx + 0 < nq ? __ldg(row + 0) : 0;
                    s.y = 4 * tx + 1 < nq ? __ldg(row + 1) : 0;
                    s.z = 4 * tx + 2 < nq ? __ldg(row + 2) : 0;
                    s.w = 4 * tx + 3 < nq ? __ldg(row + 3) : 0;
                }
                const float k24 = 1.0f / 16777216.0f;
                best[0] = fmaxf(best[0], fmaf(delta, acc[r][0], (float)s.x * k24));
                best[1] = fmaxf(best[1], fmaf(delta, acc[r][1], (float)s.y * k24));
                best[2] = fmaxf(best[2], fmaf(delta, acc[r][2], (float)s.z * k24));
                best[3] = fmaxf(best[3], fmaf(delta, acc[r][3], (float)s.w * k24));
            }
        }
        // merge the TY token rows, add the per-query-token constant, sum over query tokens
        __syncthreads();
#pragma unroll
        for (int c = 0; c < 4; ++c) red[ty * NQP + 4 * tx + c] = best[c];
        __syncthreads();
        float v = 0.f;
        if (tid < NQP && tid < nq) {
            float m = red[tid];
            for (int r = 1; r < TY; ++r) m = fmaxf(m, red[r * NQP + tid]);
            v = m + kappa * sumq[tid];
        }
        v = warp_sum(v);
        if ((tid & 31) == 0) warp_part[tid >> 5] = v;
        __syncthreads();
        if (tid == 0) {
            float total = 0.f;
            for (int w = 0; w < G4_THREADS / 32; ++w) total += warp_part[w];
            score4[(int64_t)b * n_prune + j] = total;
        }
    }
}

template <int CT, int NBITS>
static int launch_g4(const Index &ix, const Params &p, const float *queries, const int32_t *table,
                     const int32_t *pruned, float *score4, cudaStream_t st)
{
    constexpr int NQP = 4 * CT, TY = G4_THREADS / CT, TT = 4 * TY;
    const float delta = (ix.res_hi - ix.res_lo) / (float)(1 << ix.nbits);
    const float kappa = ix.res_lo + 0.5f * delta;
    const size_t smem = sizeof(float) * ((size_t)ix.D * NQP + (size_t)ix.D * TT + (size_t)TY * NQP + NQP + TT);
    auto kern = residual_maxsim_kernel<CT, NBITS>;
    if (smem > 48 * 1024)
        CHIMERA_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    // blocks per query: enough to fill the device a few times over, at most one per surviving document
    int64_t per_query = ((int64_t)ix.sm_count * 16 + p.B - 1) / p.B;
    if (per_query > p.n_prune) per_query = p.n_prune;
    if (per_query < 1) per_query = 1;
    dim3 grid((unsigned)per_query, (unsigned)p.B);
    kern<<<grid, G4_THREADS, smem, st>>>(queries, table, ix.K, p.nq, ix.D, ix.CB / 4, delta, kappa, pruned, p.n_prune,
                                         ix.cids, reinterpret_cast<const uint32_t *>(ix.codes), ix.doc_off, score4);
    CHIMERA_CUDA(cudaGetLastError());
    count_launch(SLOT_G4);
    return CHIMERA_OK;
}

int launch_residual_scores(const Index &ix, const Params &p, const float *queries, const int32_t *table,
                           const int32_t *pruned, float *score4, cudaStream_t st)
{
    const int ct = p.nq <= 32 ? 8 : (p.nq <= 64 ? 16 : 32);
    if (ix.nbits == 2) {
        if (ct == 8) return launch_g4<8, 2>(ix, p, queries, table, pruned, score4, st);
        if (ct == 16) return launch_g4<16, 2>(ix, p, queries, table, pruned, score4, st);
        return launch_g4<32, 2>(ix, p, queries, table, pruned, score4, st);
    }
    if (ct == 8) return launch_g4<8, 1>(ix, p, queries, table, pruned, score4, st);
    if (ct == 16) return launch_g4<16, 1>(ix, p, queries, table, pruned, score4, st);
    return launch_g4<32, 1>(ix, p, queries, table, pruned, score4, st);
}

}  // namespace chimera
