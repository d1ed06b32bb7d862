// The paper's GPU pipeline on RaBitQ 1-bit codes (Sec. 2.2 for the codec, Sec. 3.2 steps 2 and 3 for its use):
//   q_p = P q                                         (rotation; inner products are preserved)
//   est(i, t) = <q_p, o_p-bar> / <o_p, o_p-bar>,  <q_p, o_p-bar> = (1 / |y-bar|) (<q_p, o_b> - 1/2 sum q_p)
// evaluated as  inv_dot_t * (c * (float)(2 T - SQ_i)),  T = sum_x Xq_i[x] o_b[x],  SQ_i = sum_x Xq_i[x],
// Xq = rint(q_p * 2^22),  c = 1 / (sqrt(D) 2^22): integers plus two fp32 multiplications in a fixed order, and sums
// over query tokens in increasing order, so every result is reproducible bit for bit.
//
// This file: attaching the codes to an index, the rotation kernel, and candidate refinement by partial 1-bit scores
// (Algorithm 2; one block per (query token, posting list) as in the paper's design, atomicMax as in Algorithm 4).
// The complete 1-bit scores of the survivors run on the tensor cores (g4_residual_umma.cu, RQ variant).
#include <math.h>

#include "common.cuh"

namespace chimera {

__global__ void transpose_kernel(const float *__restrict__ in, int D, float *__restrict__ out)
{
    int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e < D * D) {
        int r = e / D, x = e % D;
        out[x * D + r] = in[e];
    }
}

int attach_rabitq(Index &ix, const float *rotation, cudaStream_t st)
{
    if (!ix.rot_t) CHIMERA_CUDA(cudaMalloc(&ix.rot_t, sizeof(float) * ix.D * ix.D));
    transpose_kernel<<<(ix.D * ix.D + 255) / 256, 256, 0, st>>>(rotation, ix.D, ix.rot_t);
    CHIMERA_CUDA(cudaGetLastError());
    CHIMERA_CUDA(cudaStreamSynchronize(st));
    return CHIMERA_OK;
}

// grid (B * nq), block D: q_p[row][r] = sum_x P[r][x] q[row][x] as one fma chain in increasing x.
__global__ void __launch_bounds__(128)
rotate_kernel(const float *__restrict__ rot_t, const float *__restrict__ q, int D, float *__restrict__ out)
{
    __shared__ float qrow[128];
    const int64_t row = blockIdx.x;
    const int r = threadIdx.x;
    if (r < D) qrow[r] = q[row * D + r];
    __syncthreads();
    if (r < D) {
        float acc = 0.0f;
        for (int x = 0; x < D; ++x) acc = fmaf(rot_t[x * D + r], qrow[x], acc);
        out[row * D + r] = acc;
    }
}

int launch_rotate(const Index &ix, const Params &p, const float *queries, float *q_rot, cudaStream_t st)
{
    rotate_kernel<<<(unsigned)((int64_t)p.B * p.nq), 128, 0, st>>>(ix.rot_t, queries, ix.D, q_rot);
    CHIMERA_CUDA(cudaGetLastError());
    count_launch(SLOT_G1);
    return CHIMERA_OK;
}

constexpr int RP_THREADS = 128;

// grid (blocks, B): zero the first n_cand[b] rows of M.
__global__ void __launch_bounds__(256)
rabitq_clear_kernel(int32_t *__restrict__ M, const int32_t *__restrict__ n_cand, int64_t maxc, int nq)
{
    const int b = blockIdx.y;
    const int64_t n = (int64_t)n_cand[b] * nq;
    int32_t *row = M + (int64_t)b * maxc * nq;
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x, stride = (int64_t)gridDim.x * blockDim.x;
    if ((nq & 3) == 0) {                               // rows are 16-byte aligned
        int4 *row4 = reinterpret_cast<int4 *>(row);
        for (int64_t e = tid; e < n / 4; e += stride) row4[e] = make_int4(0, 0, 0, 0);
    } else {
        for (int64_t e = tid; e < n; e += stride) row[e] = 0;
    }
}

// grid (nq * P, B): one block per (query token, probed list); M holds float bits (>= 0, so integer order = float order).
__global__ void __launch_bounds__(RP_THREADS)
rabitq_partial_kernel(const float *__restrict__ q_rot, int nq, int D, int P, float c, const int32_t *__restrict__ probes,
                      const int64_t *__restrict__ tok_off, const int32_t *__restrict__ tok_id,
                      const int32_t *__restrict__ tok_doc, const uint32_t *__restrict__ bits,
                      const float *__restrict__ inv_dot, const uint32_t *__restrict__ bitmap,
                      const int32_t *__restrict__ word_rank, int64_t words, int64_t maxc, int32_t *__restrict__ M)
{
    // Sec. 4.1's look-up-table form of the binary inner product: for every group of four dimensions the 16 partial
    // sums of the query token's integers are tabulated once per block (D/4 * 16 entries: cheap next to a list of a few
    // hundred tokens), so a token costs D/4 table reads and adds instead of a data-dependent loop over its set bits.
    // Integer sums: the same T in any order.
    __shared__ int32_t xq[128];
    __shared__ int32_t lut[32 * 16];
    __shared__ int s_sq;
    const int b = blockIdx.y;
    const int i = blockIdx.x / P;
    const int32_t cen = DBG_CID(probes[((int64_t)b * nq + i) * P + blockIdx.x % P]);
    const float *q = q_rot + ((int64_t)b * nq + i) * D;
    for (int x = threadIdx.x; x < D; x += RP_THREADS)
        xq[x] = __float2int_rn(fminf(fmaxf(q[x], -1.0f), 1.0f) * 4194304.0f);
    __syncthreads();
    if (threadIdx.x == 0) {
        int s = 0;
        for (int x = 0; x < D; ++x) s += xq[x];
        s_sq = s;
    }
    for (int e = threadIdx.x; e < (D >> 2) * 16; e += RP_THREADS) {
        const int g = e >> 4, v = e & 15;
        int s = 0;
#pragma unroll
        for (int t = 0; t < 4; ++t) s += ((v >> t) & 1) ? xq[4 * g + t] : 0;
        lut[e] = s;
    }
    __syncthreads();
    const int sq = s_sq;
    const int CW = D >> 5;
    const uint32_t *bm = bitmap + (int64_t)b * words;
    const int32_t *wr = word_rank + (int64_t)b * words;
    int32_t *Mb = M + (int64_t)b * maxc * nq;
    auto code_dot = [&](int64_t t) -> int {
        uint32_t word[4];                              // D <= 128: at most four words
        if (CW == 4) {                                 // 16-byte rows (the attach call checks the alignment)
            const uint4 v = __ldg(reinterpret_cast<const uint4 *>(bits + t * 4));
            word[0] = v.x; word[1] = v.y; word[2] = v.z; word[3] = v.w;
        } else {
#pragma unroll
            for (int w = 0; w < 4; ++w) word[w] = w < CW ? __ldg(bits + t * CW + w) : 0u;
        }
        int T = 0;
#pragma unroll
        for (int w = 0; w < 4; ++w)
            if (w < CW) {
#pragma unroll
                for (int k = 0; k < 8; ++k) T += lut[(8 * w + k) * 16 + ((word[w] >> (4 * k)) & 15u)];
            }
        return T;
    };
    // (the token's factor, the document's bitmap word and its rank come as arguments: they depend on the list entry
    // alone, so their loads are issued with the code loads instead of one after the other behind the score)
    auto update = [&](uint32_t d, float factor, int T, uint32_t bm_word, int32_t wr_word) {
        const float est = __fmul_rn(factor, __fmul_rn(c, (float)(2 * T - sq)));
        if (est > 0.0f) {                              // the table starts at 0 (Algorithm 2)
            const int64_t rank = wr_word + __popc(bm_word & ((1u << (d & 31)) - 1u));
            if (rank < maxc && DBG_RANK_OK(rank)) atomicMax(&Mb[rank * nq + i], __float_as_int(est));
        }
    };
    const int64_t e1 = tok_off[cen + 1];
    int64_t e = tok_off[cen] + threadIdx.x;
    for (; e + RP_THREADS < e1; e += 2 * RP_THREADS) {         // two visits per iteration, their loads issued together
        const int64_t ta = DBG_TOK(tok_id[e]), tb = DBG_TOK(tok_id[e + RP_THREADS]);
        const uint32_t da = (uint32_t)DBG_DOC(tok_doc[e]), db = (uint32_t)DBG_DOC(tok_doc[e + RP_THREADS]);
        const float fa = __ldg(inv_dot + ta), fb = __ldg(inv_dot + tb);
        const uint32_t bma = __ldg(bm + (da >> 5)), bmb = __ldg(bm + (db >> 5));
        const int32_t wra = __ldg(wr + (da >> 5)), wrb = __ldg(wr + (db >> 5));
        const int Ta = code_dot(ta), Tb = code_dot(tb);
        update(da, fa, Ta, bma, wra);
        update(db, fb, Tb, bmb, wrb);
    }
    if (e < e1) {
        const int64_t t = DBG_TOK(tok_id[e]);
        const uint32_t d = (uint32_t)DBG_DOC(tok_doc[e]);
        const float f = __ldg(inv_dot + t);
        const uint32_t bmd = __ldg(bm + (d >> 5));
        const int32_t wrd = __ldg(wr + (d >> 5));
        update(d, f, code_dot(t), bmd, wrd);
    }
}

// grid (blocks, B): F'[b][j] = M[b][j][0] + M[b][j][1] + ... in that order (fp32), one thread per candidate.
__global__ void __launch_bounds__(256)
rabitq_sum_kernel(const int32_t *__restrict__ M, const int32_t *__restrict__ n_cand, int64_t maxc, int nq,
                  int32_t *__restrict__ fprime_bits)
{
    const int b = blockIdx.y;
    const int n = n_cand[b];
    for (int j = blockIdx.x * blockDim.x + threadIdx.x; j < n; j += gridDim.x * blockDim.x) {
        const int32_t *row = M + ((int64_t)b * maxc + j) * nq;
        float s = 0.0f;
        if ((nq & 3) == 0) {
            const int4 *row4 = reinterpret_cast<const int4 *>(row);
            for (int i = 0; i < nq / 4; ++i) {
                const int4 v = row4[i];
                s = __fadd_rn(s, __int_as_float(v.x));
                s = __fadd_rn(s, __int_as_float(v.y));
                s = __fadd_rn(s, __int_as_float(v.z));
                s = __fadd_rn(s, __int_as_float(v.w));
            }
        } else {
            for (int i = 0; i < nq; ++i) s = __fadd_rn(s, __int_as_float(row[i]));
        }
        fprime_bits[(int64_t)b * maxc + j] = __float_as_int(s);
    }
}

int launch_rabitq_partial(const Index &ix, const Params &p, const Layout &L, const float *q_rot,
                          const int32_t *probes, const uint32_t *bitmap, const int32_t *word_rank,
                          const int32_t *n_cand, int32_t *partial_m, int32_t *fprime_bits, cudaStream_t st)
{
    int64_t per_query = ((int64_t)ix.sm_count * 8 + p.B - 1) / p.B;
    if (per_query < 1) per_query = 1;
    dim3 gclr((unsigned)per_query, (unsigned)p.B);
    rabitq_clear_kernel<<<gclr, 256, 0, st>>>(partial_m, n_cand, p.maxc, p.nq);
    CHIMERA_CUDA(cudaGetLastError());
    const float c = (float)(1.0 / (sqrt((double)ix.D) * 4194304.0));
    rabitq_partial_kernel<<<dim3((unsigned)(p.nq * p.P), (unsigned)p.B), RP_THREADS, 0, st>>>(
        q_rot, p.nq, ix.D, p.P, c, probes, ix.tok_off, ix.tok_id, ix.tok_doc,
        reinterpret_cast<const uint32_t *>(ix.rq_bits), ix.rq_inv, bitmap, word_rank, L.words, p.maxc, partial_m);
    CHIMERA_CUDA(cudaGetLastError());
    rabitq_sum_kernel<<<gclr, 256, 0, st>>>(partial_m, n_cand, p.maxc, p.nq, fprime_bits);
    CHIMERA_CUDA(cudaGetLastError());
    count_launch(SLOT_CI, 3);
    return CHIMERA_OK;
}

}  // namespace chimera
