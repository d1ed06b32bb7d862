// Candidate refinement with partial scores (Sec. 3.2 step 2, Algorithm 2; aggregation as in Algorithm 4): only the
// tokens retrieved in candidate generation contribute.  For query token i and each of its probed centroids, every
// token of that centroid's posting list raises M[document, i] to max(M, dist(i, token)); M starts at 0 and the partial
// score is F'(d) = sum_i M[d, i].
//
// dist(i, t) = S[cid_t, i] + llrint(delta*4*T + kappa*4*SQ_i) in Q.24 fixed point, T = sum_x Xq_i[x] u_t[x],
// SQ_i = sum_x Xq_i[x], Xq = rint(q * 2^22): integers plus one correctly rounded double expression, so the result does
// not depend on the order in which tokens are visited (integer max) nor on the machine.
//
// As in the paper's design a block serves one (query token, posting list) pair: the query token's integers sit in
// shared memory, one thread scores one document token, and the maximum goes to the score table with atomicMax while the
// thread moves on to its next token; every increase of a table entry is also added to the document's partial score, so
// no separate summation pass is needed.  The table is indexed by candidate rank (bitmap word prefix + popcount), so it has
// one 4*q_len-byte row per candidate rather than per document.
//
// Only about one cell per candidate is ever touched (a candidate owns about one retrieved token), so on large corpora
// the table is kept as an open-addressing hash table instead: key = rank * q_len + i + 1 in the high word of a 64-bit
// slot, the running maximum in the low word; a slot's key never changes once set, so the maximum is one 64-bit
// atomicMax on the slot.  The slots of a query (a power of two, at least twice the largest possible number of
// visits: q_len * nprobe * longest list) are a few MB against tens of MB of dense rows: the clear is that much
// shorter and the read-modify-writes of the queries in flight stay in L2.
#include "common.cuh"

namespace chimera {

constexpr int PS_THREADS = 128;
constexpr int HASH_MAX_PROBES = 256;     // linear probing gives up after this many slots (load factor <= 1/2)

int64_t partial_hash_slots(const Index &ix, const Params &p)
{
    if (!ix.tok_id || ix.max_tok_list <= 0) return 0;
    if ((int64_t)p.maxc * p.nq >= 0xffffffffLL) return 0;                  // keys must fit 32 bits
    if (4 * p.B <= ix.sm_count) return 0;      // few queries per call: latency counts, and a dense cell is one atomic
                                               // where a slot is a load, a compare-and-swap and a maximum (Mid, one query:
                                               // 36 us dense, 46 us hashed)
    const int64_t visits = (int64_t)p.nq * p.P * ix.max_tok_list;          // distinct cells are at most the visits
    int64_t slots = 1024;
    while (slots < 2 * visits) slots <<= 1;
    if (slots * 8 * 4 > (int64_t)p.maxc * p.nq * 4) return 0;              // worth it from a quarter of the dense size down
                                                                           // (long documents, 32 MB against 51 MB: slower)
    return slots;
}

// grid (blocks, B): zero a query's slots and the first n_cand[b] partial scores.
__global__ void __launch_bounds__(256)
hash_clear_kernel(unsigned long long *__restrict__ H, int64_t slots, int32_t *__restrict__ fprime,
                  const int32_t *__restrict__ n_cand, int64_t maxc)
{
    const int b = blockIdx.y;
    uint4 *row = reinterpret_cast<uint4 *>(H + (int64_t)b * slots);         // slots is a multiple of 1024
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x, stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t e = tid; e < slots / 2; e += stride) row[e] = make_uint4(0u, 0u, 0u, 0u);
    for (int64_t e = tid; e < n_cand[b]; e += stride) fprime[(int64_t)b * maxc + e] = 0;
}

// grid (blocks, B): zero the first n_cand[b] rows of M and the first n_cand[b] partial scores.
__global__ void __launch_bounds__(256)
partial_clear_kernel(int32_t *__restrict__ M, int32_t *__restrict__ fprime, const int32_t *__restrict__ n_cand,
                     int64_t maxc, int nq)
{
    const int b = blockIdx.y;
    const int64_t n = (int64_t)n_cand[b] * nq;
    int4 *row = reinterpret_cast<int4 *>(M + (int64_t)b * maxc * nq);      // rows are 16-byte aligned when nq % 4 == 0
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x, stride = (int64_t)gridDim.x * blockDim.x;
    if ((nq & 3) == 0 && (maxc * nq) % 4 == 0) {
        for (int64_t e = tid; e < n / 4; e += stride) row[e] = make_int4(0, 0, 0, 0);
    } else {
        int32_t *r1 = M + (int64_t)b * maxc * nq;
        for (int64_t e = tid; e < n; e += stride) r1[e] = 0;
    }
    for (int64_t e = tid; e < n_cand[b]; e += stride) fprime[(int64_t)b * maxc + e] = 0;
}

// grid (nq * P, B): one block per (query token, probed list).
template <int NBITS, bool HASH>
__global__ void __launch_bounds__(PS_THREADS)
partial_score_kernel(const float *__restrict__ queries, const int32_t *__restrict__ table, int64_t K, int nq, int D,
                     int CW, int P, float delta, float kappa, const int32_t *__restrict__ probes,
                     const int64_t *__restrict__ tok_off, const int32_t *__restrict__ tok_id,
                     const int32_t *__restrict__ tok_doc, const uint32_t *__restrict__ codes,
                     const uint32_t *__restrict__ bitmap, const int32_t *__restrict__ word_rank, int64_t words,
                     int64_t maxc, int32_t *__restrict__ M, int32_t *__restrict__ fprime, int64_t slots,
                     uint32_t *__restrict__ status)
{
    __shared__ int32_t xq[128];
    __shared__ long long s_sq;
    const int b = blockIdx.y;
    const int i = blockIdx.x / P;
    const int32_t c = DBG_CID(probes[((int64_t)b * nq + i) * P + blockIdx.x % P]);
    const float *q = queries + ((int64_t)b * nq + i) * D;
    for (int x = threadIdx.x; x < D; x += PS_THREADS) {
        float v = fminf(fmaxf(q[x], -1.0f), 1.0f);
        xq[x] = __float2int_rn(v * 4194304.0f);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        long long s = 0;
        for (int x = 0; x < D; ++x) s += xq[x];
        s_sq = s;
    }
    __syncthreads();
    const int32_t s_c = table[((int64_t)b * K + c) * nq + i];
    const double d4 = __dmul_rn((double)delta, 4.0);
    const double kterm = __dmul_rn(__dmul_rn((double)kappa, 4.0), (double)s_sq);
    const uint32_t *bm = bitmap + (int64_t)b * words;
    const int32_t *wr = word_rank + (int64_t)b * words;
    int32_t *Mb = M + (int64_t)b * maxc * nq;
    unsigned long long *Hb = reinterpret_cast<unsigned long long *>(M) + (int64_t)b * slots;
    const uint32_t slot_mask = (uint32_t)(slots - 1);
    constexpr int DPW = 32 / NBITS;
    constexpr uint32_t MASK = (1u << NBITS) - 1u;
    // One visit: the token's packed code (16-byte loads where the code size allows) against the query token's integers.
    auto code_dot = [&](int64_t t) -> int {
        const uint32_t *cw = codes + t * CW;
        uint32_t word[8];                              // at most 32 code bytes per token
        if (NBITS == 2 && CW == 8) {                   // 32-byte codes (32-byte aligned): one load
            asm volatile("ld.global.nc.v8.u32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                         : "=r"(word[0]), "=r"(word[1]), "=r"(word[2]), "=r"(word[3]), "=r"(word[4]), "=r"(word[5]),
                           "=r"(word[6]), "=r"(word[7])
                         : "l"(cw));
        } else if ((CW & 3) == 0) {
#pragma unroll
            for (int w = 0; w < 8; w += 4)
                if (w < CW) {
                    const uint4 v = __ldg(reinterpret_cast<const uint4 *>(cw + w));
                    word[w] = v.x; word[w + 1] = v.y; word[w + 2] = v.z; word[w + 3] = v.w;
                }
        } else if ((CW & 1) == 0) {
#pragma unroll
            for (int w = 0; w < 8; w += 2)
                if (w < CW) {
                    const uint2 v = __ldg(reinterpret_cast<const uint2 *>(cw + w));
                    word[w] = v.x; word[w + 1] = v.y;
                }
        } else {
#pragma unroll
            for (int w = 0; w < 8; ++w)
                if (w < CW) word[w] = __ldg(cw + w);
        }
        int T = 0;                                     // |T| <= 3 * 2^22 * |q|_1 < 2^31 for unit-norm queries
#pragma unroll
        for (int w = 0; w < 8; ++w)
            if (w < CW) {
#pragma unroll
                for (int s = 0; s < DPW; ++s) T += xq[w * DPW + s] * (int)((word[w] >> (s * NBITS)) & MASK);
            }
        return T;
    };
    // (the document's bitmap word and its rank come as arguments: they depend on the list entry alone, so their loads
    // are issued with the code loads instead of after the score is known -- one memory latency less per visit)
    auto update = [&](uint32_t d, int T, uint32_t bm_word, int32_t wr_word) {
        const double r = __dadd_rn(__dmul_rn(d4, (double)T), kterm);
        const long long dist = (long long)s_c + __double2ll_rn(r);
        if (dist > 0) {                                // the table starts at 0 (Algorithm 2)
            const int64_t rank = wr_word + __popc(bm_word & ((1u << (d & 31)) - 1u));
            if (rank < maxc && DBG_RANK_OK(rank)) {
                // F' = sum_i M[., i] is kept up to date with the increments: M only grows, integer adds commute
                int32_t old = 0;
                if (HASH) {
                    const uint32_t key = (uint32_t)(rank * nq + i) + 1u;
                    const unsigned long long mine = ((unsigned long long)key << 32) | (uint32_t)dist;
                    uint32_t h = (key * 2654435761u) & slot_mask;
                    int probes = 0;
                    for (; probes < HASH_MAX_PROBES; ++probes, h = (h + 1u) & slot_mask) {
                        unsigned long long cur = Hb[h];
                        if (cur == 0ull) {
                            cur = atomicCAS(&Hb[h], 0ull, mine);
                            if (cur == 0ull) break;                         // new cell: the old maximum is 0
                        }
                        if ((uint32_t)(cur >> 32) == key) {                 // this cell's slot (its key is final)
                            old = (int32_t)(uint32_t)atomicMax(&Hb[h], mine);
                            break;
                        }
                    }
                    if (probes == HASH_MAX_PROBES) {                        // cannot happen below half load; reported
                        atomicOr(status, ST_OVERFLOW);
                        old = (int32_t)dist;                                // no increment
                    }
                } else {
                    old = atomicMax(&Mb[rank * nq + i], (int32_t)dist);
                }
                if ((int32_t)dist > old) atomicAdd(&fprime[(int64_t)b * maxc + rank], (int32_t)dist - old);
            }
        }
    };
    // two visits per thread and iteration, their loads issued together
    const int64_t e1 = tok_off[c + 1];
    int64_t e = tok_off[c] + threadIdx.x;
    for (; e + PS_THREADS < e1; e += 2 * PS_THREADS) {
        const int64_t ta = DBG_TOK(tok_id[e]), tb2 = DBG_TOK(tok_id[e + PS_THREADS]);
        const uint32_t da = (uint32_t)DBG_DOC(tok_doc[e]), db = (uint32_t)DBG_DOC(tok_doc[e + PS_THREADS]);
        const uint32_t bma = __ldg(bm + (da >> 5)), bmb = __ldg(bm + (db >> 5));
        const int32_t wra = __ldg(wr + (da >> 5)), wrb = __ldg(wr + (db >> 5));
        const int Ta = code_dot(ta), Tb = code_dot(tb2);
        update(da, Ta, bma, wra);
        update(db, Tb, bmb, wrb);
    }
    if (e < e1) {
        const uint32_t d = (uint32_t)DBG_DOC(tok_doc[e]);
        const uint32_t bmd = __ldg(bm + (d >> 5));
        const int32_t wrd = __ldg(wr + (d >> 5));
        update(d, code_dot(DBG_TOK(tok_id[e])), bmd, wrd);
    }
}

int launch_partial_scores(const Index &ix, const Params &p, const Layout &L, const float *queries,
                          const int32_t *table, const int32_t *probes, const uint32_t *bitmap,
                          const int32_t *word_rank, const int32_t *n_cand, int32_t *partial_m, int32_t *fprime,
                          uint32_t *status, cudaStream_t st)
{
    const float delta = (ix.res_hi - ix.res_lo) / (float)(1 << ix.nbits);
    const float kappa = ix.res_lo + 0.5f * delta;
    int64_t per_query = ((int64_t)ix.sm_count * 8 + p.B - 1) / p.B;
    if (per_query < 1) per_query = 1;
    dim3 gclr((unsigned)per_query, (unsigned)p.B);
    const bool hashed = L.hash_slots > 0;
    if (hashed)
        hash_clear_kernel<<<gclr, 256, 0, st>>>(reinterpret_cast<unsigned long long *>(partial_m), L.hash_slots, fprime,
                                                n_cand, p.maxc);
    else
        partial_clear_kernel<<<gclr, 256, 0, st>>>(partial_m, fprime, n_cand, p.maxc, p.nq);
    CHIMERA_CUDA(cudaGetLastError());
    dim3 grid((unsigned)(p.nq * p.P), (unsigned)p.B);
    const uint32_t *codes = reinterpret_cast<const uint32_t *>(ix.codes);
#define PS_LAUNCH(NB, HS)                                                                                              \
    partial_score_kernel<NB, HS><<<grid, PS_THREADS, 0, st>>>(queries, table, ix.K, p.nq, ix.D, ix.CB / 4, p.P, delta, \
                                                              kappa, probes, ix.tok_off, ix.tok_id, ix.tok_doc, codes, \
                                                              bitmap, word_rank, L.words, p.maxc, partial_m, fprime,   \
                                                              L.hash_slots, status)
    if (ix.nbits == 2) {
        if (hashed) PS_LAUNCH(2, true); else PS_LAUNCH(2, false);
    } else {
        if (hashed) PS_LAUNCH(1, true); else PS_LAUNCH(1, false);
    }
#undef PS_LAUNCH
    CHIMERA_CUDA(cudaGetLastError());
    count_launch(SLOT_CI, 2);
    return CHIMERA_OK;
}

}  // namespace chimera
