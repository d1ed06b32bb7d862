// Stage 3: centroid-interaction pruning.
//   CI(d) = sum_i max_{t in d} S[cid_t, i]      (the Chamfer aggregation rule of Sec. 4.2 -- per query token the
//                                                maximum over the document's tokens, then the sum over query
//                                                tokens -- applied to the centroid scores; integers, order-free)
//   keep the n_prune candidates with the largest CI, ties towards the smaller document id.
//
// Two phases when q_len is 32 or 64: cheap bounds lo(d) <= CI(d) <= hi(d) for every candidate from an 8-bit copy of
// the table (cand_range_kernel + ci_coarse_rng_kernel; ci_coarse_kernel for tables staged in shared memory and for
// corpora of 2^31 tokens or more), the documents whose hi reaches the n_prune-th largest lo (contender kernels), then
// exact CI (ci_wide_rng_kernel over the contenders' token ranges; ci_wide_kernel without ranges) and the exact
// selection among those only.  Other q_len: exact CI for every candidate
// (ci_kernel).
//
// ci_kernel: one warp per candidate document.  The document's centroid ids are streamed with coalesced 128-byte
// loads (lane = token), each is broadcast with a shuffle, and the warp gathers the table row S[cid, :] with
// lane = query token (one 128-byte line for 32 query tokens), keeping a running maximum per lane.
//
// select_kernel: one block per query.  Radix select (11 + 11 + 10 bits) of the n_prune-th largest score, then an
// ordered compaction of the candidate list (which is ascending in id), so equal scores are resolved towards smaller
// ids and the survivors come out ascending.  With few queries per call the contender and selection steps run over 32
// blocks per query instead (contender_hist/count/write kernels, sels_* kernels), and shard_select_kernel merges the
// lists of a document-sharded search.
#include <limits.h>

#include "common.cuh"

namespace chimera {

constexpr int CI_THREADS = 256;
constexpr int CI_WARPS = CI_THREADS / 32;

template <int NQW>   // 32-column groups handled per lane
__global__ void __launch_bounds__(CI_THREADS)
ci_kernel(const int32_t *__restrict__ table, int64_t K, int nq, const int32_t *__restrict__ cand,
          const int32_t *__restrict__ n_cand, int64_t maxc, const int32_t *__restrict__ cids,
          const int64_t *__restrict__ doc_off, int32_t *__restrict__ ci)
{
    const int b = blockIdx.y;
    const int lane = threadIdx.x & 31;
    const int n = n_cand[b];
    const int32_t *tb = table + (int64_t)b * K * nq;
    const int32_t *cb = cand + (int64_t)b * maxc;
    int32_t *out = ci + (int64_t)b * maxc;
    const int warps_per_query = gridDim.x * CI_WARPS;
    for (int j = blockIdx.x * CI_WARPS + (threadIdx.x >> 5); j < n; j += warps_per_query) {
        const int64_t d = DBG_DOC(cb[j]);
        const int64_t t0 = doc_off[d], t1 = doc_off[d + 1];
        int m[NQW];
#pragma unroll
        for (int w = 0; w < NQW; ++w) m[w] = INT_MIN;
        for (int64_t base = t0; base < t1; base += 32) {
            const int cnt = (int)((t1 - base) < 32 ? (t1 - base) : 32);
            // lanes past the end repeat the last token: a duplicate cannot change a maximum
            const int32_t cidv = cids[base + (lane < cnt ? lane : cnt - 1)];
            for (int t = 0; t < cnt; t += 8) {
                int32_t c[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) c[u] = __shfl_sync(0xffffffffu, cidv, t + u);   // t + u <= 31
                int32_t v[8][NQW];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int32_t *row = tb + (int64_t)DBG_CID(c[u]) * nq;
#pragma unroll
                    for (int w = 0; w < NQW; ++w) {
                        int col = lane + 32 * w;
                        v[u][w] = (col < nq) ? __ldg(row + col) : INT_MIN;
                    }
                }
#pragma unroll
                for (int u = 0; u < 8; ++u)
#pragma unroll
                    for (int w = 0; w < NQW; ++w) m[w] = max(m[w], v[u][w]);
            }
        }
        int s = 0;
#pragma unroll
        for (int w = 0; w < NQW; ++w)
            if (lane + 32 * w < nq) s += m[w];
        s = warp_sum(s);
        if (lane == 0) out[j] = s;
    }
}

// Wide variant for q_len = 4 * LPR (LPR = 8 or 16 lanes per table row): every lane loads 16 bytes (four query
// tokens) of a row, so one load instruction of the warp covers 32 / LPR document tokens.  Lane group g = lane / LPR
// takes tokens g, g + TPL, g + 2 TPL, ... of each 32-token slab; the group maxima are merged with shuffles at the end.
template <int LPR>
__global__ void __launch_bounds__(CI_THREADS)
ci_wide_kernel(const int32_t *__restrict__ table, int64_t K, const int32_t *__restrict__ cand,
               const int32_t *__restrict__ n_cand, int64_t maxc, const int32_t *__restrict__ cids,
               const int64_t *__restrict__ doc_off, int32_t *__restrict__ ci)
{
    constexpr int NQ = 4 * LPR;
    constexpr int TPL = 32 / LPR;                 // tokens per warp-wide load
    constexpr int UNROLL = 8;
    const int b = blockIdx.y;
    const int lane = threadIdx.x & 31;
    const int grp = lane / LPR, sub = lane % LPR;
    const int n = n_cand[b];
    const int4 *tb = reinterpret_cast<const int4 *>(table + (int64_t)b * K * NQ) + sub;
    const int32_t *cb = cand + (int64_t)b * maxc;
    int32_t *out = ci + (int64_t)b * maxc;
    const int warps_per_query = gridDim.x * CI_WARPS;
    for (int j = blockIdx.x * CI_WARPS + (threadIdx.x >> 5); j < n; j += warps_per_query) {
        const int64_t d = DBG_DOC(cb[j]);
        const int64_t t0 = doc_off[d], t1 = doc_off[d + 1];
        int4 m = make_int4(INT_MIN, INT_MIN, INT_MIN, INT_MIN);
        for (int64_t base = t0; base < t1; base += 32) {
            const int cnt = (int)((t1 - base) < 32 ? (t1 - base) : 32);
            // lanes past the end repeat the last token: a duplicate cannot change a maximum
            const int32_t cidv = cids[base + (lane < cnt ? lane : cnt - 1)];
            for (int s = 0; s * TPL < cnt; s += UNROLL) {
                int4 v[UNROLL];
#pragma unroll
                for (int u = 0; u < UNROLL; ++u) {
                    int src = (s + u) * TPL + grp;
                    src = src < 32 ? src : 31;    // lane 31 holds a valid (possibly repeated) token
                    const int32_t c = __shfl_sync(0xffffffffu, cidv, src);
                    v[u] = __ldg(tb + (int64_t)DBG_CID(c) * LPR);
                }
#pragma unroll
                for (int u = 0; u < UNROLL; u += 2) {          // three-input integer maximum: two rows per instruction
                    m.x = __vimax3_s32(m.x, v[u].x, v[u + 1].x);
                    m.y = __vimax3_s32(m.y, v[u].y, v[u + 1].y);
                    m.z = __vimax3_s32(m.z, v[u].z, v[u + 1].z);
                    m.w = __vimax3_s32(m.w, v[u].w, v[u + 1].w);
                }
            }
        }
        // merge the TPL lane groups (same columns, different tokens)
#pragma unroll
        for (int o = LPR; o < 32; o <<= 1) {
            m.x = max(m.x, __shfl_xor_sync(0xffffffffu, m.x, o));
            m.y = max(m.y, __shfl_xor_sync(0xffffffffu, m.y, o));
            m.z = max(m.z, __shfl_xor_sync(0xffffffffu, m.z, o));
            m.w = max(m.w, __shfl_xor_sync(0xffffffffu, m.w, o));
        }
        // sum over the NQ columns: four per lane, LPR lanes
        int sum = m.x + m.y + m.z + m.w;
#pragma unroll
        for (int o = LPR >> 1; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        if (lane == 0) out[j] = sum;
    }
}

// The wide variant over precomputed token ranges (first token, length) of the documents to score: a warp owns a
// contiguous run of them and takes them 32 at a time -- one coalesced load of the ranges, handed out by shuffle, and the
// first centroid ids of the next document fetched while the current one is scored -- instead of the dependent chain
// id -> offsets -> centroid ids per document.
template <int LPR>
__global__ void __launch_bounds__(CI_THREADS)
ci_wide_rng_kernel(const int32_t *__restrict__ table, int64_t K, const int2 *__restrict__ rng,
                   const int32_t *__restrict__ n_docs, int64_t maxc, const int32_t *__restrict__ cids,
                   int32_t *__restrict__ ci)
{
    constexpr int NQ = 4 * LPR;
    constexpr int TPL = 32 / LPR;                 // tokens per warp-wide load
    constexpr int UNROLL = 8;
    const int b = blockIdx.y;
    const int lane = threadIdx.x & 31;
    const int grp = lane / LPR, sub = lane % LPR;
    const int n = n_docs[b];
    const int4 *tb = reinterpret_cast<const int4 *>(table + (int64_t)b * K * NQ) + sub;
    const int2 *rb = rng + (int64_t)b * maxc;
    int32_t *out = ci + (int64_t)b * maxc;
    const int warps_per_query = gridDim.x * CI_WARPS;
    const int per_warp = (n + warps_per_query - 1) / warps_per_query;
    const int wq = blockIdx.x * CI_WARPS + (threadIdx.x >> 5);
    const int j_begin = wq * per_warp < n ? wq * per_warp : n;
    const int j_end = j_begin + per_warp < n ? j_begin + per_warp : n;
    for (int jb = j_begin; jb < j_end; jb += 32) {
        const int cnt_docs = j_end - jb < 32 ? j_end - jb : 32;
        const int2 mine = lane < cnt_docs ? rb[jb + lane] : make_int2(0, 1);
        int my_sum = 0;
        int32_t nx_cid;
        {
            const int t0 = __shfl_sync(0xffffffffu, mine.x, 0), len = __shfl_sync(0xffffffffu, mine.y, 0);
            nx_cid = cids[DBG_TOK((int64_t)t0 + (lane < len - 1 ? lane : len - 1))];
        }
        for (int di = 0; di < cnt_docs; ++di) {
            const int t0 = __shfl_sync(0xffffffffu, mine.x, di), len = __shfl_sync(0xffffffffu, mine.y, di);
            int32_t cidv = nx_cid;
            if (di + 1 < cnt_docs) {
                const int n0 = __shfl_sync(0xffffffffu, mine.x, di + 1), nl = __shfl_sync(0xffffffffu, mine.y, di + 1);
                nx_cid = cids[DBG_TOK((int64_t)n0 + (lane < nl - 1 ? lane : nl - 1))];
            }
            int4 m = make_int4(INT_MIN, INT_MIN, INT_MIN, INT_MIN);
            for (int base = 0; base < len; base += 32) {
                const int cnt = len - base < 32 ? len - base : 32;
                // lanes past the end repeat the last token: a duplicate cannot change a maximum
                if (base != 0) cidv = cids[DBG_TOK((int64_t)t0 + base + (lane < cnt ? lane : cnt - 1))];
                for (int s = 0; s * TPL < cnt; s += UNROLL) {
                    int4 v[UNROLL];
#pragma unroll
                    for (int u = 0; u < UNROLL; ++u) {
                        int src = (s + u) * TPL + grp;
                        src = src < 32 ? src : 31;    // lane 31 holds a valid (possibly repeated) token
                        const int32_t c = __shfl_sync(0xffffffffu, cidv, src);
                        v[u] = __ldg(tb + (int64_t)DBG_CID(c) * LPR);
                    }
#pragma unroll
                    for (int u = 0; u < UNROLL; u += 2) {
                        m.x = __vimax3_s32(m.x, v[u].x, v[u + 1].x);
                        m.y = __vimax3_s32(m.y, v[u].y, v[u + 1].y);
                        m.z = __vimax3_s32(m.z, v[u].z, v[u + 1].z);
                        m.w = __vimax3_s32(m.w, v[u].w, v[u + 1].w);
                    }
                }
            }
#pragma unroll
            for (int o = LPR; o < 32; o <<= 1) {           // merge the TPL lane groups
                m.x = max(m.x, __shfl_xor_sync(0xffffffffu, m.x, o));
                m.y = max(m.y, __shfl_xor_sync(0xffffffffu, m.y, o));
                m.z = max(m.z, __shfl_xor_sync(0xffffffffu, m.z, o));
                m.w = max(m.w, __shfl_xor_sync(0xffffffffu, m.w, o));
            }
            int sum = m.x + m.y + m.z + m.w;
#pragma unroll
            for (int o = LPR >> 1; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
            sum = __shfl_sync(0xffffffffu, sum, 0);
            if (lane == di) my_sum = sum;
        }
        if (lane < cnt_docs) out[jb + lane] = my_sum;
    }
}

// ------------------------------------------------------------------------------------------------ coarse bounds --
// Bounds on CI from the 8-bit table U8[c, i] = clamp(S[c, i] >> 16, 0, 255) (stage 1 writes it next to the exact
// table): 256 buckets of width 2^16 over [0, 2^24), everything negative in bucket 0, everything from 255 * 2^16 up in
// bucket 255.  |S| <= 2^24 + 2^16 = SMAX: queries and centroids are at most unit-norm up to 2^-10 (checked where their
// fixed-point digits are made; a longer row is reported through the status word).  The map is monotone, so
// m_i = max_t U8[cid_t, i] is the bucket of the exact maximum:
//     2^16 m_i <= max_t S <= 2^16 m_i + 2^16 - 1        for 0 < m_i < 255,
// the lower end drops to -SMAX for m_i = 0 and the upper end rises to SMAX = 2^16 * 255 + 2^17 for m_i = 255.  With
// sum = sum_i m_i, zeros = #{i : m_i = 0}, sat = #{i : m_i = 255}:
//     lo(d) = 2^16 sum - zeros SMAX  <=  CI(d)  <=  2^16 sum + nq (2^16 - 1) + (2^16 + 1) sat = hi(d).
// (The scores that decide a maximum are positive -- a document token close to the query token -- so the buckets are
// spent on [0, 1) and a column whose best score is negative only loosens lo.)  A row of U8 is q_len bytes -- one
// 32-byte sector for 32 query
// tokens instead of four -- and a lane's 16-byte load covers 16 query tokens, so one warp load covers 32 / LPR tokens
// (LPR = q_len / 16 lanes per row).  The running maxima fold two rows per instruction with the three-input packed
// 16-bit integer maximum (see coarse_accumulate2).
// packed = sum | sat << 16 | zeros << 24 (see above)
__device__ __forceinline__ int32_t coarse_lo(int packed)
{
    return ((packed & 0xffff) << 16) - (packed >> 24) * ((1 << 24) + (1 << 16));
}
__device__ __forceinline__ int32_t coarse_hi(int packed, int nq)
{
    return ((packed & 0xffff) << 16) + nq * ((1 << 16) - 1) + ((packed >> 16) & 0xff) * ((1 << 16) + 1);
}
// The histogram key of a lower bound in the contender step: floor(lo / 2^16) clamped at 0 -- a valid, slightly smaller
// lower bound (documents with an empty column fall to the bottom, which only lowers the threshold).
__device__ __forceinline__ int coarse_key(int32_t lo) { return lo < 0 ? 0 : lo >> 16; }
// Running maxima of a lane's 16 columns in eight registers of two 16-bit fields each, updated from two rows at a time
// with the three-input packed 16-bit maximum.  A field compares as (column byte << 8 | whatever lies below it), so the
// winner's HIGH byte is the column's maximum and no widening is needed: the odd bytes of a word already sit in the high
// byte of a field (registers 4..7 take the raw words), the even bytes get there with one shift (registers 0..3).
// coarse_field() extracts a field's maximum at the end.
__device__ __forceinline__ void coarse_accumulate2(uint32_t (&m)[8], const int4 &va, const int4 &vb)
{
    const uint32_t a[4] = {(uint32_t)va.x, (uint32_t)va.y, (uint32_t)va.z, (uint32_t)va.w};
    const uint32_t b[4] = {(uint32_t)vb.x, (uint32_t)vb.y, (uint32_t)vb.z, (uint32_t)vb.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        m[k] = __vimax3_u16x2(m[k], a[k] << 8, b[k] << 8);
        m[4 + k] = __vimax3_u16x2(m[4 + k], a[k], b[k]);
    }
}
__device__ __forceinline__ int coarse_field_lo(uint32_t m) { return (int)((m >> 8) & 0xffu); }
__device__ __forceinline__ int coarse_field_hi(uint32_t m) { return (int)(m >> 24); }
// SMEM = true: the query's whole 8-bit table (K * q_len bytes) is first staged in shared memory and the row lookups
// are shared-memory loads (small K only); blocks are then larger (THREADS) because only one fits an SM.
template <int LPR, bool SMEM, int THREADS>
__global__ void __launch_bounds__(THREADS)
ci_coarse_kernel(const uint8_t *__restrict__ table8, int64_t K, const int32_t *__restrict__ cand,
                 const int32_t *__restrict__ n_cand, int64_t maxc, const int32_t *__restrict__ cids,
                 const int64_t *__restrict__ doc_off, int32_t *__restrict__ lo, int32_t *__restrict__ hi)
{
    extern __shared__ int4 smem_table[];
    constexpr int WARPS = THREADS / 32;
    constexpr int NQ = 16 * LPR;
    constexpr int TPL = 32 / LPR;                 // tokens per warp-wide load
    constexpr int STEPS = 32 / TPL;               // loads per 32-token slab (= LPR)
    constexpr int SLABS = 2;                      // 32-token slabs per iteration (more costs occupancy and loses)
    const int b = blockIdx.y;
    const int lane = threadIdx.x & 31;
    const int grp = lane / LPR, sub = lane % LPR;
    const int n = n_cand[b];
    const int4 *tb = reinterpret_cast<const int4 *>(table8 + (int64_t)b * K * NQ) + sub;
    if (SMEM) {
        const int4 *src = reinterpret_cast<const int4 *>(table8 + (int64_t)b * K * NQ);
        for (int64_t e = threadIdx.x; e < K * LPR; e += THREADS) smem_table[e] = __ldg(src + e);
        __syncthreads();
    }
    const int4 *ts = smem_table + sub;
    const int32_t *cb = cand + (int64_t)b * maxc;
    const int warps_per_query = gridDim.x * WARPS;
    // The chain candidate id -> token range -> first centroid ids is three dependent loads: it is issued one document
    // ahead, so it overlaps the row gathers of the current document.
    int64_t nx_t0 = 0, nx_t1 = 0;
    int32_t nx_cid[SLABS];
    auto prefetch = [&](int j) {
        const int64_t d = DBG_DOC(cb[j]);
        nx_t0 = doc_off[d];
        nx_t1 = doc_off[d + 1];
#pragma unroll
        for (int k = 0; k < SLABS; ++k) {
            const int64_t i = nx_t0 + 32 * k + lane;
            nx_cid[k] = cids[i < nx_t1 - 1 ? i : nx_t1 - 1];
        }
    };
    int j = blockIdx.x * WARPS + (threadIdx.x >> 5);
    if (j < n) prefetch(j);
    for (; j < n; j += warps_per_query) {
        const int64_t t0 = nx_t0, t1 = nx_t1;
        int32_t cid[SLABS];
#pragma unroll
        for (int k = 0; k < SLABS; ++k) cid[k] = nx_cid[k];
        if (j + warps_per_query < n) prefetch(j + warps_per_query);
        uint32_t m[8];
#pragma unroll
        for (int r = 0; r < 8; ++r) m[r] = 0u;
        for (int64_t base = t0; base < t1; base += 32 * SLABS) {
            // up to SLABS 32-token slabs per iteration, all their row loads in flight together; lanes past the end
            // repeat the last token (harmless for a maximum)
            if (base != t0) {
                const int64_t last = t1 - 1;
#pragma unroll
                for (int k = 0; k < SLABS; ++k) {
                    const int64_t i = base + 32 * k + lane;
                    cid[k] = cids[i < last ? i : last];
                }
            }
            int4 v[SLABS * STEPS];
#pragma unroll
            for (int k = 0; k < SLABS; ++k) {
                if (k == 0 || base + 32 * k < t1) {
#pragma unroll
                    for (int s = 0; s < STEPS; ++s) {
                        const int32_t c = __shfl_sync(0xffffffffu, cid[k], s * TPL + grp);
                        v[k * STEPS + s] = SMEM ? ts[DBG_CID(c) * LPR] : __ldg(tb + (int64_t)DBG_CID(c) * LPR);
                    }
                }
            }
#pragma unroll
            for (int k = 0; k < SLABS; ++k) {
                if (k == 0 || base + 32 * k < t1) {
#pragma unroll
                    for (int s = 0; s < STEPS; s += 2) coarse_accumulate2(m, v[k * STEPS + s], v[k * STEPS + s + 1]);
                }
            }
        }
        // Merge the lane groups (same columns, different tokens).  While a lane still holds several registers each
        // exchange keeps one half of them and hands the other half to the partner, so the data halves per step;
        // the remaining steps exchange the last register whole (those lanes end up with duplicates).
        int nreg = 8;
        uint32_t dup_mask = 0;
#pragma unroll
        for (int o = 16; o >= LPR; o >>= 1) {
            if (nreg > 1) {
                const int half = nreg >> 1;
                const bool up = (lane & o) != 0;
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    if (r < half) {
                        const uint32_t send = up ? m[r] : m[r + half];
                        const uint32_t keep = up ? m[r + half] : m[r];
                        m[r] = __vmaxu2(keep, __shfl_xor_sync(0xffffffffu, send, o));
                    }
                }
                nreg = half;
            } else {
                m[0] = __vmaxu2(m[0], __shfl_xor_sync(0xffffffffu, m[0], o));
                dup_mask |= (uint32_t)o;
            }
        }
        // every lane now holds the maxima of two columns; sum over columns (skipping duplicate lanes)
        const int u_lo = coarse_field_lo(m[0]), u_hi = coarse_field_hi(m[0]);
        int packed = 0;                                         // sum of maxima | saturated << 16 | zeros << 24
        if ((lane & dup_mask) == 0)
            packed = (u_lo + u_hi) + (((u_lo >= 255) + (u_hi >= 255)) << 16) + (((u_lo == 0) + (u_hi == 0)) << 24);
        packed = __reduce_add_sync(0xffffffffu, packed);        // sum <= 255 * 64 < 2^16, counts <= 64
        if (lane == 0) {
            lo[(int64_t)b * maxc + j] = coarse_lo(packed);
            hi[(int64_t)b * maxc + j] = coarse_hi(packed, NQ);
        }
    }
}

// Token range (first token, length) of every candidate, written once per search: the scan then finds a document's
// tokens with one coalesced load per 32 documents instead of the dependent chain id -> offsets per document.
__global__ void __launch_bounds__(256)
cand_range_kernel(const int32_t *__restrict__ cand, const int32_t *__restrict__ n_cand, int64_t maxc,
                  const int64_t *__restrict__ doc_off, int2 *__restrict__ rng)
{
    const int b = blockIdx.y;
    const int n = n_cand[b];
    for (int j = blockIdx.x * blockDim.x + threadIdx.x; j < n; j += gridDim.x * blockDim.x) {
        const int64_t d = DBG_DOC(cand[(int64_t)b * maxc + j]);
        const int64_t t0 = doc_off[d];
        rng[(int64_t)b * maxc + j] = make_int2((int)t0, (int)(doc_off[d + 1] - t0));
    }
}

// The bound scan over precomputed token ranges (corpora with fewer than 2^31 tokens).  A warp owns a contiguous run of
// the query's candidates and takes them 32 at a time: lane i loads the range of document i of the group (one coalesced
// load), the ranges are handed out by shuffle, and while document i is scanned the first centroid ids of document
// i + 1 are already being fetched -- a one-level prefetch where the per-document chain used to have three levels.
// The 32 results of a group are written back coalesced.
template <int LPR>
__device__ __forceinline__ void
ci_coarse_rng_body(const uint8_t *__restrict__ table8, int64_t K, const int2 *__restrict__ rng,
                     const int32_t *__restrict__ n_cand, int64_t maxc, const int32_t *__restrict__ cids,
                     int32_t *__restrict__ lo, int32_t *__restrict__ hi)
{
    constexpr int NQ = 16 * LPR;
    constexpr int TPL = 32 / LPR;                 // tokens per warp-wide load
    constexpr int STEPS = 32 / TPL;               // loads per 32-token slab (= LPR)
    // 32-token slabs per iteration, and whether the centroid ids of the document after next are pulled into L2.
    // Measured (bound scan, batch 256): for 32-byte rows one slab without that prefetch is the fastest of the four
    // combinations (Mid 14.21 ms against 14.45 ms for two slabs with it, 14.54 / 14.75 ms for the mixed ones; Large
    // 28.2 against 28.7 ms); for 64-byte rows two slabs with the prefetch are (long documents: 28.8 against 29.1 ms).
    constexpr int SLABS = LPR == 2 ? 1 : 2;
    constexpr bool PREFETCH_L2 = LPR != 2;
    const int b = blockIdx.y;
    const int lane = threadIdx.x & 31;
    const int grp = lane / LPR, sub = lane % LPR;
    const int n = n_cand[b];
    const int4 *tb = reinterpret_cast<const int4 *>(table8 + (int64_t)b * K * NQ) + sub;
    const int2 *rb = rng + (int64_t)b * maxc;
    const int warps_per_query = gridDim.x * CI_WARPS;
    const int per_warp = (n + warps_per_query - 1) / warps_per_query;
    const int wq = blockIdx.x * CI_WARPS + (threadIdx.x >> 5);
    const int j_begin = wq * per_warp < n ? wq * per_warp : n;
    const int j_end = j_begin + per_warp < n ? j_begin + per_warp : n;

    for (int jb = j_begin; jb < j_end; jb += 32) {
        const int cnt = j_end - jb < 32 ? j_end - jb : 32;
        const int2 mine = lane < cnt ? rb[jb + lane] : make_int2(0, 1);
        int my_lo = 0, my_hi = 0;
        int32_t nx_cid[SLABS];
        {
            const int t0 = __shfl_sync(0xffffffffu, mine.x, 0), len = __shfl_sync(0xffffffffu, mine.y, 0);
#pragma unroll
            for (int k = 0; k < SLABS; ++k) {
                const int i = 32 * k + lane;
                nx_cid[k] = cids[DBG_TOK((int64_t)t0 + (i < len - 1 ? i : len - 1))];
            }
        }
        for (int di = 0; di < cnt; ++di) {
            const int t0 = __shfl_sync(0xffffffffu, mine.x, di), len = __shfl_sync(0xffffffffu, mine.y, di);
            int32_t cid[SLABS];
#pragma unroll
            for (int k = 0; k < SLABS; ++k) cid[k] = nx_cid[k];
            if (PREFETCH_L2 && di + 2 < cnt) {         // two documents ahead: pull the centroid ids into L2
                const int p0 = __shfl_sync(0xffffffffu, mine.x, di + 2), pl = __shfl_sync(0xffffffffu, mine.y, di + 2);
                if (lane * 32 < pl) asm volatile("prefetch.global.L2 [%0];" ::"l"(cids + (int64_t)p0 + lane * 32));
            }
            if (di + 1 < cnt) {
                const int n0 = __shfl_sync(0xffffffffu, mine.x, di + 1), nl = __shfl_sync(0xffffffffu, mine.y, di + 1);
#pragma unroll
                for (int k = 0; k < SLABS; ++k) {
                    const int i = 32 * k + lane;
                    nx_cid[k] = cids[DBG_TOK((int64_t)n0 + (i < nl - 1 ? i : nl - 1))];
                }
            }
            uint32_t m[8];
#pragma unroll
            for (int r = 0; r < 8; ++r) m[r] = 0u;
            for (int base = 0; base < len; base += 32 * SLABS) {
                // lanes past the end repeat the last token (harmless for a maximum)
                int4 v[SLABS * STEPS];
#pragma unroll
                for (int k = 0; k < SLABS; ++k) {
                    if (k == 0 || base + 32 * k < len) {
#pragma unroll
                        for (int s = 0; s < STEPS; ++s) {
                            const int32_t c = __shfl_sync(0xffffffffu, cid[k], s * TPL + grp);
                            v[k * STEPS + s] = __ldg(tb + (int64_t)DBG_CID(c) * LPR);
                        }
                    }
                }
                // the centroid ids of the next iteration travel while this iteration's rows do
                if (base + 32 * SLABS < len) {
#pragma unroll
                    for (int k = 0; k < SLABS; ++k) {
                        const int i = base + 32 * SLABS + 32 * k + lane;
                        cid[k] = cids[DBG_TOK((int64_t)t0 + (i < len - 1 ? i : len - 1))];
                    }
                }
#pragma unroll
                for (int k = 0; k < SLABS; ++k) {
                    if (k == 0 || base + 32 * k < len) {
#pragma unroll
                        for (int s = 0; s < STEPS; s += 2)
                            coarse_accumulate2(m, v[k * STEPS + s], v[k * STEPS + s + 1]);
                    }
                }
            }
            // merge the lane groups (same columns, different tokens): each exchange keeps one half of the registers
            int nreg = 8;
            uint32_t dup_mask = 0;
#pragma unroll
            for (int o = 16; o >= LPR; o >>= 1) {
                if (nreg > 1) {
                    const int half = nreg >> 1;
                    const bool up = (lane & o) != 0;
#pragma unroll
                    for (int r = 0; r < 4; ++r) {
                        if (r < half) {
                            const uint32_t send = up ? m[r] : m[r + half];
                            const uint32_t keep = up ? m[r + half] : m[r];
                            m[r] = __vmaxu2(keep, __shfl_xor_sync(0xffffffffu, send, o));
                        }
                    }
                    nreg = half;
                } else {
                    m[0] = __vmaxu2(m[0], __shfl_xor_sync(0xffffffffu, m[0], o));
                    dup_mask |= (uint32_t)o;
                }
            }
            const int u_lo = coarse_field_lo(m[0]), u_hi = coarse_field_hi(m[0]);
            int packed = 0;                                         // sum of maxima | saturated << 16 | zeros << 24
            if ((lane & dup_mask) == 0)
                packed = (u_lo + u_hi) + (((u_lo >= 255) + (u_hi >= 255)) << 16) + (((u_lo == 0) + (u_hi == 0)) << 24);
            packed = __reduce_add_sync(0xffffffffu, packed);
            if (lane == di) {                                       // lane di keeps the result of document di
                my_lo = coarse_lo(packed);
                my_hi = coarse_hi(packed, NQ);
            }
        }
        if (lane < cnt) {
            lo[(int64_t)b * maxc + jb + lane] = my_lo;
            hi[(int64_t)b * maxc + jb + lane] = my_hi;
        }
    }
}

// Two launch forms of the scan.  32-byte rows: no occupancy hint (the compiler's own 64 registers, four blocks per SM;
// any hint measured slower).  64-byte rows: four blocks per SM instead of the three that the unhinted 75 registers
// give (long-document corpus: 27.1 against 28.4 ms).
template <int LPR>
__global__ void __launch_bounds__(CI_THREADS)
ci_coarse_rng_kernel(const uint8_t *__restrict__ table8, int64_t K, const int2 *__restrict__ rng,
                     const int32_t *__restrict__ n_cand, int64_t maxc, const int32_t *__restrict__ cids,
                     int32_t *__restrict__ lo, int32_t *__restrict__ hi)
{
    ci_coarse_rng_body<LPR>(table8, K, rng, n_cand, maxc, cids, lo, hi);
}
template <int LPR>
__global__ void __launch_bounds__(CI_THREADS, 4)
ci_coarse_rng_kernel_b4(const uint8_t *__restrict__ table8, int64_t K, const int2 *__restrict__ rng,
                        const int32_t *__restrict__ n_cand, int64_t maxc, const int32_t *__restrict__ cids,
                        int32_t *__restrict__ lo, int32_t *__restrict__ hi)
{
    ci_coarse_rng_body<LPR>(table8, K, rng, n_cand, maxc, cids, lo, hi);
}

bool coarse_supported(int nq) { return nq == 32 || nq == 64; }

int launch_coarse_bounds(const Index &ix, const Params &p, const uint8_t *table8, const int32_t *cand,
                         const int32_t *n_cand, int32_t *lo, int32_t *hi, int2 *rng, cudaStream_t st)
{
    const size_t table_bytes = (size_t)ix.K * p.nq;
    // the candidates' token ranges, for this scan and for the exact scoring of the contenders afterwards
    const bool use_rng = ix.T < 0x7fffffffLL && rng != nullptr;
    if (use_rng) {
        int64_t rb = ((int64_t)ix.sm_count * 8 + p.B - 1) / p.B;
        const int64_t rwant = (p.maxc + 255) / 256;
        if (rb > rwant) rb = rwant;
        if (rb < 1) rb = 1;
        cand_range_kernel<<<dim3((unsigned)rb, (unsigned)p.B), 256, 0, st>>>(cand, n_cand, p.maxc, ix.doc_off, rng);
        CHIMERA_CUDA(cudaGetLastError());
        count_launch(SLOT_CI);
    }
    if (table_bytes <= 160 * 1024) {
        // the whole 8-bit table of a query fits in shared memory: stage it once per block and look rows up there
        constexpr int T = 512;
        int64_t gx = (4LL * ix.sm_count + p.B - 1) / p.B;       // every block re-reads the table: few, long blocks
        int64_t want = (p.maxc + T / 32 - 1) / (T / 32);
        if (gx > want) gx = want;
        if (gx > 64) gx = 64;
        if (gx < 1) gx = 1;
        dim3 grid((unsigned)gx, (unsigned)p.B);
        if (p.nq == 32) {
            CHIMERA_CUDA(cudaFuncSetAttribute(ci_coarse_kernel<2, true, T>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)table_bytes));
            ci_coarse_kernel<2, true, T><<<grid, T, table_bytes, st>>>(table8, ix.K, cand, n_cand, p.maxc, ix.cids,
                                                                       ix.doc_off, lo, hi);
        } else {
            CHIMERA_CUDA(cudaFuncSetAttribute(ci_coarse_kernel<4, true, T>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)table_bytes));
            ci_coarse_kernel<4, true, T><<<grid, T, table_bytes, st>>>(table8, ix.K, cand, n_cand, p.maxc, ix.cids,
                                                                       ix.doc_off, lo, hi);
        }
        CHIMERA_CUDA(cudaGetLastError());
        count_launch(SLOT_CI);
        return CHIMERA_OK;
    }
    // Blocks per query.  Four blocks are resident per SM and the blocks of a query are adjacent in the grid, so
    // (resident blocks) / (blocks per query) queries are scanned at the same time and their 8-bit tables compete for
    // L2: enough blocks per query to keep those tables within COARSE_L2_TABLES bytes, at least enough to fill the GPU
    // when the batch is small, never more than one warp per candidate.  Measured on the Mid corpus at batch 256
    // (2 MB tables): 4 blocks per query 57 ms, 16: 23.4, 24: 18.9, 37: 16.5, 74: 16.6, 148: 16.7, 1184: 17.6; a budget
    // of 16 MB against 32 MB: Mid 16.56 / 16.52 ms, Large (8 MB tables) 36.6 / 37.2 ms; 64 MB: 21.3 and 46.7 ms.
    constexpr int64_t COARSE_L2_TABLES = 16LL << 20;
    const int64_t resident = 4LL * ix.sm_count;
    const int64_t want = (p.maxc + CI_WARPS - 1) / CI_WARPS;
    int64_t per_query = (resident * (int64_t)table_bytes + COARSE_L2_TABLES - 1) / COARSE_L2_TABLES;
    const int64_t to_fill = (2 * resident + p.B - 1) / p.B;      // two waves when the batch is small
    if (per_query < to_fill) per_query = to_fill;
    if (per_query > want) per_query = want;
    if (per_query < 1) per_query = 1;
    const unsigned gx = (unsigned)per_query;
    dim3 grid(gx, (unsigned)p.B);
    if (use_rng) {
        if (p.nq == 32)
            ci_coarse_rng_kernel<2><<<grid, CI_THREADS, 0, st>>>(table8, ix.K, rng, n_cand, p.maxc, ix.cids, lo, hi);
        else
            ci_coarse_rng_kernel_b4<4><<<grid, CI_THREADS, 0, st>>>(table8, ix.K, rng, n_cand, p.maxc, ix.cids, lo, hi);
        CHIMERA_CUDA(cudaGetLastError());
        count_launch(SLOT_CI);
        return CHIMERA_OK;
    }
    if (p.nq == 32)
        ci_coarse_kernel<2, false, CI_THREADS><<<grid, CI_THREADS, 0, st>>>(table8, ix.K, cand, n_cand, p.maxc, ix.cids,
                                                                          ix.doc_off, lo, hi);
    else
        ci_coarse_kernel<4, false, CI_THREADS><<<grid, CI_THREADS, 0, st>>>(table8, ix.K, cand, n_cand, p.maxc, ix.cids,
                                                                          ix.doc_off, lo, hi);
    CHIMERA_CUDA(cudaGetLastError());
    count_launch(SLOT_CI);
    return CHIMERA_OK;
}

// table [rows] int32 -> table8 [rows] uint8 (only needed when stage 1 did not run in this call).
__global__ void coarse_table_kernel(const int32_t *__restrict__ table, int64_t n, uint8_t *__restrict__ table8)
{
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) {
        const int v = table[i] >> 16;
        table8[i] = (uint8_t)(v < 0 ? 0 : v > 255 ? 255 : v);
    }
}
int launch_coarse_table(const Index &ix, const Params &p, const int32_t *table, uint8_t *table8, cudaStream_t st)
{
    const int64_t n = (int64_t)p.B * ix.K * p.nq;
    coarse_table_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(table, n, table8);
    CHIMERA_CUDA(cudaGetLastError());
    count_launch(SLOT_MISC);
    return CHIMERA_OK;
}

// Exact CI of a list of documents.  blocks_cap bounds the blocks per query (0 = default).
int launch_centroid_interaction(const Index &ix, const Params &p, const int32_t *table, const int32_t *cand,
                                const int32_t *n_cand, int32_t *ci, int blocks_cap, int slot, const int2 *rng,
                                cudaStream_t st)
{
    int64_t want = (p.maxc + CI_WARPS - 1) / CI_WARPS;
    int64_t cap = blocks_cap > 0 ? blocks_cap : (int64_t)ix.sm_count * 8;
    unsigned gx = (unsigned)(want < cap ? want : cap);
    if (gx < 1) gx = 1;
    dim3 grid(gx, (unsigned)p.B);
    const int nqw = (p.nq + 31) / 32;
    if (rng != nullptr && (p.nq == 32 || p.nq == 64)) {       // the listed documents' token ranges are known
        if (p.nq == 32)
            ci_wide_rng_kernel<8><<<grid, CI_THREADS, 0, st>>>(table, ix.K, rng, n_cand, p.maxc, ix.cids, ci);
        else
            ci_wide_rng_kernel<16><<<grid, CI_THREADS, 0, st>>>(table, ix.K, rng, n_cand, p.maxc, ix.cids, ci);
        CHIMERA_CUDA(cudaGetLastError());
        count_launch(slot);
        return CHIMERA_OK;
    }
    if (p.nq == 32)
        ci_wide_kernel<8><<<grid, CI_THREADS, 0, st>>>(table, ix.K, cand, n_cand, p.maxc, ix.cids, ix.doc_off, ci);
    else if (p.nq == 64)
        ci_wide_kernel<16><<<grid, CI_THREADS, 0, st>>>(table, ix.K, cand, n_cand, p.maxc, ix.cids, ix.doc_off, ci);
    else if (nqw == 1)
        ci_kernel<1><<<grid, CI_THREADS, 0, st>>>(table, ix.K, p.nq, cand, n_cand, p.maxc, ix.cids, ix.doc_off, ci);
    else if (nqw == 2)
        ci_kernel<2><<<grid, CI_THREADS, 0, st>>>(table, ix.K, p.nq, cand, n_cand, p.maxc, ix.cids, ix.doc_off, ci);
    else
        ci_kernel<4><<<grid, CI_THREADS, 0, st>>>(table, ix.K, p.nq, cand, n_cand, p.maxc, ix.cids, ix.doc_off, ci);
    CHIMERA_CUDA(cudaGetLastError());
    count_launch(slot);
    return CHIMERA_OK;
}

// ------------------------------------------------------------------------------------------------ selection ------
constexpr int SEL_THREADS = 1024;

// Exclusive prefix sum over the block (SEL_THREADS threads); *total gets the block sum.  Two barriers.
__device__ __forceinline__ int sel_block_scan(int v, int *total, int *warp_part /* [32] */)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    __syncthreads();                     // warp_part may still be read from a previous call
    if (lane == 31) warp_part[warp] = incl;
    __syncthreads();
    int pw = warp_part[lane];            // 32 warps
    int pincl = pw;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, pincl, o);
        if (lane >= o) pincl += t;
    }
    *total = __shfl_sync(0xffffffffu, pincl, 31);
    int before = __shfl_sync(0xffffffffu, pincl - pw, warp);
    return before + incl - v;
}

// Radix select (11 + 11 + 10 bits, most significant first) of the `want`-th largest value of sb[0..n) in the order of
// u = value ^ 0x80000000.  Needs n >= want >= 1.  Returns that value's u; *need_eq = how many entries equal to it
// belong to the top `want` (the rest of the top `want` are strictly greater).  Whole block, uniform.
template <class Load>     // load(j) = value j (int32)
__device__ __forceinline__ uint32_t radix_select(Load load, int n, int want_in, int *hist, int *warp_part,
                                                 uint32_t *s_prefix, int *s_want, int *need_eq)
{
    if (threadIdx.x == 0) { *s_prefix = 0u; *s_want = want_in; }
    const int shifts[3] = {21, 10, 0};
    const int widths[3] = {11, 11, 10};
    uint32_t known_mask = 0u;
    for (int pass = 0; pass < 3; ++pass) {
        const int shift = shifts[pass], bins = 1 << widths[pass];
        for (int i = threadIdx.x; i < 2048; i += SEL_THREADS) hist[i] = 0;
        __syncthreads();
        const uint32_t prefix = *s_prefix;
        const int want = *s_want;
        // eight independent loads per thread before their histogram updates (the loop is latency-bound otherwise)
        for (int base = 0; base < n; base += 8 * SEL_THREADS) {
            uint32_t u[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const int j = base + e * SEL_THREADS + threadIdx.x;
                u[e] = j < n ? ((uint32_t)load(j) ^ 0x80000000u) : 0u;
            }
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const int j = base + e * SEL_THREADS + threadIdx.x;
                if (j < n && (u[e] & known_mask) == prefix) atomicAdd(&hist[(u[e] >> shift) & (bins - 1)], 1);
            }
        }
        __syncthreads();
        // descending bins: thread t owns bins (bins-1-2t) and (bins-2-2t)
        int hi_bin = bins - 1 - 2 * (int)threadIdx.x, lo_bin = hi_bin - 1;
        int h_hi = hi_bin >= 0 ? hist[hi_bin] : 0;
        int h_lo = lo_bin >= 0 ? hist[lo_bin] : 0;
        int total;
        int before = sel_block_scan(h_hi + h_lo, &total, warp_part);
        // the wanted rank falls in the first bin whose cumulative count reaches `want`
        if (before < want && want <= before + h_hi + h_lo) {
            if (want <= before + h_hi) {
                *s_prefix = prefix | ((uint32_t)hi_bin << shift);
                *s_want = want - before;
            } else {
                *s_prefix = prefix | ((uint32_t)lo_bin << shift);
                *s_want = want - before - h_hi;
            }
        }
        known_mask |= (uint32_t)(bins - 1) << shift;
        __syncthreads();
    }
    *need_eq = *s_want;
    return *s_prefix;
}

// grid (B).  pruned[b][0..n_prune) ascending ids, -1 padded; n_pruned[b]; pruned_ci (optional): the score of each
// kept document, INT_MIN beside every -1.
__global__ void __launch_bounds__(SEL_THREADS)
select_kernel(const int32_t *__restrict__ cand, const int32_t *__restrict__ n_cand, const int32_t *__restrict__ ci,
              int64_t maxc, int n_prune, int32_t *__restrict__ pruned, int32_t *__restrict__ n_pruned,
              int32_t *__restrict__ pruned_ci)
{
    __shared__ int hist[2048];
    __shared__ int warp_part[32];
    __shared__ uint32_t s_prefix;
    __shared__ int s_want;
    const int b = blockIdx.x;
    const int n = n_cand[b];
    const int32_t *cb = cand + (int64_t)b * maxc;
    const int32_t *sb = ci + (int64_t)b * maxc;
    int32_t *out = pruned + (int64_t)b * n_prune;
    int32_t *out_ci = pruned_ci ? pruned_ci + (int64_t)b * n_prune : nullptr;

    if (n <= n_prune) {
        for (int j = threadIdx.x; j < n_prune; j += SEL_THREADS) {
            out[j] = j < n ? cb[j] : -1;
            if (out_ci) out_ci[j] = j < n ? sb[j] : INT_MIN;
        }
        if (threadIdx.x == 0) n_pruned[b] = n;
        return;
    }
    int need_eq;
    const uint32_t thr = radix_select([&](int j) { return sb[j]; }, n, n_prune, hist, warp_part, &s_prefix, &s_want,
                                      &need_eq);

    // Ordered compaction: keep u > thr, and the first need_eq entries with u == thr.  Each thread owns four
    // consecutive entries per round, so one block scan covers 4096 entries.
    int run_gt = 0, run_eq = 0;
    for (int base = 0; base < n; base += 4 * SEL_THREADS) {
        const int j0 = base + 4 * threadIdx.x;
        uint32_t u[4];
        int32_t id[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int j = j0 + e;
            u[e] = j < n ? ((uint32_t)sb[j] ^ 0x80000000u) : 0u;
            id[e] = j < n ? cb[j] : 0;
        }
        int gt = 0, eq = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            gt += (j0 + e < n && u[e] > thr) ? 1 : 0;
            eq += (j0 + e < n && u[e] == thr) ? 1 : 0;
        }
        int total;
        const int before = sel_block_scan((gt << 16) | eq, &total, warp_part);   // <= 4096 per field
        int gt_before = run_gt + (before >> 16), eq_before = run_eq + (before & 0xffff);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (j0 + e >= n) break;
            const bool is_gt = u[e] > thr, is_eq = u[e] == thr;
            if (is_gt || (is_eq && eq_before < need_eq)) {
                const int pos = gt_before + (eq_before < need_eq ? eq_before : need_eq);
                out[pos] = id[e];
                if (out_ci) out_ci[pos] = (int32_t)(u[e] ^ 0x80000000u);
            }
            gt_before += is_gt ? 1 : 0;
            eq_before += is_eq ? 1 : 0;
        }
        run_gt += total >> 16;
        run_eq += total & 0xffff;
    }
    if (threadIdx.x == 0) n_pruned[b] = n_prune;
}

// grid (B).  Contenders for the top n_prune: with tau = the n_prune-th largest lower bound, every document of the
// true top n_prune has hi >= CI >= (n_prune-th largest CI) >= tau.  Writes their ids (ascending) and their number.
// The lower bounds are lo = 2^16 sum - zeros (2^24 + 64) with sum = the sum of nq 8-bit maxima (coarse_lo), so
// coarse_key(lo) = floor(lo / 2^16), clamped at 0, is a key of at most 14 bits and 2^16 key <= lo: one histogram sweep
// over CONT_BINS bins (two neighbouring keys share a bin for q_len 64; tau is then the smaller of the two, still a
// valid lower threshold) finds tau without radix passes.
constexpr int CONT_BINS = 8192;
__global__ void __launch_bounds__(SEL_THREADS)
contender_kernel(const int32_t *__restrict__ cand, const int32_t *__restrict__ n_cand, const int32_t *__restrict__ lo,
                 const int32_t *__restrict__ hi, int64_t maxc, int n_prune, int nq, int32_t *__restrict__ cont,
                 int32_t *__restrict__ n_cont, const int2 *__restrict__ rng, int2 *__restrict__ cont_rng)
{
    __shared__ int hist[CONT_BINS];
    __shared__ int warp_part[32];
    __shared__ int s_bin;
    const int b = blockIdx.x;
    const int n = n_cand[b];
    const int32_t *cb = cand + (int64_t)b * maxc;
    const int32_t *lb = lo + (int64_t)b * maxc;
    const int32_t *hb = hi + (int64_t)b * maxc;
    int32_t *out = cont + (int64_t)b * maxc;
    const int2 *rb = rng ? rng + (int64_t)b * maxc : nullptr;
    int2 *orng = cont_rng ? cont_rng + (int64_t)b * maxc : nullptr;
    if (n <= n_prune) {
        for (int j = threadIdx.x; j < n; j += SEL_THREADS) {
            out[j] = cb[j];
            if (orng) orng[j] = rb[j];
        }
        if (threadIdx.x == 0) n_cont[b] = n;
        return;
    }
    const int bin_shift = 255 * nq < CONT_BINS ? 0 : 1;            // q_len 32: one sum per bin; q_len 64: two
    for (int i = threadIdx.x; i < CONT_BINS; i += SEL_THREADS) hist[i] = 0;
    __syncthreads();
    for (int base = 0; base < n; base += 16 * SEL_THREADS) {
        int32_t v[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) {
            const int j = base + e * SEL_THREADS + threadIdx.x;
            v[e] = j < n ? lb[j] : 0;
        }
#pragma unroll
        for (int e = 0; e < 16; ++e) {
            const int j = base + e * SEL_THREADS + threadIdx.x;
            if (j < n) atomicAdd(&hist[coarse_key(v[e]) >> bin_shift], 1);
        }
    }
    __syncthreads();
    // descending bins, CONT_BINS / SEL_THREADS consecutive bins per thread
    constexpr int PER = CONT_BINS / SEL_THREADS;
    const int first_bin = CONT_BINS - 1 - PER * (int)threadIdx.x;  // this thread owns first_bin, first_bin - 1, ...
    int h[PER], mine = 0;
#pragma unroll
    for (int e = 0; e < PER; ++e) { h[e] = hist[first_bin - e]; mine += h[e]; }
    int total;
    int before = sel_block_scan(mine, &total, warp_part);
    if (before < n_prune && n_prune <= before + mine) {
#pragma unroll
        for (int e = 0; e < PER; ++e) {
            if (before < n_prune && n_prune <= before + h[e]) s_bin = first_bin - e;
            before += h[e];
        }
    }
    __syncthreads();
    const int32_t tau = (s_bin << bin_shift) << 16;                 // smallest lower bound of that bin
    // ordered compaction, eight consecutive entries per thread and round (one block scan per 8192 entries); the ids
    // are only read for the few entries that are kept
    int run = 0;
    for (int base = 0; base < n; base += 8 * SEL_THREADS) {
        const int j0 = base + 8 * threadIdx.x;
        int32_t hv[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) hv[e] = j0 + e < n ? hb[j0 + e] : INT_MIN;
        int keep = 0;
#pragma unroll
        for (int e = 0; e < 8; ++e) keep += (j0 + e < n && hv[e] >= tau) ? 1 : 0;
        int tot;
        int pos = run + sel_block_scan(keep, &tot, warp_part);
#pragma unroll
        for (int e = 0; e < 8; ++e)
            if (j0 + e < n && hv[e] >= tau) {
                out[pos] = cb[j0 + e];
                if (orng) orng[pos] = rb[j0 + e];
                ++pos;
            }
        run += tot;
    }
    if (threadIdx.x == 0) n_cont[b] = run;
}

// Document-sharded search, grid (B): the global top n_prune of the shards' local top-n_prune lists.  all_ids / all_ci
// are [world][B][n_prune] (global document ids ascending within a shard, -1 / INT_MIN padded); shards own ascending,
// disjoint id ranges in rank order, so walking rank by rank visits the valid entries in ascending id order and ties
// resolve towards the smaller id exactly as in select_kernel.  Of the selected documents this shard keeps its own
// (ids in [doc_base, doc_base + n_local)) as local ids: pruned[b][0..n_prune) ascending, -1 padded; n_pruned[b].
__global__ void __launch_bounds__(SEL_THREADS)
shard_select_kernel(const int32_t *__restrict__ all_ids, const int32_t *__restrict__ all_ci, int world, int B,
                    int n_prune, long long doc_base, long long n_local, int32_t *__restrict__ pruned,
                    int32_t *__restrict__ n_pruned)
{
    __shared__ int hist[2048];
    __shared__ int warp_part[32];
    __shared__ uint32_t s_prefix;
    __shared__ int s_want;
    const int b = blockIdx.x;
    const int n = world * n_prune;
    auto at = [&](int j) { return ((int64_t)(j / n_prune) * B + b) * n_prune + j % n_prune; };
    int32_t *out = pruned + (int64_t)b * n_prune;

    // number of valid entries
    int valid = 0;
    for (int j = threadIdx.x; j < n; j += SEL_THREADS) valid += all_ids[at(j)] >= 0 ? 1 : 0;
    int total_valid;
    sel_block_scan(valid, &total_valid, warp_part);
    uint32_t thr = 0u;              // keep everything valid
    int need_eq = 0;
    if (total_valid > n_prune)
        thr = radix_select([&](int j) { return all_ci[at(j)]; }, n, n_prune, hist, warp_part, &s_prefix, &s_want,
                           &need_eq);
    const bool keep_all = total_valid <= n_prune;

    int run_eq = 0, run_own = 0;
    for (int base = 0; base < n; base += 4 * SEL_THREADS) {
        const int j0 = base + 4 * threadIdx.x;
        uint32_t u[4];
        int32_t id[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int j = j0 + e;
            id[e] = j < n ? all_ids[at(j)] : -1;
            u[e] = id[e] >= 0 ? ((uint32_t)all_ci[at(j)] ^ 0x80000000u) : 0u;
        }
        int eq = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) eq += (id[e] >= 0 && !keep_all && u[e] == thr) ? 1 : 0;
        int total_eq;
        int eq_before = run_eq + sel_block_scan(eq, &total_eq, warp_part);
        bool own[4];
        int n_own = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            bool kept = id[e] >= 0;
            if (kept && !keep_all) {
                const bool is_eq = u[e] == thr;
                kept = u[e] > thr || (is_eq && eq_before < need_eq);
                eq_before += is_eq ? 1 : 0;
            }
            own[e] = kept && id[e] >= doc_base && id[e] < doc_base + n_local;
            n_own += own[e] ? 1 : 0;
        }
        int total_own;
        int pos = run_own + sel_block_scan(n_own, &total_own, warp_part);
#pragma unroll
        for (int e = 0; e < 4; ++e)
            if (own[e]) out[pos++] = (int32_t)(id[e] - doc_base);
        run_eq += total_eq;
        run_own += total_own;
    }
    for (int j = run_own + threadIdx.x; j < n_prune; j += SEL_THREADS) out[j] = -1;
    if (threadIdx.x == 0) n_pruned[b] = run_own;
}

int launch_shard_select(const Params &p, const int32_t *all_ids, const int32_t *all_ci, int world, int64_t doc_base,
                        int64_t n_local, int32_t *pruned, int32_t *n_pruned, cudaStream_t st)
{
    shard_select_kernel<<<(unsigned)p.B, SEL_THREADS, 0, st>>>(all_ids, all_ci, world, p.B, p.n_prune,
                                                               (long long)doc_base, (long long)n_local, pruned,
                                                               n_pruned);
    CHIMERA_CUDA(cudaGetLastError());
    count_launch(SLOT_SELECT);
    return CHIMERA_OK;
}

// The same selection spread over CONT_SPLIT blocks per query, for calls with few queries: one block reads its arrays
// at one SM's bandwidth (about 40 us for 100k candidates), which is most of the stage's latency when a single query is
// served.  Three kernels: slice histograms added into a global one; every block finds tau from it and counts its
// slice's contenders; every block writes its contenders behind those of the slices before it (ascending ids kept).
// Scratch: `scratch[b * maxc ...]` holds the histogram (CONT_BINS), the slice counts (CONT_SPLIT) and tau.
constexpr int CONT_SPLIT = 32;

__device__ __forceinline__ void cont_slice(int n, int g, int *j0, int *j1)
{
    const int per = (n + CONT_SPLIT - 1) / CONT_SPLIT;
    *j0 = g * per < n ? g * per : n;
    *j1 = (g + 1) * per < n ? (g + 1) * per : n;
}

__global__ void __launch_bounds__(SEL_THREADS)
contender_hist_kernel(const int32_t *__restrict__ n_cand, const int32_t *__restrict__ lo, int64_t maxc, int n_prune,
                      int nq, int32_t *__restrict__ scratch)
{
    __shared__ int hist[CONT_BINS];
    const int b = blockIdx.y, n = n_cand[b];
    if (n <= n_prune) return;                          // everything is a contender: no threshold needed
    int j0, j1;
    cont_slice(n, blockIdx.x, &j0, &j1);
    const int32_t *lb = lo + (int64_t)b * maxc;
    const int bin_shift = 255 * nq < CONT_BINS ? 0 : 1;
    for (int i = threadIdx.x; i < CONT_BINS; i += SEL_THREADS) hist[i] = 0;
    __syncthreads();
    for (int j = j0 + threadIdx.x; j < j1; j += SEL_THREADS)
        atomicAdd(&hist[coarse_key(lb[j]) >> bin_shift], 1);
    __syncthreads();
    int32_t *gh = scratch + (int64_t)b * maxc;
    for (int i = threadIdx.x; i < CONT_BINS; i += SEL_THREADS)
        if (hist[i]) atomicAdd(&gh[i], hist[i]);
}

__global__ void __launch_bounds__(SEL_THREADS)
contender_count_kernel(const int32_t *__restrict__ n_cand, const int32_t *__restrict__ hi, int64_t maxc, int n_prune,
                       int nq, int32_t *__restrict__ scratch)
{
    __shared__ int warp_part[32];
    __shared__ int s_bin;
    const int b = blockIdx.y, n = n_cand[b];
    int32_t *gh = scratch + (int64_t)b * maxc;
    int32_t tau = INT_MIN;
    if (n > n_prune) {
        const int bin_shift = 255 * nq < CONT_BINS ? 0 : 1;
        constexpr int PER = CONT_BINS / SEL_THREADS;
        const int first_bin = CONT_BINS - 1 - PER * (int)threadIdx.x;
        int h[PER], mine = 0;
#pragma unroll
        for (int e = 0; e < PER; ++e) { h[e] = gh[first_bin - e]; mine += h[e]; }
        int total;
        int before = sel_block_scan(mine, &total, warp_part);
        if (before < n_prune && n_prune <= before + mine) {
#pragma unroll
            for (int e = 0; e < PER; ++e) {
                if (before < n_prune && n_prune <= before + h[e]) s_bin = first_bin - e;
                before += h[e];
            }
        }
        __syncthreads();
        tau = (s_bin << bin_shift) << 16;
    }
    int j0, j1;
    cont_slice(n, blockIdx.x, &j0, &j1);
    const int32_t *hb = hi + (int64_t)b * maxc;
    int keep = 0;
    for (int j = j0 + threadIdx.x; j < j1; j += SEL_THREADS) keep += hb[j] >= tau ? 1 : 0;
    int total;
    sel_block_scan(keep, &total, warp_part);
    if (threadIdx.x == 0) {
        gh[CONT_BINS + blockIdx.x] = total;
        if (blockIdx.x == 0) gh[CONT_BINS + CONT_SPLIT] = tau;
    }
}

__global__ void __launch_bounds__(SEL_THREADS)
contender_write_kernel(const int32_t *__restrict__ cand, const int32_t *__restrict__ n_cand,
                       const int32_t *__restrict__ hi, int64_t maxc, const int32_t *__restrict__ scratch,
                       int32_t *__restrict__ cont, int32_t *__restrict__ n_cont, const int2 *__restrict__ rng,
                       int2 *__restrict__ cont_rng)
{
    __shared__ int warp_part[32];
    const int b = blockIdx.y, n = n_cand[b], g = blockIdx.x;
    const int32_t *gh = scratch + (int64_t)b * maxc;
    const int32_t tau = gh[CONT_BINS + CONT_SPLIT];
    int offset = 0;
    for (int s = 0; s < g; ++s) offset += gh[CONT_BINS + s];
    int j0, j1;
    cont_slice(n, g, &j0, &j1);
    const int32_t *cb = cand + (int64_t)b * maxc;
    const int32_t *hb = hi + (int64_t)b * maxc;
    int32_t *out = cont + (int64_t)b * maxc;
    const int2 *rb = rng ? rng + (int64_t)b * maxc : nullptr;
    int2 *orng = cont_rng ? cont_rng + (int64_t)b * maxc : nullptr;
    int run = offset;
    for (int base = j0; base < j1; base += 4 * SEL_THREADS) {
        const int q0 = base + 4 * threadIdx.x;
        int32_t hv[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) hv[e] = q0 + e < j1 ? hb[q0 + e] : INT_MIN;
        int keep = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) keep += (q0 + e < j1 && hv[e] >= tau) ? 1 : 0;
        int tot;
        int pos = run + sel_block_scan(keep, &tot, warp_part);
#pragma unroll
        for (int e = 0; e < 4; ++e)
            if (q0 + e < j1 && hv[e] >= tau) {
                out[pos] = cb[q0 + e];
                if (orng) orng[pos] = rb[q0 + e];
                ++pos;
            }
        run += tot;
    }
    if (g == CONT_SPLIT - 1 && threadIdx.x == 0) n_cont[b] = run;
}

// scratch: an int32 [B][maxc] array that is free during this step (the exact-CI output buffer).
int launch_contenders(const Index &ix, const Params &p, const int32_t *cand, const int32_t *n_cand, const int32_t *lo,
                      const int32_t *hi, int32_t *cont, int32_t *n_cont, int32_t *scratch, const int2 *rng,
                      int2 *cont_rng, cudaStream_t st)
{
    if (ix.T >= 0x7fffffffLL) { rng = nullptr; cont_rng = nullptr; }      // the bound scan wrote no ranges
    if (4 * p.B <= ix.sm_count && p.maxc >= CONT_BINS + CONT_SPLIT + 1) {
        // few queries: CONT_SPLIT blocks each
        CHIMERA_CUDA(cudaMemset2DAsync(scratch, sizeof(int32_t) * (size_t)p.maxc, 0, sizeof(int32_t) * CONT_BINS,
                                       (size_t)p.B, st));
        const dim3 grid(CONT_SPLIT, (unsigned)p.B);
        contender_hist_kernel<<<grid, SEL_THREADS, 0, st>>>(n_cand, lo, p.maxc, p.n_prune, p.nq, scratch);
        CHIMERA_CUDA(cudaGetLastError());
        contender_count_kernel<<<grid, SEL_THREADS, 0, st>>>(n_cand, hi, p.maxc, p.n_prune, p.nq, scratch);
        CHIMERA_CUDA(cudaGetLastError());
        contender_write_kernel<<<grid, SEL_THREADS, 0, st>>>(cand, n_cand, hi, p.maxc, scratch, cont, n_cont, rng, cont_rng);
        CHIMERA_CUDA(cudaGetLastError());
        count_launch(SLOT_SELECT, 3);
        return CHIMERA_OK;
    }
    contender_kernel<<<(unsigned)p.B, SEL_THREADS, 0, st>>>(cand, n_cand, lo, hi, p.maxc, p.n_prune, p.nq, cont,
                                                            n_cont, rng, cont_rng);
    CHIMERA_CUDA(cudaGetLastError());
    count_launch(SLOT_SELECT);
    return CHIMERA_OK;
}

// ------------------------------------------------------------------------------------------------------------------
// The same selection spread over SELS_SPLIT blocks per query, for calls with few queries (one block reads its arrays at
// one SM's bandwidth; with a single query that is most of the stage's latency).  Five kernels, each block working on a
// contiguous slice of the candidates: three radix passes whose slice histograms are added into global ones (every block
// of the next kernel re-derives the chosen digit from the global histogram, which is cheap), a count of the entries
// above and at the threshold per slice, and the ordered write behind the slices before it.
// Scratch per query (int32): hist[0] 2048, hist[1] 2048, hist[2] 1024, greater[SELS_SPLIT], equal[SELS_SPLIT].
constexpr int SELS_SPLIT = 32;
constexpr int SELS_SCRATCH = 2048 + 2048 + 1024 + 2 * SELS_SPLIT;

__device__ __forceinline__ void sels_slice(int n, int g, int *j0, int *j1)
{
    const int per = (n + SELS_SPLIT - 1) / SELS_SPLIT;
    *j0 = g * per < n ? g * per : n;
    *j1 = (g + 1) * per < n ? (g + 1) * per : n;
}

// The digit (bin) of `bins` descending-cumulative bins that holds rank `want`, and the rank left inside it.
// Whole block, uniform result.
__device__ __forceinline__ void sels_find(const int32_t *__restrict__ hist, int bins, int want, int *warp_part,
                                          int *s_out /* [2] */, int *bin, int *want_rest)
{
    const int hi_bin = bins - 1 - 2 * (int)threadIdx.x, lo_bin = hi_bin - 1;
    const int h_hi = hi_bin >= 0 ? hist[hi_bin] : 0;
    const int h_lo = lo_bin >= 0 ? hist[lo_bin] : 0;
    int total;
    const int before = sel_block_scan(h_hi + h_lo, &total, warp_part);
    if (before < want && want <= before + h_hi + h_lo) {
        if (want <= before + h_hi) { s_out[0] = hi_bin; s_out[1] = want - before; }
        else { s_out[0] = lo_bin; s_out[1] = want - before - h_hi; }
    }
    __syncthreads();
    *bin = s_out[0];
    *want_rest = s_out[1];
    __syncthreads();
}

// PASS 0, 1, 2: histogram of the pass's digit over the slice's entries that match the digits chosen so far.
template <int PASS>
__global__ void __launch_bounds__(SEL_THREADS)
sels_hist_kernel(const int32_t *__restrict__ n_cand, const int32_t *__restrict__ ci, int64_t maxc, int n_prune,
                 int32_t *__restrict__ scratch)
{
    __shared__ int hist[2048];
    __shared__ int warp_part[32];
    __shared__ int s_out[2];
    const int b = blockIdx.y, n = n_cand[b];
    if (n <= n_prune) return;
    int32_t *sc = scratch + (int64_t)b * SELS_SCRATCH;
    uint32_t prefix = 0u, mask = 0u;
    int want = n_prune;
    if (PASS >= 1) {
        int bin;
        sels_find(sc, 2048, want, warp_part, s_out, &bin, &want);
        prefix = (uint32_t)bin << 21;
        mask = 0x7ffu << 21;
    }
    if (PASS >= 2) {
        int bin;
        sels_find(sc + 2048, 2048, want, warp_part, s_out, &bin, &want);
        prefix |= (uint32_t)bin << 10;
        mask |= 0x7ffu << 10;
    }
    constexpr int SHIFT = PASS == 0 ? 21 : PASS == 1 ? 10 : 0;
    constexpr int BINS = PASS == 2 ? 1024 : 2048;
    for (int i = threadIdx.x; i < BINS; i += SEL_THREADS) hist[i] = 0;
    __syncthreads();
    int j0, j1;
    sels_slice(n, blockIdx.x, &j0, &j1);
    const int32_t *sb = ci + (int64_t)b * maxc;
    for (int j = j0 + threadIdx.x; j < j1; j += SEL_THREADS) {
        const uint32_t u = (uint32_t)sb[j] ^ 0x80000000u;
        if ((u & mask) == prefix) atomicAdd(&hist[(u >> SHIFT) & (BINS - 1)], 1);
    }
    __syncthreads();
    int32_t *gh = sc + (PASS == 0 ? 0 : PASS == 1 ? 2048 : 4096);
    for (int i = threadIdx.x; i < BINS; i += SEL_THREADS)
        if (hist[i]) atomicAdd(&gh[i], hist[i]);
}

// The threshold (all three digits) and how many entries equal to it belong to the top n_prune.
__device__ __forceinline__ uint32_t sels_threshold(const int32_t *sc, int n_prune, int *warp_part, int *s_out, int *need_eq)
{
    int b1, b2, b3, want = n_prune;
    sels_find(sc, 2048, want, warp_part, s_out, &b1, &want);
    sels_find(sc + 2048, 2048, want, warp_part, s_out, &b2, &want);
    sels_find(sc + 4096, 1024, want, warp_part, s_out, &b3, &want);
    *need_eq = want;
    return ((uint32_t)b1 << 21) | ((uint32_t)b2 << 10) | (uint32_t)b3;
}

__global__ void __launch_bounds__(SEL_THREADS)
sels_count_kernel(const int32_t *__restrict__ n_cand, const int32_t *__restrict__ ci, int64_t maxc, int n_prune,
                  int32_t *__restrict__ scratch)
{
    __shared__ int warp_part[32];
    __shared__ int s_out[2];
    const int b = blockIdx.y, n = n_cand[b];
    if (n <= n_prune) return;
    int32_t *sc = scratch + (int64_t)b * SELS_SCRATCH;
    int need_eq;
    const uint32_t thr = sels_threshold(sc, n_prune, warp_part, s_out, &need_eq);
    int j0, j1;
    sels_slice(n, blockIdx.x, &j0, &j1);
    const int32_t *sb = ci + (int64_t)b * maxc;
    int gt = 0, eq = 0;
    for (int j = j0 + threadIdx.x; j < j1; j += SEL_THREADS) {
        const uint32_t u = (uint32_t)sb[j] ^ 0x80000000u;
        gt += u > thr ? 1 : 0;
        eq += u == thr ? 1 : 0;
    }
    int total;
    sel_block_scan((gt << 16) | eq, &total, warp_part);        // a slice has fewer than 2^15 entries (launcher)
    if (threadIdx.x == 0) {
        sc[5120 + blockIdx.x] = total >> 16;
        sc[5120 + SELS_SPLIT + blockIdx.x] = total & 0xffff;
    }
}

__global__ void __launch_bounds__(SEL_THREADS)
sels_write_kernel(const int32_t *__restrict__ cand, const int32_t *__restrict__ n_cand, const int32_t *__restrict__ ci,
                  int64_t maxc, int n_prune, const int32_t *__restrict__ scratch, int32_t *__restrict__ pruned,
                  int32_t *__restrict__ n_pruned, int32_t *__restrict__ pruned_ci)
{
    __shared__ int warp_part[32];
    __shared__ int s_out[2];
    const int b = blockIdx.y, n = n_cand[b], g = blockIdx.x;
    const int32_t *cb = cand + (int64_t)b * maxc;
    const int32_t *sb = ci + (int64_t)b * maxc;
    int32_t *out = pruned + (int64_t)b * n_prune;
    int32_t *out_ci = pruned_ci ? pruned_ci + (int64_t)b * n_prune : nullptr;
    int j0, j1;
    sels_slice(n, g, &j0, &j1);
    if (n <= n_prune) {                                     // everything survives; the last block pads
        for (int j = j0 + threadIdx.x; j < j1; j += SEL_THREADS) {
            out[j] = cb[j];
            if (out_ci) out_ci[j] = sb[j];
        }
        if (g == SELS_SPLIT - 1) {
            for (int j = n + threadIdx.x; j < n_prune; j += SEL_THREADS) {
                out[j] = -1;
                if (out_ci) out_ci[j] = INT_MIN;
            }
            if (threadIdx.x == 0) n_pruned[b] = n;
        }
        return;
    }
    const int32_t *sc = scratch + (int64_t)b * SELS_SCRATCH;
    int need_eq;
    const uint32_t thr = sels_threshold(sc, n_prune, warp_part, s_out, &need_eq);
    int run_gt = 0, run_eq = 0;
    for (int s = 0; s < g; ++s) {
        run_gt += sc[5120 + s];
        run_eq += sc[5120 + SELS_SPLIT + s];
    }
    for (int base = j0; base < j1; base += 4 * SEL_THREADS) {
        const int q0 = base + 4 * threadIdx.x;
        uint32_t u[4];
        int32_t id[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int j = q0 + e;
            u[e] = j < j1 ? ((uint32_t)sb[j] ^ 0x80000000u) : 0u;
            id[e] = j < j1 ? cb[j] : 0;
        }
        int gt = 0, eq = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            gt += (q0 + e < j1 && u[e] > thr) ? 1 : 0;
            eq += (q0 + e < j1 && u[e] == thr) ? 1 : 0;
        }
        int total;
        const int before = sel_block_scan((gt << 16) | eq, &total, warp_part);
        int gt_before = run_gt + (before >> 16), eq_before = run_eq + (before & 0xffff);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (q0 + e >= j1) break;
            const bool is_gt = u[e] > thr, is_eq = u[e] == thr;
            if (is_gt || (is_eq && eq_before < need_eq)) {
                const int pos = gt_before + (eq_before < need_eq ? eq_before : need_eq);
                out[pos] = id[e];
                if (out_ci) out_ci[pos] = (int32_t)(u[e] ^ 0x80000000u);
            }
            gt_before += is_gt ? 1 : 0;
            eq_before += is_eq ? 1 : 0;
        }
        run_gt += total >> 16;
        run_eq += total & 0xffff;
    }
    if (g == 0 && threadIdx.x == 0) n_pruned[b] = n_prune;
}

// Queries per call up to which the selection is spread over several blocks, and the scratch it needs.
bool select_split_used(const Index &ix, const Params &p) { return 4 * p.B <= ix.sm_count; }
size_t select_split_scratch_bytes(const Index &ix, const Params &p)
{
    return select_split_used(ix, p) ? sizeof(int32_t) * (size_t)p.B * SELS_SCRATCH : 0;
}

// scratch: select_split_scratch_bytes() bytes, or NULL (one block per query then).
int launch_select(const Index &ix, const Params &p, const int32_t *cand, const int32_t *n_cand, const int32_t *ci,
                  int32_t *pruned, int32_t *n_pruned, int32_t *pruned_ci, int32_t *scratch, cudaStream_t st)
{
    // the slices must stay below 2^15 entries (two counters packed in an int) and be worth five launches
    if (scratch != nullptr && select_split_used(ix, p) && p.maxc >= 16384 && p.maxc < (int64_t)SELS_SPLIT * 32767) {
        CHIMERA_CUDA(cudaMemsetAsync(scratch, 0, select_split_scratch_bytes(ix, p), st));
        const dim3 grid(SELS_SPLIT, (unsigned)p.B);
        sels_hist_kernel<0><<<grid, SEL_THREADS, 0, st>>>(n_cand, ci, p.maxc, p.n_prune, scratch);
        sels_hist_kernel<1><<<grid, SEL_THREADS, 0, st>>>(n_cand, ci, p.maxc, p.n_prune, scratch);
        sels_hist_kernel<2><<<grid, SEL_THREADS, 0, st>>>(n_cand, ci, p.maxc, p.n_prune, scratch);
        sels_count_kernel<<<grid, SEL_THREADS, 0, st>>>(n_cand, ci, p.maxc, p.n_prune, scratch);
        sels_write_kernel<<<grid, SEL_THREADS, 0, st>>>(cand, n_cand, ci, p.maxc, p.n_prune, scratch, pruned, n_pruned,
                                                        pruned_ci);
        CHIMERA_CUDA(cudaGetLastError());
        count_launch(SLOT_SELECT, 5);
        return CHIMERA_OK;
    }
    select_kernel<<<(unsigned)p.B, SEL_THREADS, 0, st>>>(cand, n_cand, ci, p.maxc, p.n_prune, pruned, n_pruned,
                                                         pruned_ci);
    CHIMERA_CUDA(cudaGetLastError());
    count_launch(SLOT_SELECT);
    return CHIMERA_OK;
}

}  // namespace chimera
