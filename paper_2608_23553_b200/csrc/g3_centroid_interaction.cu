// Stage 3: centroid-interaction pruning.
//   CI(d) = sum_i max_{t in d} S[cid_t, i]      (the Chamfer aggregation rule of Sec. 4.2 -- per query token the
//                                                maximum over the document's tokens, then the sum over query
//                                                tokens -- applied to the centroid scores; integers, order-free)
//   keep the n_prune candidates with the largest CI, ties towards the smaller document id.
//
// ci_kernel: one warp per candidate document.  The document's centroid ids are streamed with coalesced 128-byte
// loads (lane = token), each is broadcast with a shuffle, and the warp gathers the table row S[cid, :] with
// lane = query token (one 128-byte line for 32 query tokens), keeping a running maximum per lane.
//
// select_kernel: one block per query.  Radix select (11 + 11 + 10 bits) of the n_prune-th largest CI, then an
// ordered compaction of the candidate list (which is ascending in id), so equal scores are resolved towards smaller
// ids and the survivors come out ascending.
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
        const int64_t d = cb[j];
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
                    const int32_t *row = tb + (int64_t)c[u] * nq;
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

// Wide variant for q_len = 4 * LPR (LPR = 8, 16 or 32 lanes per table row): every lane loads 16 bytes (four query
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
    constexpr int UNROLL = 4;
    const int b = blockIdx.y;
    const int lane = threadIdx.x & 31;
    const int grp = lane / LPR, sub = lane % LPR;
    const int n = n_cand[b];
    const int4 *tb = reinterpret_cast<const int4 *>(table + (int64_t)b * K * NQ) + sub;
    const int32_t *cb = cand + (int64_t)b * maxc;
    int32_t *out = ci + (int64_t)b * maxc;
    const int warps_per_query = gridDim.x * CI_WARPS;
    for (int j = blockIdx.x * CI_WARPS + (threadIdx.x >> 5); j < n; j += warps_per_query) {
        const int64_t d = cb[j];
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
                    v[u] = __ldg(tb + (int64_t)c * LPR);
                }
#pragma unroll
                for (int u = 0; u < UNROLL; ++u) {
                    m.x = max(m.x, v[u].x);
                    m.y = max(m.y, v[u].y);
                    m.z = max(m.z, v[u].z);
                    m.w = max(m.w, v[u].w);
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

int launch_centroid_interaction(const Index &ix, const Params &p, const int32_t *table, const int32_t *cand,
                                const int32_t *n_cand, int32_t *ci, cudaStream_t st)
{
    int64_t want = (p.maxc + CI_WARPS - 1) / CI_WARPS;
    int64_t cap = (int64_t)ix.sm_count * 8;
    unsigned gx = (unsigned)(want < cap ? want : cap);
    if (gx < 1) gx = 1;
    dim3 grid(gx, (unsigned)p.B);
    const int nqw = (p.nq + 31) / 32;
    if (p.nq == 32)
        ci_wide_kernel<8><<<grid, CI_THREADS, 0, st>>>(table, ix.K, cand, n_cand, p.maxc, ix.cids, ix.doc_off, ci);
    else if (p.nq == 64)
        ci_wide_kernel<16><<<grid, CI_THREADS, 0, st>>>(table, ix.K, cand, n_cand, p.maxc, ix.cids, ix.doc_off, ci);
    else if (p.nq == 128)
        ci_wide_kernel<32><<<grid, CI_THREADS, 0, st>>>(table, ix.K, cand, n_cand, p.maxc, ix.cids, ix.doc_off, ci);
    else if (nqw == 1)
        ci_kernel<1><<<grid, CI_THREADS, 0, st>>>(table, ix.K, p.nq, cand, n_cand, p.maxc, ix.cids, ix.doc_off, ci);
    else if (nqw == 2)
        ci_kernel<2><<<grid, CI_THREADS, 0, st>>>(table, ix.K, p.nq, cand, n_cand, p.maxc, ix.cids, ix.doc_off, ci);
    else
        ci_kernel<4><<<grid, CI_THREADS, 0, st>>>(table, ix.K, p.nq, cand, n_cand, p.maxc, ix.cids, ix.doc_off, ci);
    CHIMERA_CUDA(cudaGetLastError());
    count_launch(SLOT_CI);
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

// grid (B).  pruned[b][0..n_prune) ascending ids, -1 padded; n_pruned[b].
__global__ void __launch_bounds__(SEL_THREADS)
select_kernel(const int32_t *__restrict__ cand, const int32_t *__restrict__ n_cand, const int32_t *__restrict__ ci,
              int64_t maxc, int n_prune, int32_t *__restrict__ pruned, int32_t *__restrict__ n_pruned)
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

    if (n <= n_prune) {
        for (int j = threadIdx.x; j < n_prune; j += SEL_THREADS) out[j] = j < n ? cb[j] : -1;
        if (threadIdx.x == 0) n_pruned[b] = n;
        return;
    }

    // Radix select on u = ci ^ 0x80000000 (unsigned order = signed order), most significant digit first.
    if (threadIdx.x == 0) { s_prefix = 0u; s_want = n_prune; }
    const int shifts[3] = {21, 10, 0};
    const int widths[3] = {11, 11, 10};
    uint32_t known_mask = 0u;
    for (int pass = 0; pass < 3; ++pass) {
        const int shift = shifts[pass], bins = 1 << widths[pass];
        for (int i = threadIdx.x; i < 2048; i += SEL_THREADS) hist[i] = 0;
        __syncthreads();
        const uint32_t prefix = s_prefix;
        const int want = s_want;
        for (int j = threadIdx.x; j < n; j += SEL_THREADS) {
            uint32_t u = (uint32_t)sb[j] ^ 0x80000000u;
            if ((u & known_mask) == prefix) atomicAdd(&hist[(u >> shift) & (bins - 1)], 1);
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
                s_prefix = prefix | ((uint32_t)hi_bin << shift);
                s_want = want - before;
            } else {
                s_prefix = prefix | ((uint32_t)lo_bin << shift);
                s_want = want - before - h_hi;
            }
        }
        known_mask |= (uint32_t)(bins - 1) << shift;
        __syncthreads();
    }
    const uint32_t thr = s_prefix;       // the n_prune-th largest value
    const int need_eq = s_want;          // how many entries equal to it are kept (the first ones in id order)

    // Ordered compaction: keep u > thr, and the first need_eq entries with u == thr.
    int run_gt = 0, run_eq = 0;
    for (int base = 0; base < n; base += SEL_THREADS) {
        int j = base + threadIdx.x;
        uint32_t u = j < n ? ((uint32_t)sb[j] ^ 0x80000000u) : 0u;
        int gt = (j < n && u > thr) ? 1 : 0;
        int eq = (j < n && u == thr) ? 1 : 0;
        int total;
        int before = sel_block_scan((gt << 16) | eq, &total, warp_part);   // <= 1024 per field
        int gt_before = run_gt + (before >> 16), eq_before = run_eq + (before & 0xffff);
        bool keep = gt || (eq && eq_before < need_eq);
        if (keep) out[gt_before + (eq_before < need_eq ? eq_before : need_eq)] = cb[j];
        run_gt += total >> 16;
        run_eq += total & 0xffff;
    }
    if (threadIdx.x == 0) n_pruned[b] = n_prune;
}

int launch_select(const Index &ix, const Params &p, const int32_t *cand, const int32_t *n_cand, const int32_t *ci,
                  int32_t *pruned, int32_t *n_pruned, cudaStream_t st)
{
    (void)ix;
    select_kernel<<<(unsigned)p.B, SEL_THREADS, 0, st>>>(cand, n_cand, ci, p.maxc, p.n_prune, pruned, n_pruned);
    CHIMERA_CUDA(cudaGetLastError());
    count_launch(SLOT_SELECT);
    return CHIMERA_OK;
}

}  // namespace chimera
