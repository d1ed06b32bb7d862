// Stage 4 on the tensor cores (q_len <= 64): residual-decode MaxSim of the surviving documents (Definition 1 on the
// decoded tokens),
//   score(d) = sum_i max_{t in d} <q_i, c_{cid_t} + r^(code_t)>
//            = sum_i [ max_t ( S[cid_t, i] + delta * sum_x q_i[x] u_t[x] ) + (lo + delta/2) * sum_x q_i[x] ].
// The code contraction sum_x q_i[x] u_t[x] is a dense [tokens x D] x [D x q_len] product with tiny integer entries on
// one side, so it runs as an exact integer MMA: the bucket indices u (0..3) are int8, the query is the same three
// int8 digit planes of rint(q * 2^22) that stage 1 built, and tcgen05.mma kind::i8 gives sum_x u digit_a exactly in
// int32; the three planes are recombined in fp32 (relative error 2^-24).
//
// A CTA owns one query and a run of its surviving documents, whose tokens form one stream cut into tiles of 128
// (MMA M).  Per tile: every thread expands the packed code of one token into 128 int8 values (two integer
// multiplications and two masks per four dimensions) and writes them with one tcgen05.st into its lane of the A
// operand IN TENSOR MEMORY (32 columns behind the accumulators; through shared memory the same row cost eight
// 16-byte stores per thread, and the load/store pipe is what this kernel is short of); one thread issues D/32 MMAs
// (N = 3 * padded q_len: the three digit planes side by side, loaded once per CTA by TMA); the accumulators come back
// with tcgen05.ld, get the centroid term from the stage-1 table, and go to shared memory, where each warp folds its
// 32 tokens into per-document maxima (a warp whose tokens are all of one document reads 16 bytes per lane and row
// quarter instead of a word per row).  Tensor memory: 128 or 256 columns per CTA, so several CTAs share an SM and
// overlap each other's phases.  All mbarrier waits are bounded.
#include <math.h>

#include "common.cuh"
#include "umma.cuh"

namespace chimera {

constexpr int G4U_THREADS = 128;
constexpr int G4U_TOK = 128;             // tokens per tile (MMA M)
constexpr int G4U_MAX_DOCS = 32;         // documents per CTA, at most

__device__ __forceinline__ uint32_t f_order(float f)
{
    uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float f_unorder(uint32_t o)
{
    return __uint_as_float((o & 0x80000000u) ? (o & 0x7fffffffu) : ~o);
}

// One code byte (four 2-bit bucket indices, dimension 4g+t in bits [2t, 2t+1]) -> four int8 values, one per byte.
// Both multiplications only place copies at disjoint bit positions, so they are shifts-and-ors without carries.
__device__ __forceinline__ uint32_t spread2(uint32_t byte)
{
    const uint32_t x = (byte * 0x1001u) & 0x000F000Fu;       // low nibble at bit 0, high nibble at bit 16
    return (x * 0x41u) & 0x03030303u;                        // second index of each nibble moved up one byte
}
// Four 1-bit codes (a nibble, dimension t in bit t) -> four int8 values 0/1: bit t lands at bit 8t of the product
// (the other copies fall on bits that the mask drops; all partial products occupy distinct bits).
__device__ __forceinline__ uint32_t spread1(uint32_t nibble) { return (nibble * 0x00204081u) & 0x01010101u; }

// RQ = true scores RaBitQ 1-bit codes instead (Sec. 2.2; the GPU half of the paper's document scoring): the same
// contraction T = sum_x Xq[x] b[x] against the digit planes of the ROTATED query, then
// est = inv_dot_t * (c * (float)(2 T - SQ_i)) with SQ_i = sum_x Xq_i[x] and c = 1 / (sqrt(D) 2^22); no centroid term;
// query tokens are summed in increasing order in fp32 so that the score is reproducible bit for bit.
template <int NQP, int NBITS, bool RQ>
__global__ void __launch_bounds__(G4U_THREADS)
residual_maxsim_umma(const __grid_constant__ CUtensorMap map_q, const float *__restrict__ queries,
                     const int32_t *__restrict__ table, int64_t K, int nq, int D, int CW, float delta, float kappa,
                     const int32_t *__restrict__ pruned, int n_prune, int docs_per_cta,
                     const int32_t *__restrict__ cids, const uint32_t *__restrict__ codes,
                     const float *__restrict__ factors, const int64_t *__restrict__ doc_off,
                     float *__restrict__ score4, uint32_t *status, long long wait_limit, int skip_loads)
{
    constexpr int N = 3 * NQP;                               // MMA N: three digit planes side by side
    constexpr uint32_t TMEM_COLS = N <= 96 ? 128 : 256;
    constexpr uint32_t A_COL = N;                            // the expanded codes: 32 columns behind the accumulators
    static_assert(N + 32 <= TMEM_COLS, "accumulators and the A operand share the allocation");
    constexpr uint32_t B_BYTES = N * 128;
    // Value rows (one per token, floats) in shared memory.  PACKED (q_len <= 32, residual codes): a row is exactly 128
    // bytes and its 16-byte groups are XOR-swizzled with the row number, so the row-per-thread writes and the
    // lane = column reads are both conflict-free without padding: 16 KB, which with the query planes and the
    // per-document maxima keeps the CTA at 32 KB and lets the SM run with a small shared-memory carve-out, i.e. more L1
    // for the scattered score-table rows (Mid, batch 256: 2.72 -> 2.41 ms against padded rows; forcing the largest
    // carve-out brings 2.71 ms back).  The RaBitQ variant gathers no rows and is faster with padded rows (pitch
    // NQP + 4, read with lane = column: conflict-free), as are 64-token queries.
    constexpr bool ON_A = NQP == 32 && !RQ;
    constexpr int VP = ON_A ? 32 : NQP + 4;
    constexpr uint32_t V_BYTES = sizeof(float) * G4U_TOK * VP;       // a multiple of 1024 for every variant
    static_assert(V_BYTES % 1024 == 0, "the query planes behind the value rows stay 1024-byte aligned");
    constexpr uint32_t IDESC = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) |
                               ((uint32_t)(G4U_TOK >> 4) << 24);

    extern __shared__ uint8_t smem_raw[];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;
    __shared__ int s_off[G4U_MAX_DOCS + 1];                  // stream offset of each document
    __shared__ long long s_t0[G4U_MAX_DOCS];                 // first global token of each document
    __shared__ float s_sumq[NQP];
    __shared__ int s_sq[NQP];                                // RQ: sum_x rint(q_p[x] * 2^22) per query token
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gen = smem_raw + (base - smem_u32(smem_raw));   // generic pointer to the aligned area
    float *vals = reinterpret_cast<float *>(gen);                                            // [128][VP]
    const uint32_t sB = base + V_BYTES;                                                      // [3][NQP][128] int8
    uint32_t *docmax = reinterpret_cast<uint32_t *>(gen + V_BYTES + B_BYTES);                // [MAX_DOCS][NQP]
    const uint32_t bars = smem_u32(docmax + G4U_MAX_DOCS * NQP);
    const uint32_t bar_b = (bars + 7u) & ~7u, bar_mma = bar_b + 8;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int b = blockIdx.y;
    const int j0 = blockIdx.x * docs_per_cta;
    int nd = n_prune - j0;
    if (nd > docs_per_cta) nd = docs_per_cta;

    if (tid == 0) {
        mbar_init(bar_b, 1);
        mbar_init(bar_mma, 1);
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        // stream offsets of this CTA's documents (padding slots have id -1 and no tokens): lane = document, one
        // round of loads, then a prefix sum of the lengths
        int32_t d = -1;
        if (lane < nd) d = pruned[(int64_t)b * n_prune + j0 + lane];
        long long t0 = 0;
        int len = 0;
        if (d >= 0) {
            d = DBG_DOC(d);
            t0 = doc_off[d];
            len = (int)(doc_off[d + 1] - t0);
        }
        int incl = len;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        if (lane < nd) {
            s_off[lane] = incl - len;
            s_t0[lane] = t0;
        }
        if (lane == 31) s_off[nd] = incl;          // lanes past nd add nothing
    }
    if (warp == 0) {
        __syncwarp();
        tmem_alloc(&s_tmem_base, TMEM_COLS);
    }
    for (int e = tid; e < G4U_MAX_DOCS * NQP; e += G4U_THREADS) docmax[e] = 0u;     // below every real value
    // sum_x q_i[x] per query token: four threads per row, each a quarter of the row with 16-byte loads
    for (int i = tid >> 2; i < NQP; i += G4U_THREADS / 4) {
        float sum = 0.f;
        int si = 0;
        if (i < nq) {
            const int quarter = D >> 2;               // D is a multiple of 32
            const float4 *src = reinterpret_cast<const float4 *>(queries + ((int64_t)b * nq + i) * D + (tid & 3) * quarter);
            for (int x = 0; x < (quarter >> 2); ++x) {
                const float4 v = __ldg(src + x);
                sum += (v.x + v.y) + (v.z + v.w);
                si += __float2int_rn(fminf(fmaxf(v.x, -1.0f), 1.0f) * 4194304.0f) +
                      __float2int_rn(fminf(fmaxf(v.y, -1.0f), 1.0f) * 4194304.0f) +
                      __float2int_rn(fminf(fmaxf(v.z, -1.0f), 1.0f) * 4194304.0f) +
                      __float2int_rn(fminf(fmaxf(v.w, -1.0f), 1.0f) * 4194304.0f);
            }
        }
        sum += __shfl_xor_sync(0xffffffffu, sum, 1);
        si += __shfl_xor_sync(0xffffffffu, si, 1);
        sum += __shfl_xor_sync(0xffffffffu, sum, 2);
        si += __shfl_xor_sync(0xffffffffu, si, 2);
        if ((tid & 3) == 0) { s_sumq[i] = sum; s_sq[i] = si; }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem_base;
    const int total = s_off[nd];
    const int n_tiles = (total + G4U_TOK - 1) / G4U_TOK;

    // skip_loads (test hook): no load is issued, so the first wait below runs into its limit with nothing in flight
    if (tid == 0 && !skip_loads) {   // the query's three digit planes, side by side: rows [p * NQP, (p + 1) * NQP)
        mbar_expect_tx(bar_b, B_BYTES);
        for (int p = 0; p < 3; ++p) tma_load_3d(sB + p * NQP * 128, &map_q, 0, b * nq, p, bar_b);
    }

    const int32_t *tb = table + (int64_t)b * K * nq;
    const bool vec_rows = (nq & 3) == 0;
    const bool wide_rows = (nq & 7) == 0;          // rows are then 32-byte aligned (the table is 256-byte aligned)
    const int k_steps = D >> 5;
    const float code_scale = delta * (1.0f / 4194304.0f);    // delta * 2^-22
    bool alive = true;
    constexpr int MAXCW = 8;                                  // 32 code bytes per token at most

    // Token of stream position s (this thread's row of a tile): local document, centroid id, packed code words.
    int dl_hint = 0;
    auto fetch = [&](int tile, int &dl, int32_t &cid, uint32_t (&cw)[MAXCW]) {
        const int s = tile * G4U_TOK + tid;
        dl = -1;
        cid = -1;
        if (s < total) {
            while (dl_hint + 1 < nd && s_off[dl_hint + 1] <= s) ++dl_hint;    // positions only move forward
            dl = dl_hint;
            const long long t = DBG_TOK(s_t0[dl] + (s - s_off[dl]));
            cid = RQ ? __float_as_int(factors[t]) : cids[t];     // RQ: the slot carries the token's factor bits (> 0)
            const uint32_t *src = codes + t * CW;
            if (NBITS == 2 && CW == 8) {                  // 32-byte codes (32-byte aligned): one load
                asm volatile("ld.global.nc.v8.u32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                             : "=r"(cw[0]), "=r"(cw[1]), "=r"(cw[2]), "=r"(cw[3]), "=r"(cw[4]), "=r"(cw[5]), "=r"(cw[6]),
                               "=r"(cw[7])
                             : "l"(src));
            } else if ((CW & 3) == 0) {                   // 16-byte aligned codes
#pragma unroll
                for (int w = 0; w < MAXCW; w += 4)
                    if (w < CW) {
                        const uint4 v = __ldg(reinterpret_cast<const uint4 *>(src + w));
                        cw[w] = v.x; cw[w + 1] = v.y; cw[w + 2] = v.z; cw[w + 3] = v.w;
                    }
            } else if ((CW & 1) == 0) {
#pragma unroll
                for (int w = 0; w < MAXCW; w += 2)
                    if (w < CW) {
                        const uint2 v = __ldg(reinterpret_cast<const uint2 *>(src + w));
                        cw[w] = v.x; cw[w + 1] = v.y;
                    }
            } else {
#pragma unroll
                for (int w = 0; w < MAXCW; ++w)
                    if (w < CW) cw[w] = __ldg(src + w);
            }
        }
    };

    int dl, dl_next = -1;
    int32_t cid, cid_next = -1;
    uint32_t cw[MAXCW], cw_next[MAXCW];
    if (n_tiles > 0) fetch(0, dl_next, cid_next, cw_next);

    for (int tile = 0; tile < n_tiles; ++tile) {
        dl = dl_next;
        cid = cid_next;
#pragma unroll
        for (int w = 0; w < MAXCW; ++w) cw[w] = cw_next[w];

        // ---- expand this thread's token into lane `tid` of the A operand in tensor memory (128 int8 = 32 columns) ----
        {
            uint32_t row[32];
#pragma unroll
            for (int x = 0; x < 32; ++x) row[x] = 0u;
            if (dl >= 0) {
#pragma unroll
                for (int w = 0; w < MAXCW; ++w) {
                    if (w < CW) {
                        const uint32_t word = cw[w];
                        if (NBITS == 2) {
                            row[4 * w + 0] = spread2(word & 255u);
                            row[4 * w + 1] = spread2((word >> 8) & 255u);
                            row[4 * w + 2] = spread2((word >> 16) & 255u);
                            row[4 * w + 3] = spread2(word >> 24);
                        } else if (w < 4) {                  // 1 bit per dimension: at most four words
#pragma unroll
                            for (int h = 0; h < 8; ++h) row[8 * w + h] = spread1((word >> (4 * h)) & 15u);
                        }
                    }
                }
            }
            tmem_st32(tmem + ((uint32_t)(warp * 32) << 16) + A_COL, row);
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        }
        tc_fence_before();
        __syncthreads();

        // ---- one thread issues the MMAs --------------------------------------------------------------------------
        if (tid == 0) {
            bool ok = true;
            if (tile == 0) ok = mbar_wait(bar_b, 0, wait_limit);
            if (ok) {
                tc_fence_after();
                const uint64_t db = umma_desc(sB);
                for (int k = 0; k < k_steps; ++k) umma_i8_ts(tmem, tmem + A_COL + 8 * k, db + 2 * k, IDESC, k > 0 ? 1u : 0u);
                umma_commit(bar_mma);
            } else {
                s_abort = 1;
            }
        }
        __syncwarp();

        // ---- while the tensor core works: this token's row of the score table, and the next tile's token -----------
        int4 sv[NQP / 4];
        if (!RQ && cid >= 0) {
            const int32_t *srow = tb + (int64_t)DBG_CID(cid) * nq;
#pragma unroll
            for (int g = 0; g < NQP / 4; ++g) {
                const int col = 4 * g;
                if (wide_rows && col + 7 < nq) {
                    // 32 bytes per load: half as many line lookups per row as with 16-byte pieces
                    if ((g & 1) == 0)
                        asm volatile("ld.global.nc.v8.s32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                                     : "=r"(sv[g].x), "=r"(sv[g].y), "=r"(sv[g].z), "=r"(sv[g].w), "=r"(sv[g + 1].x),
                                       "=r"(sv[g + 1].y), "=r"(sv[g + 1].z), "=r"(sv[g + 1].w)
                                     : "l"(srow + col));
                } else if (wide_rows && (g & 1) == 1 && col + 3 < nq) {
                    // second half of a 32-byte load issued at g - 1
                } else if (vec_rows && col + 3 < nq) {
                    sv[g] = __ldg(reinterpret_cast<const int4 *>(srow + col));
                } else {
                    sv[g].x = col + 0 < nq ? __ldg(srow + col + 0) : 0;
                    sv[g].y = col + 1 < nq ? __ldg(srow + col + 1) : 0;
                    sv[g].z = col + 2 < nq ? __ldg(srow + col + 2) : 0;
                    sv[g].w = col + 3 < nq ? __ldg(srow + col + 3) : 0;
                }
            }
        }
        if (tile + 1 < n_tiles) {
            fetch(tile + 1, dl_next, cid_next, cw_next);
            // the next token's score-table row is a scattered 4 * q_len-byte read that misses L2 (a batch's tables
            // are far larger): ask for it now so that HBM latency passes during this tile's epilogue
            // (measured: a gain for q_len <= 32, a loss for the two-line rows of longer queries)
            if (!RQ && NQP == 32 && cid_next >= 0) {
                const char *row = reinterpret_cast<const char *>(tb + (int64_t)DBG_CID(cid_next) * nq);
                for (int off = 0; off < nq * 4; off += 128) asm volatile("prefetch.global.L2 [%0];" ::"l"(row + off));
            }
        }

        const bool ok = mbar_wait(bar_mma, tile & 1, wait_limit);
        if (!__syncthreads_and(ok && !*(volatile int *)&s_abort)) {
            if (tid == 0) atomicOr(status, ST_TIMEOUT);
            alive = false;
            break;
        }
        tc_fence_after();
        __syncwarp();

        // ---- accumulators -> values of this thread's token for every query token -----------------------------------
        const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
        float *vrow = vals + tid * VP;
#pragma unroll
        for (int ch = 0; ch < NQP / 16; ++ch) {
            int32_t a0[16], a1[16], a2[16];
            tmem_ld16(lane_addr + 0 * NQP + ch * 16, a0);
            tmem_ld16(lane_addr + 1 * NQP + ch * 16, a1);
            tmem_ld16(lane_addr + 2 * NQP + ch * 16, a2);
            tmem_ld_wait();
            if (cid >= 0) {
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    const int4 q4 = RQ ? make_int4(0, 0, 0, 0) : sv[ch * 4 + g];
                    const int32_t se[4] = {q4.x, q4.y, q4.z, q4.w};
                    float val[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int o = 4 * g + e;
                        // |sum_x u_x Xq_x| <= 3 * 2^22 * |q|_1 < 2^31: the plane recombination fits int32
                        const int32_t T = a0[o] + a1[o] * 256 + a2[o] * 65536;
                        if (RQ)
                            val[e] = __fmul_rn(__int_as_float(cid), __fmul_rn(kappa, (float)(2 * T - s_sq[ch * 16 + o])));
                        else
                            val[e] = fmaf(code_scale, (float)T, (float)se[e] * (1.0f / 16777216.0f));
                    }
                    const int grp = ch * 4 + g;               // 16-byte group of the row
                    *reinterpret_cast<float4 *>(vrow + 4 * (ON_A ? grp ^ (tid & 7) : grp)) =
                        make_float4(val[0], val[1], val[2], val[3]);
                }
            }
        }
        tc_fence_before();
        __syncwarp();

        // ---- fold this warp's 32 tokens into the per-document maxima (lane = query token) -------------------------
        {
            const int prev = __shfl_up_sync(0xffffffffu, dl, 1);
            const uint32_t valid = __ballot_sync(0xffffffffu, dl >= 0);
            uint32_t starts = __ballot_sync(0xffffffffu, dl >= 0 && (lane == 0 || dl != prev));
            const int n_rows = __popc(valid);                 // valid rows are a prefix of the warp's rows
            if (ON_A && starts == 1u && valid == 0xffffffffu) {
                // The warp's 32 tokens belong to one document (most tiles of a long document): lane = (four columns,
                // a quarter of the rows), eight 16-byte loads per lane instead of 32 scalar ones, then two exchange
                // steps among the four lanes of a column group.
                const int grp = lane & 7, sub = lane >> 3;
                const float *vb = vals + warp * 32 * VP;
                float4 m = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int r = sub + 4 * j;
                    const float4 v = *reinterpret_cast<const float4 *>(vb + r * VP + ((grp ^ (r & 7)) << 2));
                    m.x = fmaxf(m.x, v.x); m.y = fmaxf(m.y, v.y); m.z = fmaxf(m.z, v.z); m.w = fmaxf(m.w, v.w);
                }
#pragma unroll
                for (int o = 8; o <= 16; o <<= 1) {
                    m.x = fmaxf(m.x, __shfl_xor_sync(0xffffffffu, m.x, o));
                    m.y = fmaxf(m.y, __shfl_xor_sync(0xffffffffu, m.y, o));
                    m.z = fmaxf(m.z, __shfl_xor_sync(0xffffffffu, m.z, o));
                    m.w = fmaxf(m.w, __shfl_xor_sync(0xffffffffu, m.w, o));
                }
                const int doc = __shfl_sync(0xffffffffu, dl, 0);
                // lane (grp, sub) publishes column 4 grp + sub
                const float mine = sub == 0 ? m.x : sub == 1 ? m.y : sub == 2 ? m.z : m.w;
                atomicMax(&docmax[doc * NQP + 4 * grp + sub], f_order(mine));
                starts = 0u;
            }
            while (starts) {
                const int a = __ffs(starts) - 1;
                starts &= starts - 1;
                const int e = starts ? __ffs(starts) - 1 : n_rows;
                const int doc = __shfl_sync(0xffffffffu, dl, a);
                float m0, m1 = 0.f;
                if (ON_A) {
                    // column `lane` of row r sits in group (lane / 4) ^ (r & 7)
                    const float *vw = vals + warp * 32 * VP + (lane & 3);
                    m0 = vw[a * VP + ((((lane >> 2) ^ a) & 7) << 2)];
                    for (int r = a + 1; r < e; ++r) m0 = fmaxf(m0, vw[r * VP + ((((lane >> 2) ^ r) & 7) << 2)]);
                } else {
                    const float *vp = vals + (warp * 32 + a) * VP + lane;
                    m0 = vp[0];
                    m1 = NQP > 32 ? vp[32] : 0.f;
                    for (int r = a + 1; r < e; ++r) {
                        vp += VP;
                        m0 = fmaxf(m0, vp[0]);
                        if (NQP > 32) m1 = fmaxf(m1, vp[32]);
                    }
                }
                atomicMax(&docmax[doc * NQP + lane], f_order(m0));
                if (NQP > 32) atomicMax(&docmax[doc * NQP + 32 + lane], f_order(m1));
            }
            // the value rows of this warp are rewritten by the next tile's epilogue, each lane its own row, while the
            // fold above reads the rows of other lanes: all lanes finish reading first
            __syncwarp();
        }
    }

    if (n_tiles == 0 && tid == 0 && !skip_loads) mbar_wait(bar_b, 0, wait_limit);   // never leave with the TMA load in flight
    tc_fence_before();
    __syncthreads();

    // ---- per document: add the per-query-token constant, sum over query tokens ----------------------------------------
    if (alive) {
        for (int dl = warp; dl < nd; dl += G4U_THREADS / 32) {
            const int32_t d = pruned[(int64_t)b * n_prune + j0 + dl];
            float v = 0.f;
            if (RQ) {                                   // fixed summation order: reproducible bits
                if (d >= 0 && lane == 0)
                    for (int i = 0; i < nq; ++i) v = __fadd_rn(v, f_unorder(docmax[dl * NQP + i]));
            } else if (d >= 0) {
                if (lane < nq) v = f_unorder(docmax[dl * NQP + lane]) + kappa * s_sumq[lane];
                if (NQP > 32 && 32 + lane < nq) v += f_unorder(docmax[dl * NQP + 32 + lane]) + kappa * s_sumq[32 + lane];
            }
            v = warp_sum(v);
            if (lane == 0) score4[(int64_t)b * n_prune + j0 + dl] = d >= 0 ? v : -INFINITY;
        }
    }
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem, TMEM_COLS);
    }
}

template <int NQP, int NBITS, bool RQ>
static int launch_g4_umma(const Index &ix, const Params &p, const float *queries, const int8_t *qdig,
                          const int32_t *table, const int32_t *pruned, float *score4, uint32_t *status, cudaStream_t st)
{
    constexpr int N = 3 * NQP;
    const float delta = (ix.res_hi - ix.res_lo) / (float)(1 << ix.nbits);
    // RQ: the kappa slot carries c = 1 / (sqrt(D) * 2^22)
    const float kappa = RQ ? (float)(1.0 / (sqrt((double)ix.D) * 4194304.0)) : ix.res_lo + 0.5f * delta;
    CUtensorMap map_q;
    int rc = make_plane_map(&map_q, qdig, (int64_t)p.B * p.nq, NQP);
    if (rc) return rc;
    // value rows (128-byte rows for q_len <= 32 with residual codes, padded rows otherwise), query planes, maxima
    size_t smem = 1024 + sizeof(float) * G4U_TOK * (NQP == 32 && !RQ ? 32 : NQP + 4) + (size_t)N * 128 +
                  sizeof(uint32_t) * G4U_MAX_DOCS * NQP + 32;
    // No more CTAs may become resident on an SM than its 512 tensor-memory columns serve: one more would sit in
    // tcgen05.alloc with its registers and shared memory until another leaves (64-token queries: three CTAs of 66 KB
    // fit an SM, two get tensor memory; measured 5.97 -> 8.92 ms).  Registers cap the 128-column residual variants at
    // four; the 256-column variants ask for a third of an SM's shared memory plus one byte.  (The 128-column RaBitQ
    // variant, whose tiles are short, measured the same with and without such a cap and has none.)
    if (N > 96 && smem < 227 * 1024 / 3 + 1) smem = 227 * 1024 / 3 + 1;
    auto kern = residual_maxsim_umma<NQP, NBITS, RQ>;
    CHIMERA_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    // documents per CTA: about four CTAs per SM in total, at most 32 documents each (with few queries per call a CTA
    // gets one or two documents, so that the call's latency is a tile or two and not a chain of them)
    int64_t dpc = ((int64_t)p.n_prune * p.B + 4LL * ix.sm_count - 1) / (4LL * ix.sm_count);
    if (dpc < 1) dpc = 1;
    if (dpc > G4U_MAX_DOCS) dpc = G4U_MAX_DOCS;
    if (dpc > p.n_prune) dpc = p.n_prune;
    dim3 grid((unsigned)((p.n_prune + dpc - 1) / dpc), (unsigned)p.B);
    const uint32_t *code_words = reinterpret_cast<const uint32_t *>(RQ ? ix.rq_bits : ix.codes);
    kern<<<grid, G4U_THREADS, smem, st>>>(map_q, queries, table, ix.K, p.nq, ix.D, RQ ? ix.D / 32 : ix.CB / 4, delta,
                                          kappa, pruned, p.n_prune, (int)dpc, ix.cids, code_words, ix.rq_inv, ix.doc_off,
                                          score4, status, wait_limit_cycles(), fault_skip_tma_loads());
    CHIMERA_CUDA(cudaGetLastError());
    count_launch(SLOT_G4);
    return CHIMERA_OK;
}

bool residual_umma_supported(int nq) { return nq <= 64; }

int launch_residual_scores_umma(const Index &ix, const Params &p, const float *queries, const int8_t *qdig,
                                const int32_t *table, const int32_t *pruned, float *score4, uint32_t *status,
                                cudaStream_t st)
{
    if (ix.nbits == 2) {
        if (p.nq <= 32) return launch_g4_umma<32, 2, false>(ix, p, queries, qdig, table, pruned, score4, status, st);
        return launch_g4_umma<64, 2, false>(ix, p, queries, qdig, table, pruned, score4, status, st);
    }
    if (p.nq <= 32) return launch_g4_umma<32, 1, false>(ix, p, queries, qdig, table, pruned, score4, status, st);
    return launch_g4_umma<64, 1, false>(ix, p, queries, qdig, table, pruned, score4, status, st);
}

// Complete 1-bit scores of the surviving documents on the RaBitQ codes; q_rot / qdig_rot belong to the rotated queries.
int launch_rabitq_scores_umma(const Index &ix, const Params &p, const float *q_rot, const int8_t *qdig_rot,
                              const int32_t *pruned, float *score4, uint32_t *status, cudaStream_t st)
{
    if (p.nq <= 32) return launch_g4_umma<32, 1, true>(ix, p, q_rot, qdig_rot, nullptr, pruned, score4, status, st);
    return launch_g4_umma<64, 1, true>(ix, p, q_rot, qdig_rot, nullptr, pruned, score4, status, st);
}

}  // namespace chimera
