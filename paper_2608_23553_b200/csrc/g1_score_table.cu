// Stage 1: score table S[c, i] = <q_i, centroid_c> for every query token and every centroid (Definition 1's inner
// product), evaluated exactly in integers:
//     Xq = rint(q * 2^22), Xc = rint(c * 2^22),  T = sum_d Xq[d] * Xc[d],  S = floor((T + 2^19) / 2^20)   (Q.24).
// Each 23-bit integer is split into three balanced base-256 digits, so T = sum_{a,b} 256^(a+b) P_ab with the nine
// digit-plane products P_ab = sum_d qa[d] * cb[d] being int8 x int8 -> int32 contractions (exact in any order).
// Products of equal weight a+b share an accumulator (five accumulators, each |.| < 2^23); the epilogue recombines
// them with shifts (in 32-bit arithmetic, see combine_digits) and rounds.
//
// The contraction runs on the 5th-generation tensor cores: tcgen05.mma kind::i8 (int8 operands, int32 accumulators in
// tensor memory), M = 128 centroids, K = 32 dimensions per instruction.  One CTA owns a tile of 128 centroids for its
// whole life and keeps their three digit planes IN TENSOR MEMORY (the A operand of the instruction is read from there:
// lane = centroid, 32 bytes per K step), so only the query digits come from shared memory and the 48 KB that the tile
// would take there go to a deeper pipeline of query tiles.  A query tile is 32 query-token rows; its three digit planes
// are K-major rows with a 128-byte pitch (dimensions beyond D are zero), brought into 128-byte-swizzled shared memory
// one after the other by TMA (one plain per-CTA cp.async.bulk.tensor load per tile, no multicast), four tiles deep, so
// that one instruction with N = 96 multiplies a centroid digit plane with all three query planes (see the schedule at
// the MMA loop).  Tensor memory per CTA: 5 accumulators x 32 columns + 96 columns of centroid digits = 256 columns, so
// two CTAs share an SM.  A producer warp issues the loads and the MMAs; eight warps drain the accumulators (two per
// tensor-memory lane quarter, a pair of eight-column chunks each).  A draining warp hands the accumulators back as soon
// as its tcgen05.ld's have landed in registers, so the next tile's MMAs run while it recombines and stores.  An
// isolated loop of these instructions runs at half a cycle per column of N (8,192 multiply-adds per SM cycle) but
// never faster than ~45 cycles per instruction, which is why the instructions here are N = 96 wide (48 cycles).
// Every wait on an mbarrier is bounded; a wait that gives up sets the workspace's TIMEOUT status bit, and the CTA
// waits (bounded) for its loads in flight, frees its tensor memory and returns.
#include <cuda.h>

#include "common.cuh"
#include "umma.cuh"

namespace chimera {

constexpr int G1_M = 128;            // centroids per tile (MMA M)
constexpr int G1_N = 32;             // query-token rows per tile (MMA N)
constexpr int G1_ROW_BYTES = 128;    // digit-plane row pitch = padded dimension count
constexpr int G1_WPQ = 2;            // draining warps per tensor-memory lane quarter
constexpr int G1_DRAIN_WARPS = 4 * G1_WPQ;
constexpr int G1_THREADS = 32 * (G1_DRAIN_WARPS + 1);      // + the producer warp
constexpr int G1_STAGES = 4;         // query tiles in flight
constexpr int G1_TMEM_COLS = 256;
constexpr int G1_ACC_COLS = 5 * G1_N;                      // accumulators in columns [0, 160)
constexpr int G1_A_COL = G1_ACC_COLS;                      // centroid digits in columns [160, 256): 32 per plane
constexpr uint32_t G1_B_PLANE = G1_N * G1_ROW_BYTES;       // 4 KB
constexpr uint32_t G1_B_LOAD = 3 * G1_B_PLANE;             // 12 KB: the three digit planes of a tile, one after the other
constexpr uint32_t G1_B_STAGE = 5 * G1_B_PLANE;            // 20 KB: + 64 rows of zeros (see the MMA schedule)
constexpr uint32_t G1_SMEM = G1_STAGES * G1_B_STAGE + 1024 /* alignment slack */ + 64 /* barriers */;
static_assert(G1_ACC_COLS + 96 <= G1_TMEM_COLS, "accumulators and centroid digits share the allocation");

// floor((T + 2^19) / 2^20) with T = a0 + 2^8 a1 + 2^16 a2 + 2^24 a3 + 2^32 a4, in 32-bit arithmetic.  Split T as
// u + 2^16 v with u = a0 + 2^8 a1 (|a0| < 2^23, |a1| < 2^23: no overflow together with the rounding constant) and
// v = a2 + 2^8 a3 + 2^16 a4.  v is about T / 2^16, which fits 32 bits whenever the result does (|S| < 2^31 means
// |T| < 2^51; here |T| < 2^45), so computing it modulo 2^32 loses nothing.  Nested floor divisions compose:
// floor((x + 2^16 v) / 2^20) = floor((floor(x / 2^16) + v) / 2^4) for any integers x, v; arithmetic right shifts are
// floor divisions.
__device__ __forceinline__ int32_t combine_digits(int32_t a0, int32_t a1, int32_t a2, int32_t a3, int32_t a4)
{
    const int32_t u = a0 + (a1 << 8) + (1 << 19);
    const int32_t v = a2 + (int32_t)((uint32_t)a3 << 8) + (int32_t)((uint32_t)a4 << 16);
    return ((u >> 16) + v) >> 4;
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// Which centroid tiles a launch covers, and whether it feeds the probe stage (FILTER).
//   tile_stride == 0: every tile (tile = blockIdx.x).
//   tile_stride  > 1, sample != 0: the sample tiles 0, s, 2s, ... (tile = blockIdx.x * s).
//   tile_stride  > 1, sample == 0: all the others (the j-th tile that is not a multiple of s).
// FILTER (only with the "others"): thr[row] holds, for every query-token row, a lower bound on the score of the row's
// nprobe-th best centroid (found on the sample); every score >= thr[row] goes, as a (score, centroid) key, into that
// row's queue (keys[row][cap], counted in cnt[row]; entries past cap are dropped and the count tells).  The top nprobe
// of a row are then in its queue, so the probe stage never reads the table again.
struct G1Tiles {
    int tile_stride, sample;
    const int32_t *thr;
    int32_t *cnt;
    unsigned long long *keys;
    int cap;
};

// grid (centroid tiles of the launch, n_splits).  Each CTA: one centroid tile, query-row tiles
// [blockIdx.y * tiles_per_split, ...).  KS = D / 32 MMA steps per digit-plane product.
template <int KS, bool FILTER>
__global__ void __launch_bounds__(G1_THREADS)
score_table_umma(const int8_t *__restrict__ cdig, const __grid_constant__ CUtensorMap map_q, int64_t K, int nq,
                 int64_t q_rows, int n_tiles, int tiles_per_split, int32_t *__restrict__ table,
                 uint8_t *__restrict__ table8, uint32_t *status, long long wait_limit, int skip_loads, G1Tiles tiles)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint32_t s_tmem_base;
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sB = base;                                  // G1_STAGES x (3 planes x 4 KB + 8 KB of zeros)
    const uint32_t bars = sB + G1_STAGES * G1_B_STAGE;
    const uint32_t bar_full = bars;                            // [G1_STAGES]: a query tile has landed
    const uint32_t bar_mma = bars + 8 * G1_STAGES;             // a tile's accumulators are complete
    const uint32_t bar_empty = bar_mma + 8;                    // every draining warp has the accumulators in registers
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    int c_tile = (int)blockIdx.x;
    if (tiles.tile_stride > 1)
        c_tile = tiles.sample ? c_tile * tiles.tile_stride : c_tile + c_tile / (tiles.tile_stride - 1) + 1;
    const int64_t c0 = (int64_t)c_tile * G1_M;
    const int t_begin = blockIdx.y * tiles_per_split;
    int t_end = t_begin + tiles_per_split;
    if (t_end > n_tiles) t_end = n_tiles;
    const int my_tiles = t_end > t_begin ? t_end - t_begin : 0;

    if (tid == 0) {
        for (int s = 0; s < G1_STAGES; ++s) mbar_init(bar_full + 8 * s, 1);
        mbar_init(bar_mma, 1);
        mbar_init(bar_empty, G1_DRAIN_WARPS);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        __syncwarp();
        tmem_alloc(&s_tmem_base, G1_TMEM_COLS);
    }
    // the 64 zero rows behind each stage's planes (the loads never touch them); only the stages this CTA will use
    const uint32_t used_stages = my_tiles < G1_STAGES ? (uint32_t)my_tiles : (uint32_t)G1_STAGES;
    for (uint32_t e = tid; e < used_stages * (G1_B_STAGE - G1_B_LOAD) / 16; e += G1_THREADS) {
        const uint32_t per = (G1_B_STAGE - G1_B_LOAD) / 16;
        const uint32_t addr = sB + (e / per) * G1_B_STAGE + G1_B_LOAD + (e % per) * 16;
        asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(addr), "r"(0u) : "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // visible to the tensor core's reads
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem_base;

    // the first query tiles are requested before the centroid tile is fetched, so the two latencies overlap.
    // skip_loads (test hook): no load is issued and no bytes are expected, so the producer's first wait runs into its
    // limit with nothing in flight
    int issued = 0;                                            // producer thread: tiles whose load has been issued
    auto load_tile = [&](int it) {
        const uint32_t bar = bar_full + 8 * (it % G1_STAGES);
        mbar_expect_tx(bar, G1_B_LOAD);
        tma_load_3d(sB + (it % G1_STAGES) * G1_B_STAGE, &map_q, 0, (t_begin + it) * G1_N, 0, bar);
    };
    if (warp == G1_DRAIN_WARPS && lane == 0 && !skip_loads)
        for (; issued < my_tiles && issued < G1_STAGES; ++issued) load_tile(issued);

    // ---- the centroid tile's digit planes into tensor memory: one warp per lane quarter, lane = centroid ------------
    if (warp < 4) {
        const int64_t c = c0 + warp * 32 + lane;
        const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16) + G1_A_COL;
        for (int p = 0; p < 3; ++p) {
            uint32_t r[32];
            if (c < K) {
                const uint4 *src = reinterpret_cast<const uint4 *>(cdig + ((int64_t)p * K + c) * G1_ROW_BYTES);
#pragma unroll
                for (int x = 0; x < 8; ++x) {
                    const uint4 v = __ldg(src + x);
                    r[4 * x] = v.x; r[4 * x + 1] = v.y; r[4 * x + 2] = v.z; r[4 * x + 3] = v.w;
                }
            } else {
#pragma unroll
                for (int x = 0; x < 32; ++x) r[x] = 0u;
            }
            tmem_st32(lane_addr + p * 32, r);
        }
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    // instruction descriptors: D = S32, A and B signed 8-bit, both K-major, M = 128, N = 96 or 160
    constexpr uint32_t IDESC_BASE = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(G1_M >> 4) << 24);
    constexpr uint32_t IDESC_3 = IDESC_BASE | ((uint32_t)((3 * G1_N) >> 3) << 17);
    constexpr uint32_t IDESC_5 = IDESC_BASE | ((uint32_t)((5 * G1_N) >> 3) << 17);

    if (warp == G1_DRAIN_WARPS) {
        // ================================================================================= producer (one thread) ===
        if (lane == 0) {
            bool ok = true;
            int it = 0;
            for (; it < my_tiles; ++it) {
                const int stage = it % G1_STAGES;
                ok = mbar_wait(bar_full + 8 * stage, (it / G1_STAGES) & 1, wait_limit);
                // the previous tile's accumulators are in the draining warps' registers: its MMAs are complete (so
                // its stage of query digits is free) and tensor memory may be overwritten
                if (ok && it > 0) ok = mbar_wait(bar_empty, (it - 1) & 1, wait_limit);
                if (!ok) break;
                tc_fence_after();
                // The stage holds the query's digit planes a = 0, 1, 2 as 96 consecutive B rows, and the accumulators
                // of weight w = 0..4 are consecutive groups of 32 columns.  One instruction with the centroids' digit
                // plane b as A and all 96 rows as B therefore adds the products of weight b, b + 1, b + 2 to the
                // accumulators starting at column 32 b: three instructions of N = 96 per K step instead of nine of
                // N = 32 (an instruction takes N / 2 cycles but at least ~45: -8 % on the whole kernel).  The very
                // first instruction runs over 160 rows (the last 64 are zeros) without accumulating, which clears
                // weights 3 and 4.
                const uint64_t db0 = umma_desc(sB + stage * G1_B_STAGE);
#pragma unroll
                for (int k = 0; k < KS; ++k) {
#pragma unroll
                    for (int bdig = 0; bdig < 3; ++bdig) {     // centroid digit
                        if (k == 0 && bdig == 0)
                            umma_i8_ts(tmem, tmem + G1_A_COL, db0, IDESC_5, 0u);
                        else
                            umma_i8_ts(tmem + bdig * G1_N, tmem + G1_A_COL + bdig * 32 + 8 * k, db0 + (uint64_t)(2 * k),
                                       IDESC_3, 1u);
                    }
                }
                umma_commit(bar_mma);
                // refill the stage that the previous tile used
                if (it > 0 && issued < my_tiles && !skip_loads) {
                    load_tile(issued);                         // issued == it - 1 + G1_STAGES: the same stage
                    ++issued;
                }
            }
            if (!ok) {
                atomicOr(status, ST_TIMEOUT);
                // loads in flight write this CTA's shared memory: wait for them (bounded) before leaving
                if (!skip_loads)
                    for (int j = it; j < issued; ++j)
                        mbar_wait(bar_full + 8 * (j % G1_STAGES), (j / G1_STAGES) & 1, wait_limit);
            } else if (my_tiles > 0) {
                // the last tile's MMAs read shared memory and tensor memory: complete before the CTA leaves
                if (!mbar_wait(bar_mma, (my_tiles - 1) & 1, wait_limit)) atomicOr(status, ST_TIMEOUT);
            }
        }
    } else {
        // ============================================================================================ draining warps ===
        // warp w reads tensor-memory lanes 32 (w % 4) ... + 31 (its centroids); the G1_WPQ warps of a lane quarter
        // take one pair of adjacent eight-column chunks each
        const int quad = warp & 3;
        const int64_t c = c0 + quad * 32 + lane;
        const uint32_t lane_addr = tmem + ((uint32_t)(quad * 32) << 16);
        const uint32_t unq = (uint32_t)nq, rows32 = (uint32_t)q_rows;
        const int first_chunk = 2 * (warp >> 2);
        unsigned long long pend_key = 0ull, *pend_dst = nullptr;   // FILTER: this thread's last key, not stored yet
        int pend_slot = 0;
        for (int it = 0; it < my_tiles; ++it) {
            const int t = t_begin + it;
            // FILTER: the thresholds of this warp's 16 query-token rows (the same for every lane), asked for before
            // the wait
            int32_t thr_v[16];
            if (FILTER) {
                const uint32_t r0 = (uint32_t)t * G1_N + (uint32_t)first_chunk * 8;
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    int4 v = make_int4(0x7fffffff, 0x7fffffff, 0x7fffffff, 0x7fffffff);     // rows past the end
                    if (r0 + 4 * g < rows32) v = __ldg(reinterpret_cast<const int4 *>(tiles.thr + r0) + g);
                    thr_v[4 * g] = v.x; thr_v[4 * g + 1] = v.y; thr_v[4 * g + 2] = v.z; thr_v[4 * g + 3] = v.w;
                }
            }
            // (the vote makes the decision uniform: the tensor-memory loads below need the whole warp)
            if (!__all_sync(0xffffffffu, mbar_wait(bar_mma, it & 1, wait_limit))) {
                if (lane == 0) atomicOr(status, ST_TIMEOUT);
                break;
            }
            tc_fence_after();
            int32_t accs[2][5][8];
#pragma unroll
            for (int ch = 0; ch < 2; ++ch)
#pragma unroll
                for (int w = 0; w < 5; ++w) tmem_ld8(lane_addr + w * G1_N + (first_chunk + ch) * 8, accs[ch][w]);
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_empty);             // the accumulators may be overwritten from here on

            // (query, token) coordinates of the tile's first row: one 32-bit division per tile
            const uint32_t tile_qb = ((uint32_t)t * G1_N) / unq, tile_qi = (uint32_t)t * G1_N - tile_qb * unq;
            uint32_t w8_carry[2] = {0u, 0u};                  // 8-bit words of the even chunk of the pair
#pragma unroll
            for (int ch = 0; ch < 2; ++ch) {
                const int chunk = first_chunk + ch;
                int32_t out[8];
#pragma unroll
                for (int e = 0; e < 8; ++e)
                    out[e] = combine_digits(accs[ch][0][e], accs[ch][1][e], accs[ch][2][e], accs[ch][3][e], accs[ch][4][e]);
                // first query-token row of this chunk and its (query, token) coordinates (rows fit 32 bits:
                // n_queries * q_len < 2^23)
                const uint32_t r0 = (uint32_t)t * G1_N + (uint32_t)chunk * 8;
                uint32_t qb = tile_qb, qi = tile_qi + (uint32_t)chunk * 8;      // chunk * 8 < 32: few subtractions
                while (qi >= unq) { qi -= unq; ++qb; }
                if (FILTER && c < K) {
                    bool any = false;
#pragma unroll
                    for (int e = 0; e < 8; ++e) any |= out[e] >= thr_v[ch * 8 + e];
                    if (any) {                  // about nprobe x tile_stride keys per row in all: one lane of a warp
                                                // every few chunks
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            if (out[e] >= thr_v[ch * 8 + e]) {  // (rows past the end have the largest threshold and
                                                                //  zero digits: they never pass)
                                // The slot comes back from the atomic hundreds of cycles later; the key is stored
                                // only when this thread's next key turns up (or at the end), so nobody waits for it.
                                if (pend_key && pend_slot < tiles.cap) pend_dst[pend_slot] = pend_key;
                                const uint32_t row = r0 + e;
                                pend_key = key_int(out[e], (int32_t)c);
                                pend_dst = tiles.keys + (int64_t)row * tiles.cap;
                                pend_slot = atomicAdd(tiles.cnt + row, 1);
                            }
                        }
                    }
                }
                if (c < K && r0 < rows32) {
                    if (table8 != nullptr) {
                        // coarse copy for the bound phase of stage 3: clamp(S >> 16, 0, 255); q_len is a multiple
                        // of 16 here, so the 8 rows of a chunk belong to one query and the store is 8-byte aligned
                        uint32_t w[2];
#pragma unroll
                        for (int g = 0; g < 2; ++g) {
                            uint32_t v[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) v[e] = (uint32_t)__vimin_s32_relu(out[4 * g + e] >> 16, 255);
                            w[g] = __byte_perm(__byte_perm(v[0], v[1], 0x0040), __byte_perm(v[2], v[3], 0x0040), 0x5410);
                        }
                        // a warp's two chunks are adjacent (16 query tokens of one query): one 16-byte store for the pair
                        if (ch == 0) {
                            w8_carry[0] = w[0];
                            w8_carry[1] = w[1];
                        } else {
                            *reinterpret_cast<uint4 *>(table8 + ((int64_t)qb * K + c) * nq + qi - 8) =
                                make_uint4(w8_carry[0], w8_carry[1], w[0], w[1]);
                        }
                    }
                    if ((nq & 7) == 0) {
                        // the chunk's eight values are consecutive tokens of one query, 32-byte aligned: one store
                        asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(
                                         table + ((int64_t)qb * K + c) * nq + qi),
                                     "r"(out[0]), "r"(out[1]), "r"(out[2]), "r"(out[3]), "r"(out[4]), "r"(out[5]),
                                     "r"(out[6]), "r"(out[7])
                                     : "memory");
                    } else if ((nq & 3) == 0) {
#pragma unroll
                        for (int e = 0; e < 8; e += 4) {
                            if (r0 + e < rows32)                          // q_rows is a multiple of 4 here
                                *reinterpret_cast<int4 *>(table + ((int64_t)qb * K + c) * nq + qi) =
                                    make_int4(out[e], out[e + 1], out[e + 2], out[e + 3]);
                            qi += 4;
                            if (qi >= unq) { qi -= unq; ++qb; }           // groups of four never straddle two queries
                        }
                    } else {
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            if (r0 + e < rows32) table[((int64_t)qb * K + c) * nq + qi] = out[e];
                            if (++qi == unq) { qi = 0; ++qb; }
                        }
                    }
                }
            }
        }
        if (FILTER && pend_key && pend_slot < tiles.cap) pend_dst[pend_slot] = pend_key;
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem, G1_TMEM_COLS);
    }
}

// ------------------------------------------------------------------------------------------------ host side ------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

// Digit planes [3][rows][128] int8 as a 3-D tensor (128 bytes, rows, 3 planes); box = (128, box_rows, box_planes);
// rows past the end read as zeros.
int make_plane_map(CUtensorMap *map, const int8_t *planes, int64_t rows, int box_rows, int box_planes)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return fail(CHIMERA_CUDA_ERROR, "cuTensorMapEncodeTiled is not available from the driver");
    cuuint64_t dims[3] = {(cuuint64_t)G1_ROW_BYTES, (cuuint64_t)rows, 3};
    cuuint64_t strides[2] = {(cuuint64_t)G1_ROW_BYTES, (cuuint64_t)rows * G1_ROW_BYTES};
    cuuint32_t box[3] = {(cuuint32_t)G1_ROW_BYTES, (cuuint32_t)box_rows, (cuuint32_t)box_planes};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, (void *)planes, dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(CHIMERA_CUDA_ERROR, "cuTensorMapEncodeTiled failed with code %d", (int)r);
    return CHIMERA_OK;
}

// One launch of the kernel over `c_tiles` centroid tiles (see G1Tiles for which).
template <bool FILTER>
static int launch_g1_tiles(const Index &ix, const Params &p, const CUtensorMap &map_q, int c_tiles, int32_t *table,
                           uint8_t *table8, uint32_t *status, const G1Tiles &tiles, cudaStream_t st)
{
    const int64_t rows = (int64_t)p.B * p.nq;
    const int n_tiles = (int)((rows + G1_N - 1) / G1_N);
    // about eight waves of two CTAs per SM, so the last wave is mostly full; a launch over few centroid tiles (the
    // sample) fills one wave instead, because a CTA's start-up costs as much as three tiles
    int splits = c_tiles < 2 * ix.sm_count ? (2 * ix.sm_count) / c_tiles : (16 * ix.sm_count + c_tiles - 1) / c_tiles;
    if (splits > n_tiles) splits = n_tiles;
    if (splits < 1) splits = 1;
    const int tiles_per_split = (n_tiles + splits - 1) / splits;
    dim3 grid((unsigned)c_tiles, (unsigned)((n_tiles + tiles_per_split - 1) / tiles_per_split));
    const long long limit = wait_limit_cycles();
    const int skip = fault_skip_tma_loads();
#define CHIMERA_G1_LAUNCH(KS)                                                                                          \
    do {                                                                                                               \
        CHIMERA_CUDA(cudaFuncSetAttribute(score_table_umma<KS, FILTER>, cudaFuncAttributeMaxDynamicSharedMemorySize,   \
                                          (int)G1_SMEM));                                                              \
        score_table_umma<KS, FILTER><<<grid, G1_THREADS, G1_SMEM, st>>>(ix.cdig, map_q, ix.K, p.nq, rows, n_tiles,     \
                                                                        tiles_per_split, table, table8, status, limit, \
                                                                        skip, tiles);                                  \
    } while (0)
    switch (ix.D / 32) {                       // MMA steps of 32 dimensions
    case 1: CHIMERA_G1_LAUNCH(1); break;
    case 2: CHIMERA_G1_LAUNCH(2); break;
    case 3: CHIMERA_G1_LAUNCH(3); break;
    default: CHIMERA_G1_LAUNCH(4); break;
    }
#undef CHIMERA_G1_LAUNCH
    CHIMERA_CUDA(cudaGetLastError());
    return CHIMERA_OK;
}

int launch_score_table(const Index &ix, const Params &p, const float *queries, int8_t *qdig, int32_t *table,
                       uint8_t *table8, uint32_t *status, cudaStream_t st)
{
    const int64_t rows = (int64_t)p.B * p.nq;
    int rc = launch_digits(queries, rows, ix.D, qdig, status, st);
    if (rc) return rc;
    CUtensorMap map_q;
    if ((rc = make_plane_map(&map_q, qdig, rows, G1_N, 3))) return rc;        // one load brings a tile's three planes
    const G1Tiles all = {0, 0, nullptr, nullptr, nullptr, 0};
    if ((rc = launch_g1_tiles<false>(ix, p, map_q, (int)((ix.K + G1_M - 1) / G1_M), table, table8, status, all, st)))
        return rc;
    count_launch(SLOT_G1, 2);
    return CHIMERA_OK;
}

// Stages 1 and 2a together (Sec. 3.2 step 1 on top of Definition 1's products): the table of a sample of the centroid
// tiles first, from it a lower bound per query token on the score of the token's true nprobe-th best centroid, then
// the rest of the table with every score at or above that bound queued beside it (the sample's own scores are queued
// by a scan of their rows), and the nprobe best keys of each queue.  The result is the exact top nprobe by (score
// descending, centroid id ascending): a centroid that belongs to it has a score >= the bound, so it is queued.
// A query with a token whose queue overflowed is redone by the table scan of the separate probe stage.
int launch_score_table_probes(const Index &ix, const Params &p, const Layout &L, const float *queries, int8_t *qdig,
                              int32_t *table, uint8_t *table8, char *ws, uint32_t *status, cudaStream_t st)
{
    const int64_t rows = (int64_t)p.B * p.nq;
    int rc = launch_digits(queries, rows, ix.D, qdig, status, st);
    if (rc) return rc;
    CUtensorMap map_q;
    if ((rc = make_plane_map(&map_q, qdig, rows, G1_N, 3))) return rc;
    const int c_tiles = (int)((ix.K + G1_M - 1) / G1_M);
    const int stride = L.pq_stride;
    const int n_sample = (c_tiles + stride - 1) / stride;
    int32_t *thr = (int32_t *)(ws + L.pq_thr), *cnt = (int32_t *)(ws + L.pq_cnt);
    unsigned long long *keys = (unsigned long long *)(ws + L.pq_keys);

    const G1Tiles sample = {stride, 1, nullptr, nullptr, nullptr, 0};
    if ((rc = launch_g1_tiles<false>(ix, p, map_q, n_sample, table, table8, status, sample, st))) return rc;
    if ((rc = launch_probe_sample(ix, p, L, table, ws, n_sample, st))) return rc;
    const G1Tiles rest = {stride, 0, thr, cnt, keys, L.pq_cap};
    if ((rc = launch_g1_tiles<true>(ix, p, map_q, c_tiles - n_sample, table, table8, status, rest, st))) return rc;
    count_launch(SLOT_G1, 3);
    return CHIMERA_OK;
}

}  // namespace chimera
