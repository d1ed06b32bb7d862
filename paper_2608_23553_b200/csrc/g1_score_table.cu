// Stage 1: score table S[c, i] = <q_i, centroid_c> for every query token and every centroid (Definition 1's inner
// product), evaluated exactly in integers:
//     Xq = rint(q * 2^22), Xc = rint(c * 2^22),  T = sum_d Xq[d] * Xc[d],  S = floor((T + 2^19) / 2^20)   (Q.24).
// Each 23-bit integer is split into three balanced base-256 digits, so T = sum_{a,b} 256^(a+b) P_ab with the nine
// digit-plane products P_ab = sum_d qa[d] * cb[d] being int8 x int8 -> int32 contractions (exact in any order).
// Products of equal weight a+b share an accumulator (five accumulators, each |.| < 2^23); the epilogue recombines
// them with shifts (in 32-bit arithmetic, see combine_digits) and rounds.
//
// The contraction runs on the 5th-generation tensor cores: tcgen05.mma kind::i8 (int8 operands, int32 accumulators in
// tensor memory), M = 128 centroids x N = 48 query tokens x K = 32 dimensions per instruction.  Both operands are
// K-major digit planes with a 128-byte row pitch (dimensions beyond D are zero), brought into 128-byte-swizzled shared
// memory by TMA (plain per-CTA cp.async.bulk.tensor loads, no multicast).  One CTA owns a tile of 128 centroids (its
// three digit planes stay in shared memory) and walks over tiles of 48 query-token rows, double-buffering the query
// planes.  The five accumulators take 240 of the 256 tensor-memory columns a CTA allocates, so two CTAs share an SM and
// one's epilogue overlaps the other's MMAs.  Twelve warps drain the accumulators (three per tensor-memory lane quarter,
// chunks of eight columns, the next chunk's tcgen05.ld issued ahead) and store 32 bytes of the table per chunk.  Every wait on an mbarrier is bounded; a wait that gives up sets the
// workspace's TIMEOUT status bit and the CTA frees its tensor memory and returns.
#include <cuda.h>

#include "common.cuh"
#include "umma.cuh"

namespace chimera {

constexpr int G1_M = 128;            // centroids per tile (MMA M)
constexpr int G1_N = 48;             // query-token rows per tile (MMA N)
constexpr int G1_ROW_BYTES = 128;    // digit-plane row pitch = padded dimension count
constexpr int G1_WPQ = 3;              // warps per tensor-memory lane quarter that drain the accumulators (2: 1.53 ms,
                                       // 3: 1.43 ms, 6: 1.76 ms on the Mid corpus at batch 256)
constexpr int G1_THREADS = 128 * G1_WPQ;
constexpr int G1_TMEM_COLS = 256;
constexpr uint32_t G1_A_PLANE = G1_M * G1_ROW_BYTES;      // 16 KB
constexpr uint32_t G1_B_PLANE = G1_N * G1_ROW_BYTES;      // 6 KB
constexpr uint32_t G1_SMEM = 3 * G1_A_PLANE + 2 * 3 * G1_B_PLANE + 1024 /* alignment slack */ + 64 /* barriers */;

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

// grid (ceil(K / 128), n_splits).  Each CTA: centroid tile blockIdx.x, query-row tiles [blockIdx.y * tiles_per_split, ...).
template <int KS>
__global__ void __launch_bounds__(G1_THREADS)
score_table_umma(const __grid_constant__ CUtensorMap map_c, const __grid_constant__ CUtensorMap map_q, int64_t K,
                 int nq, int64_t q_rows, int n_tiles, int tiles_per_split, int32_t *__restrict__ table,
                 uint8_t *__restrict__ table8, uint32_t *status, long long wait_limit, int skip_loads)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sA = base;                                  // 3 planes x 16 KB
    const uint32_t sB = base + 3 * G1_A_PLANE;                 // 2 stages x 3 planes x 6 KB
    const uint32_t bars = sB + 2 * 3 * G1_B_PLANE;             // full_a, full_b[2], mma_done
    const uint32_t bar_a = bars, bar_b0 = bars + 8, bar_mma = bars + 24;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int64_t c0 = (int64_t)blockIdx.x * G1_M;
    const int t_begin = blockIdx.y * tiles_per_split;
    int t_end = t_begin + tiles_per_split;
    if (t_end > n_tiles) t_end = n_tiles;

    if (tid == 0) {
        mbar_init(bar_a, 1);
        mbar_init(bar_b0, 1);
        mbar_init(bar_b0 + 8, 1);
        mbar_init(bar_mma, 1);
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        __syncwarp();
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem_base)),
                     "r"(G1_TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = s_tmem_base;

    // instruction descriptor: D = S32, A and B signed 8-bit, both K-major, N = 48, M = 128
    constexpr uint32_t IDESC = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(G1_N >> 3) << 17) |
                               ((uint32_t)(G1_M >> 4) << 24);

    // skip_loads (test hook): no load is issued and no bytes are expected, so the waits below run into their limit
    // with nothing in flight
    if (tid == 0 && t_begin < t_end && !skip_loads) {
        mbar_expect_tx(bar_a, 3 * G1_A_PLANE);
        for (int p = 0; p < 3; ++p) tma_load_3d(sA + p * G1_A_PLANE, &map_c, 0, (int)c0, p, bar_a);
        mbar_expect_tx(bar_b0, 3 * G1_B_PLANE);
        for (int p = 0; p < 3; ++p) tma_load_3d(sB + p * G1_B_PLANE, &map_q, 0, t_begin * G1_N, p, bar_b0);
    }

    for (int t = t_begin; t < t_end; ++t) {
        const int it = t - t_begin, stage = it & 1;
        if (tid == 0) {
            bool ok = true;
            if (t + 1 < t_end && !skip_loads) {   // the other stage was released by the previous tile's completed MMAs
                const uint32_t nb = bar_b0 + 8 * (stage ^ 1);
                mbar_expect_tx(nb, 3 * G1_B_PLANE);
                for (int p = 0; p < 3; ++p)
                    tma_load_3d(sB + ((stage ^ 1) * 3 + p) * G1_B_PLANE, &map_q, 0, (t + 1) * G1_N, p, nb);
            }
            if (it == 0) ok = mbar_wait(bar_a, 0, wait_limit);
            if (ok) ok = mbar_wait(bar_b0 + 8 * stage, (it >> 1) & 1, wait_limit);
            if (ok) {
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                // accumulator w = digit weight a + b; fully unrolled, so every descriptor is a base plus a constant
                const uint64_t da0 = umma_desc(sA), db0 = umma_desc(sB + stage * 3 * G1_B_PLANE);
#pragma unroll
                for (int w = 0; w < 5; ++w) {
#pragma unroll
                    for (int a = 0; a < 3; ++a) {          // query digit
                        const int bdig = w - a;            // centroid digit
                        if (bdig < 0 || bdig > 2) continue;
                        const bool first = (a == (w > 2 ? w - 2 : 0));
#pragma unroll
                        for (int k = 0; k < KS; ++k)
                            umma_i8(tmem + w * G1_N, da0 + (uint64_t)(bdig * (G1_A_PLANE >> 4) + 2 * k),
                                    db0 + (uint64_t)(a * (G1_B_PLANE >> 4) + 2 * k), IDESC, (first && k == 0) ? 0u : 1u);
                    }
                }
                umma_commit(bar_mma);
            } else {
                s_abort = 1;
                atomicOr(status, ST_TIMEOUT);
            }
        }
        __syncwarp();
        // everybody waits for the accumulators (bounded), then drains them
        const bool ok = mbar_wait(bar_mma, it & 1, wait_limit);
        if (!__syncthreads_and(ok && !*(volatile int *)&s_abort)) {      // uniform decision for the whole CTA
            if (tid == 0) atomicOr(status, ST_TIMEOUT);
            break;
        }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        __syncwarp();
        // warp w reads tensor-memory lanes 32 (w % 4) ... + 31 (its centroids); the G1_WPQ warps of a lane quarter
        // take the chunks of eight query-token columns in turn
        const int quad = warp & 3;
        const int64_t c = c0 + quad * 32 + lane;
        const uint32_t lane_addr = tmem + ((uint32_t)(quad * 32) << 16);
        const uint32_t unq = (uint32_t)nq, rows32 = (uint32_t)q_rows;
        // (query, token) coordinates of the tile's first row: one 32-bit division per tile
        const uint32_t tile_qb = ((uint32_t)t * G1_N) / unq, tile_qi = (uint32_t)t * G1_N - tile_qb * unq;
        // Each warp takes one pair of adjacent chunks.  The tensor-memory loads of the next
        // chunk are issued before the current one is recombined and stored, so their latency hides behind that work.
        uint32_t w8_carry[2] = {0u, 0u};                  // 8-bit words of the even chunk of a pair
        auto emit = [&](const int32_t (&acc)[5][8], const int chunk) {
            int32_t out[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) out[e] = combine_digits(acc[0][e], acc[1][e], acc[2][e], acc[3][e], acc[4][e]);
            // first query-token row of this chunk and its (query, token) coordinates (rows fit 32 bits:
            // n_queries * q_len < 2^23)
            const uint32_t r0 = (uint32_t)t * G1_N + (uint32_t)chunk * 8;
            uint32_t qb = tile_qb, qi = tile_qi + (uint32_t)chunk * 8;      // chunk * 8 < 48: few subtractions
            while (qi >= unq) { qi -= unq; ++qb; }
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
                    if ((chunk & 1) == 0) {
                        w8_carry[0] = w[0];
                        w8_carry[1] = w[1];
                    } else {
                        *reinterpret_cast<uint4 *>(table8 + ((int64_t)qb * K + c) * nq + qi - 8) =
                            make_uint4(w8_carry[0], w8_carry[1], w[0], w[1]);
                    }
                }
                if ((nq & 7) == 0) {
                    // the chunk's eight values are consecutive tokens of one query, 32-byte aligned: one store
                    if (r0 < rows32)                                  // q_rows is a multiple of 8 here
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
        };
        constexpr int CHUNKS_PER_WARP = (G1_N / 8) / G1_WPQ;
        static_assert(CHUNKS_PER_WARP == 2, "a warp drains one pair of adjacent chunks");
        const int first_chunk = 2 * (warp >> 2);
        int32_t accs[2][5][8];
#pragma unroll
        for (int w = 0; w < 5; ++w) tmem_ld8(lane_addr + w * G1_N + first_chunk * 8, accs[0][w]);
#pragma unroll
        for (int it = 0; it < CHUNKS_PER_WARP; ++it) {
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            if (it + 1 < CHUNKS_PER_WARP) {
#pragma unroll
                for (int w = 0; w < 5; ++w)
                    tmem_ld8(lane_addr + w * G1_N + (first_chunk + (it + 1)) * 8, accs[(it + 1) & 1][w]);
            }
            emit(accs[it & 1], first_chunk + it);
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();                   // accumulators drained before the next tile overwrites them
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(G1_TMEM_COLS) : "memory");
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

// Digit planes [3][rows][128] int8 as a 3-D tensor (128 bytes, rows, 3 planes); box = (128, box_rows, 1); rows past
// the end read as zeros.
int make_plane_map(CUtensorMap *map, const int8_t *planes, int64_t rows, int box_rows)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return fail(CHIMERA_CUDA_ERROR, "cuTensorMapEncodeTiled is not available from the driver");
    cuuint64_t dims[3] = {(cuuint64_t)G1_ROW_BYTES, (cuuint64_t)rows, 3};
    cuuint64_t strides[2] = {(cuuint64_t)G1_ROW_BYTES, (cuuint64_t)rows * G1_ROW_BYTES};
    cuuint32_t box[3] = {(cuuint32_t)G1_ROW_BYTES, (cuuint32_t)box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, (void *)planes, dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(CHIMERA_CUDA_ERROR, "cuTensorMapEncodeTiled failed with code %d", (int)r);
    return CHIMERA_OK;
}

int launch_score_table(const Index &ix, const Params &p, const float *queries, int8_t *qdig, int32_t *table,
                       uint8_t *table8, uint32_t *status, cudaStream_t st)
{
    const int64_t rows = (int64_t)p.B * p.nq;
    int rc = launch_digits(queries, rows, ix.D, qdig, status, st);
    if (rc) return rc;
    CUtensorMap map_c, map_q;
    if ((rc = make_plane_map(&map_c, ix.cdig, ix.K, G1_M))) return rc;
    if ((rc = make_plane_map(&map_q, qdig, rows, G1_N))) return rc;
    const int c_tiles = (int)((ix.K + G1_M - 1) / G1_M);
    const int n_tiles = (int)((rows + G1_N - 1) / G1_N);
    // about eight waves of two CTAs per SM, so the last wave is mostly full
    int splits = (16 * ix.sm_count + c_tiles - 1) / c_tiles;
    if (splits > n_tiles) splits = n_tiles;
    if (splits < 1) splits = 1;
    const int tiles_per_split = (n_tiles + splits - 1) / splits;
    dim3 grid((unsigned)c_tiles, (unsigned)((n_tiles + tiles_per_split - 1) / tiles_per_split));
    const long long limit = wait_limit_cycles();
    const int skip = fault_skip_tma_loads();
#define CHIMERA_G1_LAUNCH(KS)                                                                                          \
    do {                                                                                                               \
        CHIMERA_CUDA(cudaFuncSetAttribute(score_table_umma<KS>, cudaFuncAttributeMaxDynamicSharedMemorySize,           \
                                          (int)G1_SMEM));                                                              \
        score_table_umma<KS><<<grid, G1_THREADS, G1_SMEM, st>>>(map_c, map_q, ix.K, p.nq, rows, n_tiles,               \
                                                                tiles_per_split, table, table8, status, limit, skip);  \
    } while (0)
    switch (ix.D / 32) {                       // MMA steps of 32 dimensions
    case 1: CHIMERA_G1_LAUNCH(1); break;
    case 2: CHIMERA_G1_LAUNCH(2); break;
    case 3: CHIMERA_G1_LAUNCH(3); break;
    default: CHIMERA_G1_LAUNCH(4); break;
    }
#undef CHIMERA_G1_LAUNCH
    CHIMERA_CUDA(cudaGetLastError());
    count_launch(SLOT_G1, 2);
    return CHIMERA_OK;
}

}  // namespace chimera
