// Proximity graph over the centroids and its search: the replacement of the exhaustive centroid scan (stage 1 +
// stage 2a) that the paper uses (Sec. 3.1: a proximity-graph index built on the IVF centroids; Algorithm 1, line
// searchCAGRA; Sec. 2.3 for how such a graph is searched).
//
// Graph (index time): node c is linked to the `degree` other centroids with the largest fixed-point inner product
// S_fx(c, c'), ties towards the smaller id, best first.  It is built with the library's own exact machinery: the
// centroids take the place of query tokens in the stage-1 tensor-core kernel and stage 2a picks each row's best
// degree + 1 entries, of which the centroid itself is dropped.
//
// Search (query time): one warp per query token runs a best-first search with a bounded result list:
//   - the entry points floor(j K / n_entries), j < n_entries, are visited (scored, marked, offered to the list);
//   - repeatedly the first list member that has not been expanded is expanded: each of its graph neighbours that was
//     never visited is visited; the search ends when every list member is expanded or after max_expansions expansions;
//   - the list keeps the best `beam` visited centroids by (score descending, id ascending).
// The score is the exact S_fx(q, c) = floor((sum_d Xq[d] Xc[d] + 2^19) / 2^20) in 64-bit integers, so the list after
// each step is the best `beam` of everything offered so far whatever the order of evaluation, and the visited set, the
// probes and their scores are reproducible bit for bit.  The list lives in registers (two 64-bit keys per lane, sorted
// by slot = lane + 32 j), the visited set is a bitmap in global memory owned by the warp.
#include "common.cuh"

namespace chimera {

constexpr int GP_WARPS = 4;              // query tokens (warps) per block
constexpr int GP_PIPE = 8;               // centroid rows in flight per warp while scoring

// Xc[c][d] = rint(centroid * 2^22), recombined from the three balanced base-256 digit planes of the index.
__global__ void xc_kernel(const int8_t *__restrict__ cdig, int64_t K, int D, int32_t *__restrict__ xc)
{
    const int64_t n = K * D;
    const int64_t plane = K * 128;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (int64_t)gridDim.x * blockDim.x) {
        const int64_t c = e / D;
        const int d = (int)(e % D);
        const int64_t at = c * 128 + d;
        xc[e] = (int)cdig[at] + 256 * (int)cdig[plane + at] + 65536 * (int)cdig[2 * plane + at];
    }
}

// probes [rows][R + 1] of centroids c0 .. c0 + rows - 1 (each row best first) -> graph rows: the centroid itself is
// dropped (or the last entry, when identical twins with smaller ids pushed it out of the list).
__global__ void graph_rows_kernel(const int32_t *__restrict__ probes, int64_t c0, int rows, int R,
                                  int32_t *__restrict__ graph)
{
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= rows) return;
    const int32_t *pr = probes + (int64_t)r * (R + 1);
    int32_t *out = graph + (c0 + r) * R;
    int w = 0;
    for (int e = 0; e <= R && w < R; ++e)
        if (pr[e] != (int32_t)(c0 + r)) out[w++] = pr[e];
}

int build_graph(Index &ix, const float *centroids, int R, cudaStream_t st)
{
    if (R < 1 || R > CHIMERA_MAX_NPROBE - 1 || R > ix.K - 1)
        return fail(CHIMERA_INVALID_ARG, "degree must be in [1, min(%d, n_centroids - 1)], got %d", CHIMERA_MAX_NPROBE - 1, R);
    cudaFree(ix.graph);
    cudaFree(ix.xc);
    ix.graph = nullptr;
    ix.xc = nullptr;
    ix.graph_deg = 0;
    int32_t *graph = nullptr, *xc = nullptr;
    char *ws = nullptr;
    float *qbuf = nullptr;
    auto cleanup = [&]() { cudaFree(ws); cudaFree(qbuf); };
    auto drop = [&]() { cleanup(); cudaFree(graph); cudaFree(xc); };
    // pseudo-queries of 32 centroids each; as many per call as keep the score table near 512 MB
    constexpr int NQ = 32;
    int64_t bq = (512LL << 20) / (ix.K * NQ * 4);
    if (bq < 1) bq = 1;
    if (bq > 64) bq = 64;
    const int64_t need = (ix.K + NQ - 1) / NQ;
    if (bq > need) bq = need;
    Params p;
    p.B = (int32_t)bq; p.nq = NQ; p.P = R + 1; p.n_prune = 1; p.k = 1; p.maxc = 1;
    const Layout L = make_layout(ix, p);
    const int rows_per_call = (int)bq * NQ;
    cudaError_t e = cudaMalloc(&graph, sizeof(int32_t) * (size_t)ix.K * R);
    if (e == cudaSuccess) e = cudaMalloc(&xc, sizeof(int32_t) * (size_t)ix.K * ix.D);
    if (e == cudaSuccess) e = cudaMalloc(&ws, L.total);
    if (e == cudaSuccess) e = cudaMalloc(&qbuf, sizeof(float) * (size_t)rows_per_call * ix.D);
    if (e != cudaSuccess) {
        drop();
        return fail(CHIMERA_CUDA_ERROR, "cudaMalloc (centroid graph): %s", cudaGetErrorString(e));
    }
    xc_kernel<<<(unsigned)(8 * ix.sm_count), 256, 0, st>>>(ix.cdig, ix.K, ix.D, xc);
    uint32_t *status = (uint32_t *)(ws + L.status);
    int8_t *qdig = (int8_t *)(ws + L.qdig);
    int32_t *table = (int32_t *)(ws + L.table);
    unsigned long long *part = (unsigned long long *)(ws + L.part);
    int32_t *probes = (int32_t *)(ws + L.probes);
    int rc = CHIMERA_OK;
    for (int64_t c0 = 0; c0 < ix.K && rc == CHIMERA_OK; c0 += rows_per_call) {
        const int rows = (int)(ix.K - c0 < rows_per_call ? ix.K - c0 : rows_per_call);
        e = cudaMemcpyAsync(qbuf, centroids + c0 * ix.D, sizeof(float) * (size_t)rows * ix.D, cudaMemcpyDeviceToDevice, st);
        if (e == cudaSuccess && rows < rows_per_call)
            e = cudaMemsetAsync(qbuf + (size_t)rows * ix.D, 0, sizeof(float) * (size_t)(rows_per_call - rows) * ix.D, st);
        if (e != cudaSuccess) { rc = fail(CHIMERA_CUDA_ERROR, "copy (centroid graph): %s", cudaGetErrorString(e)); break; }
        if ((rc = launch_score_table(ix, p, qbuf, qdig, table, nullptr, status, st))) break;
        if ((rc = launch_probes(ix, p, L, table, part, probes, st))) break;
        graph_rows_kernel<<<(unsigned)((rows + 127) / 128), 128, 0, st>>>(probes, c0, rows, R, graph);
    }
    if (rc == CHIMERA_OK) {
        e = cudaGetLastError();
        if (e == cudaSuccess) e = cudaStreamSynchronize(st);
        if (e != cudaSuccess) rc = fail(CHIMERA_CUDA_ERROR, "centroid graph build: %s", cudaGetErrorString(e));
    }
    if (rc != CHIMERA_OK) {
        cudaStreamSynchronize(st);
        drop();
        return rc;
    }
    cleanup();
    ix.graph = graph;
    ix.xc = xc;
    ix.graph_deg = R;
    return CHIMERA_OK;
}

// ------------------------------------------------------------------------------------------------ search ---------
// List key: a larger key ranks first.  Score in the high word, then the id (smaller id = larger key), and in bit 0
// whether the member is still to be expanded; ids differ by at least 2 in this field, so the flag never decides an
// order.  A valid key is non-zero.
__device__ __forceinline__ unsigned long long gp_key(int32_t score, int32_t id)
{
    return ((unsigned long long)((uint32_t)score ^ 0x80000000u) << 32) | ((uint32_t)(0x7FFFFFFF - id) << 1) | 1ull;
}
__device__ __forceinline__ int32_t gp_id(unsigned long long key) { return 0x7FFFFFFF - (int32_t)((uint32_t)key >> 1); }
__device__ __forceinline__ int32_t gp_score(unsigned long long key) { return (int32_t)((uint32_t)(key >> 32) ^ 0x80000000u); }

// grid (ceil(tokens / GP_WARPS)); visited: [tokens][vwords] zeroed by the caller.
__global__ void __launch_bounds__(GP_WARPS * 32)
graph_probe_kernel(const float *__restrict__ queries, int64_t n_tokens, int D, const int32_t *__restrict__ xc,
                   const int32_t *__restrict__ graph, int R, int64_t K, int n_entries, int beam, int max_exp,
                   int nprobe, uint32_t *__restrict__ visited, int64_t vwords, int32_t *__restrict__ out_probes,
                   int32_t *__restrict__ out_scores, int32_t *__restrict__ out_nvis)
{
    const int lane = threadIdx.x & 31;
    const int64_t token = (int64_t)blockIdx.x * GP_WARPS + (threadIdx.x >> 5);
    if (token >= n_tokens) return;                       // whole warps leave together
    const bool has_dims = 4 * lane < D;                  // lane owns dimensions 4 lane .. 4 lane + 3
    int xq[4] = {0, 0, 0, 0};
    if (has_dims) {
        const float4 v = __ldg(reinterpret_cast<const float4 *>(queries + token * D) + lane);
        xq[0] = __float2int_rn(fminf(fmaxf(v.x, -1.0f), 1.0f) * 4194304.0f);
        xq[1] = __float2int_rn(fminf(fmaxf(v.y, -1.0f), 1.0f) * 4194304.0f);
        xq[2] = __float2int_rn(fminf(fmaxf(v.z, -1.0f), 1.0f) * 4194304.0f);
        xq[3] = __float2int_rn(fminf(fmaxf(v.w, -1.0f), 1.0f) * 4194304.0f);
    }
    uint32_t *vis = visited + token * vwords;
    unsigned long long key0 = 0ull, key1 = 0ull;         // list slots lane and 32 + lane, best first
    int n_vis = 0;

    // offer a scored centroid (warp-uniform arguments) to the list
    auto offer = [&](int32_t n, int32_t s) {
        const unsigned long long x = gp_key(s, n);
        const int pos = __popc(__ballot_sync(0xffffffffu, (key0 >> 1) > (x >> 1))) +
                        __popc(__ballot_sync(0xffffffffu, (key1 >> 1) > (x >> 1)));
        if (pos >= beam) return;                          // ranks behind a full list
        const unsigned long long up0 = __shfl_up_sync(0xffffffffu, key0, 1), up1 = __shfl_up_sync(0xffffffffu, key1, 1);
        const unsigned long long last0 = __shfl_sync(0xffffffffu, key0, 31);
        const int s0 = lane, s1 = 32 + lane;
        if (s1 > pos) key1 = lane == 0 ? last0 : up1;
        else if (s1 == pos) key1 = x;
        if (s0 > pos) key0 = up0;
        else if (s0 == pos) key0 = x;
        if (s0 >= beam) key0 = 0ull;                      // the member pushed past the end falls off
        if (s1 >= beam) key1 = 0ull;
    };
    // exact S_fx(q, c) from a lane's four products
    auto finish_score = [&](const int4 &c) -> int32_t {
        long long s = 0;
        if (has_dims) s = (long long)xq[0] * c.x + (long long)xq[1] * c.y + (long long)xq[2] * c.z + (long long)xq[3] * c.w;
        // |s| < 2^46: the low 24 bits and the rest are summed over the warp separately (both fit 32 bits)
        const uint32_t lo = __reduce_add_sync(0xffffffffu, (uint32_t)(s & 0xffffff));
        const int32_t hi = __reduce_add_sync(0xffffffffu, (int32_t)(s >> 24));
        const long long t = ((long long)hi << 24) + (long long)lo;
        return (int32_t)((t + (1LL << 19)) >> 20);
    };
    // visit up to 32 centroids, one per lane: mark, then score the unvisited ones GP_PIPE rows at a time
    auto visit = [&](int32_t n, bool valid) {
        bool fresh = false;
        if (valid) {
            n = DBG_CID(n);
            const uint32_t bit = 1u << (n & 31);
            fresh = (atomicOr(&vis[n >> 5], bit) & bit) == 0u;
        }
        uint32_t todo = __ballot_sync(0xffffffffu, fresh);
        n_vis += __popc(todo);
        while (todo) {
            int32_t ids[GP_PIPE];
            int4 rows[GP_PIPE];
            int cnt = 0;
#pragma unroll
            for (int u = 0; u < GP_PIPE; ++u) {
                if (todo) {
                    const int src = __ffs(todo) - 1;
                    todo &= todo - 1;
                    ids[u] = __shfl_sync(0xffffffffu, n, src);
                    rows[u] = make_int4(0, 0, 0, 0);
                    if (has_dims) rows[u] = __ldg(reinterpret_cast<const int4 *>(xc + (int64_t)ids[u] * D) + lane);
                    cnt = u + 1;
                }
            }
#pragma unroll
            for (int u = 0; u < GP_PIPE; ++u)
                if (u < cnt) offer(ids[u], finish_score(rows[u]));
        }
    };

    for (int j0 = 0; j0 < n_entries; j0 += 32) {
        const int j = j0 + lane;
        visit((int32_t)(((long long)j * K) / n_entries), j < n_entries);
    }
    for (int done = 0; done < max_exp; ++done) {
        const uint32_t u0 = __ballot_sync(0xffffffffu, (key0 & 1ull) != 0ull);
        const uint32_t u1 = __ballot_sync(0xffffffffu, (key1 & 1ull) != 0ull);
        if ((u0 | u1) == 0u) break;                      // every member expanded
        int32_t p;
        if (u0) {
            const int src = __ffs(u0) - 1;
            p = gp_id(__shfl_sync(0xffffffffu, key0, src));
            if (lane == src) key0 &= ~1ull;
        } else {
            const int src = __ffs(u1) - 1;
            p = gp_id(__shfl_sync(0xffffffffu, key1, src));
            if (lane == src) key1 &= ~1ull;
        }
        for (int r0 = 0; r0 < R; r0 += 32) {
            const int r = r0 + lane;
            visit(r < R ? graph[(int64_t)p * R + r] : 0, r < R);
        }
    }
    for (int r = lane; r < nprobe; r += 32) {
        const unsigned long long k = r < 32 ? key0 : key1;   // r = lane or lane + 32
        out_probes[token * nprobe + r] = k ? gp_id(k) : -1;
        if (out_scores) out_scores[token * nprobe + r] = k ? gp_score(k) : INT32_MIN;
    }
    if (out_nvis && lane == 0) out_nvis[token] = n_vis;
}

size_t graph_scratch_bytes(const Index &ix, int64_t n_tokens)
{
    return (size_t)n_tokens * (size_t)((ix.K + 31) / 32) * sizeof(uint32_t);
}

int check_graph_params(const Index &ix, const GraphSearch &g, int nprobe)
{
    if (!ix.graph) return fail(CHIMERA_INVALID_ARG, "the centroid graph is not built (chimera_index_build_graph)");
    if (g.beam < nprobe || g.beam > 64) return fail(CHIMERA_INVALID_ARG, "beam must be in [nprobe, 64], got %d", g.beam);
    if (g.n_entries < nprobe || g.n_entries > ix.K)
        return fail(CHIMERA_INVALID_ARG, "n_entries must be in [nprobe, n_centroids], got %d", g.n_entries);
    if (g.max_expansions < 0) return fail(CHIMERA_INVALID_ARG, "max_expansions must be >= 0");
    return CHIMERA_OK;
}

int launch_graph_probes(const Index &ix, const float *queries, int64_t n_tokens, int nprobe, const GraphSearch &g,
                        uint32_t *visited, int32_t *out_probes, int32_t *out_scores, int32_t *out_nvis, cudaStream_t st)
{
    const int64_t vwords = (ix.K + 31) / 32;
    CHIMERA_CUDA(cudaMemsetAsync(visited, 0, graph_scratch_bytes(ix, n_tokens), st));
    const unsigned blocks = (unsigned)((n_tokens + GP_WARPS - 1) / GP_WARPS);
    graph_probe_kernel<<<blocks, GP_WARPS * 32, 0, st>>>(queries, n_tokens, ix.D, ix.xc, ix.graph, ix.graph_deg, ix.K,
                                                         g.n_entries, g.beam, g.max_expansions, nprobe, visited, vwords,
                                                         out_probes, out_scores, out_nvis);
    CHIMERA_CUDA(cudaGetLastError());
    count_launch(SLOT_PROBE, 1);
    return CHIMERA_OK;
}

}  // namespace chimera
