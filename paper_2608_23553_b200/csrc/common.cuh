// Shared declarations of libchimera's translation units (host side + small device helpers).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>

#include "chimera.h"

namespace chimera {

// ---------------------------------------------------------------------------------------------------------------
// Index: everything resident on the device between searches.
// ---------------------------------------------------------------------------------------------------------------
struct Index {
    int device = 0;
    int sm_count = 0;
    int D = 0, nbits = 0, CB = 0;     // dim, residual bits per dim, code bytes per token
    int64_t K = 0, N = 0, T = 0;
    float res_lo = 0.f, res_hi = 0.f;
    const int32_t *cids = nullptr;    // [T]        borrowed
    const uint8_t *codes = nullptr;   // [T, CB]    borrowed
    int64_t *doc_off = nullptr;       // [N+1]      owned: first token of each document
    int8_t *cdig = nullptr;           // [3][K][128] owned: balanced base-256 digits of rint(c * 2^22), zero padded
    int64_t *ivf_off = nullptr;       // [K+1]      owned
    int32_t *ivf_doc = nullptr;       // [ivf_len]  owned: unique document ids per centroid, unordered
    int64_t ivf_len = 0;
    int32_t max_doclen = 0;
    // token-level posting lists (only after chimera_index_enable_partial): per centroid its tokens and their documents
    int64_t *tok_off = nullptr;       // [K+1]      owned
    int32_t *tok_id = nullptr;        // [T]        owned: token ids per centroid, unordered
    int32_t *tok_doc = nullptr;       // [T]        owned: document of each listed token
    int64_t max_tok_list = 0;         // longest token list
    // RaBitQ 1-bit codes (only after chimera_index_attach_rabitq)
    const uint8_t *rq_bits = nullptr; // [T, D/8]   borrowed: sign bits of the rotated tokens
    const float *rq_inv = nullptr;    // [T]        borrowed: 1 / <o_p, o_p-bar>
    float *rot_t = nullptr;           // [D][D]     owned: transposed rotation, rot_t[x * D + r] = P[r][x]
    // proximity graph over the centroids (only after chimera_index_build_graph)
    int32_t *graph = nullptr;         // [K][graph_deg] owned: nearest other centroids of each centroid, best first
    int32_t *xc = nullptr;            // [K][D]     owned: rint(centroid * 2^22)
    int graph_deg = 0;
};

// Parameters of the graph search that can stand in for stage 1 + stage 2a (g7_graph.cu).
struct GraphSearch {
    int32_t beam = 0, n_entries = 0, max_expansions = 0;
};

// Device status bits kept in the first word of a workspace.
enum : uint32_t { ST_OVERFLOW = 1u, ST_BAD_QUERY = 2u, ST_TIMEOUT = 4u, ST_BAD_INDEX = 8u };
constexpr int STATUS_WORD_CANARY = 8;   // status[8]: first damaged guard region found by the debug build's check

// ---------------------------------------------------------------------------------------------------------------
// Workspace layout (all offsets 256-byte aligned).
// ---------------------------------------------------------------------------------------------------------------
struct Params {
    int32_t B, nq, P, n_prune, k;
    int64_t maxc;                     // candidate capacity per query
};

constexpr int MAX_GUARDS = 48;
struct Layout {
    // debug builds (CHIMERA_DEBUG) put a 256-byte guard region behind every region below; guards[i] is its offset
    size_t guards[MAX_GUARDS];
    int n_guards;
    size_t status;        // uint32[64]
    size_t q_stage;       // float  [B, nq, D]        (host-entry staging of the queries)
    size_t out_ids;       // int32  [B, k]            (host-entry staging)
    size_t out_scores;    // float  [B, k]
    size_t qdig;          // int8   [3][B*nq][128]
    size_t table;         // int32  [B][K][nq]
    size_t table8;        // uint8  [B][K][nq]        coarse copy: min((S + 2^24 + 64) >> 17, 255)
    size_t part;          // uint64 [B][n_part][P][nq] partial top-P keys
    size_t probes;        // int32  [B][nq][P]
    size_t pq_gmax;       // int32  [B][pq_groups][nq] stages 1 + 2a together: largest score of each group of sample rows,
    size_t pq_thr;        // int32  [B*nq]            score bound per query-token row,
    size_t pq_cnt;        // int32  [B*nq]            keys queued for the row,
    size_t pq_keys;       // uint64 [B*nq][pq_cap]    the keys,
    size_t pq_ovf;        // int32  [B]               1 = a queue of this query overflowed (redo by the table scan)
    size_t bitmap;        // uint32 [B][words]
    size_t chunk_cnt;     // int32  [B][n_chunks + 1]
    size_t cand;          // int32  [B][maxc]
    size_t n_cand;        // int32  [B]
    size_t ci;            // int32  [B][maxc]         exact CI of the contenders (of every candidate: generic q_len / tap)
    size_t lo;            // int32  [B][maxc]         lower bound on CI of every candidate
    size_t hi;            // int32  [B][maxc]         upper bound
    size_t cont;          // int32  [B][maxc]         contender ids, ascending
    size_t cand_rng;      // int2   [B][maxc]         (first token, length) of each candidate (bound scan)
    size_t cont_rng;      // int2   [B][maxc]         the same for the contenders
    size_t n_cont;        // int32  [B]
    size_t pruned;        // int32  [B][n_prune]
    size_t word_rank;     // int32  [B][words]        candidates before each bitmap word (document -> candidate index)
    size_t partial_m;     // int32  [B][maxc][nq]     per (candidate, query token) best retrieved-token score, or
                          // uint64 [B][hash_slots]   the same as an open-addressing table (see partial_hash_slots)
    int64_t hash_slots;   // slots per query of that table; 0 = the dense form
    size_t graph_vis;     // uint32 [B*nq][K/32]      visited centroids of the graph search (only with a centroid graph)
    size_t q_rot;         // float  [B, nq, D]        rotated queries (RaBitQ pipeline)
    size_t qdig_rot;      // int8   [3][B*nq][128]    their digit planes
    size_t n_pruned;      // int32  [B]
    size_t pruned_ci;     // int32  [B][n_prune] stage-3 score of each survivor (document-sharded search)
    size_t sel_scratch;   // int32  histograms and slice counts of the multi-block selection (few queries per call)
    size_t score4;        // float  [B][n_prune]
    size_t total;
    // derived sizes
    int32_t pq_stride;    // every pq_stride-th centroid tile is a sample tile; 0 = stages 1 and 2a run separately
    int32_t pq_cap;       // keys per queue
    int32_t pq_groups;    // groups of sample rows per query (one maximum each)
    int32_t n_part;       // partial lists per query in the probe stage
    int32_t probe_blocks; // blocks per query in the probe stage
    int64_t words;        // bitmap words per query
    int32_t n_chunks;     // bitmap chunks per query
};

constexpr int PROBE_WARPS = 8;          // warps per block in the probe stage (each keeps its own partial list)
constexpr int BITMAP_CHUNK_WORDS = 1024; // bitmap words per compaction block

Layout make_layout(const Index &ix, const Params &p);

// ---------------------------------------------------------------------------------------------------------------
// Error text (thread local) and helpers.
// ---------------------------------------------------------------------------------------------------------------
int fail(int code, const char *fmt, ...);
#define CHIMERA_CUDA(call)                                                                      \
    do {                                                                                        \
        cudaError_t e__ = (call);                                                               \
        if (e__ != cudaSuccess)                                                                 \
            return ::chimera::fail(CHIMERA_CUDA_ERROR, "%s: %s", #call, cudaGetErrorString(e__)); \
    } while (0)

// ---------------------------------------------------------------------------------------------------------------
// Profiling hooks (api.cu).
// ---------------------------------------------------------------------------------------------------------------
// Limit of the bounded device-side waits and the test hook that makes them run out (api.cu; chimera_test_wait_fault).
long long wait_limit_cycles();
int fault_skip_tma_loads();

enum Slot { SLOT_G1 = 0, SLOT_PROBE, SLOT_GATHER, SLOT_CI, SLOT_SELECT, SLOT_G4, SLOT_TOPK, SLOT_MISC, SLOT_CI_EXACT };
void count_launch(int slot, int n = 1);

// ---------------------------------------------------------------------------------------------------------------
// Stage launchers (one per .cu file).  Each only enqueues kernels on `st` and returns a chimera_status.
// ---------------------------------------------------------------------------------------------------------------
int build_index_device(Index &ix, const float *centroids, const int32_t *doclens, cudaStream_t st);
// rows x D float32 in [-1, 1] -> three int8 digit planes [3][rows][128] (zero padded); out-of-range elements set
// ST_BAD_QUERY.
int launch_digits(const float *x, int64_t rows, int D, int8_t *dig, uint32_t *status, cudaStream_t st);

// table8 may be NULL (no coarse copy wanted).
int launch_score_table(const Index &ix, const Params &p, const float *queries, int8_t *qdig, int32_t *table,
                       uint8_t *table8, uint32_t *status, cudaStream_t st);
int launch_probes(const Index &ix, const Params &p, const Layout &L, const int32_t *table, unsigned long long *part,
                  int32_t *probes, cudaStream_t st);
// Stages 1 and 2a together (g1_score_table.cu), used when the layout has pq_stride > 0, and its probe-side pieces
// (g2_probe.cu): the sample's top nprobe and bounds; the final top nprobe from sample list and queues, with the table
// scan as the fallback for queries whose queue overflowed.
int probe_sample_stride(int64_t K, int nq, int P);       // host arithmetic only
int probe_queue_stride(const Index &ix, const Params &p);
int probe_queue_cap();
int probe_sample_groups(const Index &ix, int stride);
int launch_score_table_probes(const Index &ix, const Params &p, const Layout &L, const float *queries, int8_t *qdig,
                              int32_t *table, uint8_t *table8, char *ws, uint32_t *status, cudaStream_t st);
int launch_probe_sample(const Index &ix, const Params &p, const Layout &L, const int32_t *table, char *ws,
                        int n_sample_tiles, cudaStream_t st);
int launch_probe_merge(const Index &ix, const Params &p, const Layout &L, const int32_t *table, char *ws, cudaStream_t st);
int launch_gather(const Index &ix, const Params &p, const Layout &L, const int32_t *probes, uint32_t *bitmap,
                  int32_t *chunk_cnt, int32_t *cand, int32_t *n_cand, int32_t *word_rank, uint32_t *status,
                  cudaStream_t st);
// Token-level posting lists for the partial-score refinement (allocates; index_build.cu).
int build_token_lists(Index &ix, cudaStream_t st);
// Candidate refinement with partial scores (Algorithm 2): fprime[b][j] for every candidate.
// Slots per query (a power of two) of the hashed score table of the partial-score refinement, 0 when the dense table
// is used (no token lists, few queries per call, keys that do not fit 32 bits, or a dense table less than four times
// as large).
int64_t partial_hash_slots(const Index &ix, const Params &p);
int launch_partial_scores(const Index &ix, const Params &p, const Layout &L, const float *queries,
                          const int32_t *table, const int32_t *probes, const uint32_t *bitmap,
                          const int32_t *word_rank, const int32_t *n_cand, int32_t *partial_m, int32_t *fprime, uint32_t *status,
                          cudaStream_t st);
bool coarse_supported(int nq);
int launch_coarse_table(const Index &ix, const Params &p, const int32_t *table, uint8_t *table8, cudaStream_t st);
// rng: int2 [B][maxc] scratch for the candidates' token ranges (may be NULL: per-document offset lookups instead).
int launch_coarse_bounds(const Index &ix, const Params &p, const uint8_t *table8, const int32_t *cand,
                         const int32_t *n_cand, int32_t *lo, int32_t *hi, int2 *rng, cudaStream_t st);
// scratch: an int32 [B][maxc] array that is free during this step.
// rng / cont_rng (may be NULL): the candidates' token ranges and where to put those of the contenders.
int launch_contenders(const Index &ix, const Params &p, const int32_t *cand, const int32_t *n_cand, const int32_t *lo,
                      const int32_t *hi, int32_t *cont, int32_t *n_cont, int32_t *scratch, const int2 *rng,
                      int2 *cont_rng, cudaStream_t st);
// rng (may be NULL): the token ranges of the listed documents, in list order.
int launch_centroid_interaction(const Index &ix, const Params &p, const int32_t *table, const int32_t *cand,
                                const int32_t *n_cand, int32_t *ci, int blocks_cap, int slot, const int2 *rng,
                                cudaStream_t st);
// pruned_ci (may be NULL): the score of each kept document, INT_MIN in the padding.
// scratch: select_split_scratch_bytes() bytes (few queries per call: several blocks per query), or NULL.
bool select_split_used(const Index &ix, const Params &p);
size_t select_split_scratch_bytes(const Index &ix, const Params &p);
int launch_select(const Index &ix, const Params &p, const int32_t *cand, const int32_t *n_cand, const int32_t *ci,
                  int32_t *pruned, int32_t *n_pruned, int32_t *pruned_ci, int32_t *scratch, cudaStream_t st);
// Document-sharded search: the global top-n_prune of the shards' lists and the final top-k merge.
int launch_shard_export(const Params &p, const int32_t *pruned, const int32_t *pruned_ci, int64_t doc_base,
                        int32_t *out_ids, int32_t *out_ci, cudaStream_t st);
int launch_shard_select(const Params &p, const int32_t *all_ids, const int32_t *all_ci, int world, int64_t doc_base,
                        int64_t n_local, int32_t *pruned, int32_t *n_pruned, cudaStream_t st);
int launch_add_base(int32_t *ids, int64_t n, int64_t doc_base, cudaStream_t st);
int launch_shard_merge_topk(const int32_t *all_ids, const float *all_scores, int world, int B, int k, int32_t *out_ids,
                            float *out_scores, cudaStream_t st);
int launch_residual_scores(const Index &ix, const Params &p, const float *queries, const int32_t *table,
                           const int32_t *pruned, float *score4, cudaStream_t st);
// Tensor-core variant of stage 4 for q_len <= 64; qdig = the query digit planes of stage 1.
bool residual_umma_supported(int nq);
int launch_residual_scores_umma(const Index &ix, const Params &p, const float *queries, const int8_t *qdig,
                                const int32_t *table, const int32_t *pruned, float *score4, uint32_t *status,
                                cudaStream_t st);
int launch_rabitq_scores_umma(const Index &ix, const Params &p, const float *q_rot, const int8_t *qdig_rot,
                              const int32_t *pruned, float *score4, uint32_t *status, cudaStream_t st);
// g7_graph.cu
int build_graph(Index &ix, const float *centroids, int degree, cudaStream_t st);
size_t graph_scratch_bytes(const Index &ix, int64_t n_tokens);
int check_graph_params(const Index &ix, const GraphSearch &g, int nprobe);
// visited: graph_scratch_bytes(ix, n_tokens) bytes; out_scores / out_nvis may be NULL.
int launch_graph_probes(const Index &ix, const float *queries, int64_t n_tokens, int nprobe, const GraphSearch &g,
                        uint32_t *visited, int32_t *out_probes, int32_t *out_scores, int32_t *out_nvis, cudaStream_t st);
// rabitq.cu
int attach_rabitq(Index &ix, const float *rotation, cudaStream_t st);
int launch_rotate(const Index &ix, const Params &p, const float *queries, float *q_rot, cudaStream_t st);
int launch_rabitq_partial(const Index &ix, const Params &p, const Layout &L, const float *q_rot,
                          const int32_t *probes, const uint32_t *bitmap, const int32_t *word_rank,
                          const int32_t *n_cand, int32_t *partial_m, int32_t *fprime_bits, cudaStream_t st);
int launch_topk(const Index &ix, const Params &p, const int32_t *pruned, const float *score4, int32_t *out_ids,
                float *out_scores, cudaStream_t st);

// ---------------------------------------------------------------------------------------------------------------
// Debug build (-DCHIMERA_DEBUG, libchimera_debug.so): every index that a kernel is about to gather through (centroid
// id, document id, token position, candidate rank) is checked first.  An index out of range sets ST_BAD_INDEX in the
// status word of the running search and is replaced by 0 (DBG_*) or its access is skipped (DBG_*_OK), so the kernel
// never touches memory outside its arrays.  The limits and the status pointer of the running search live in one
// device variable, so a debug build serves one search at a time.  In release builds the macros vanish.
// ---------------------------------------------------------------------------------------------------------------
#ifdef CHIMERA_DEBUG
struct DbgLimits { uint32_t *status; long long K, N, T, maxc; };
extern __device__ DbgLimits chimera_dbg;
__device__ __forceinline__ bool dbg_in_range(long long x, long long n)
{
    if (x >= 0 && x < n) return true;
    if (chimera_dbg.status) atomicOr(chimera_dbg.status, ST_BAD_INDEX);
    return false;
}
template <class I> __device__ __forceinline__ I dbg_index(I x, long long n) { return dbg_in_range((long long)x, n) ? x : (I)0; }
#define DBG_CID(c) ::chimera::dbg_index((c), ::chimera::chimera_dbg.K)
#define DBG_DOC(d) ::chimera::dbg_index((d), ::chimera::chimera_dbg.N)
#define DBG_TOK(t) ::chimera::dbg_index((t), ::chimera::chimera_dbg.T)
#define DBG_DOC_OK(d) ::chimera::dbg_in_range((long long)(d), ::chimera::chimera_dbg.N)
#define DBG_RANK_OK(r) ::chimera::dbg_in_range((long long)(r), ::chimera::chimera_dbg.maxc)
#else
#define DBG_CID(c) (c)
#define DBG_DOC(d) (d)
#define DBG_TOK(t) (t)
#define DBG_DOC_OK(d) true
#define DBG_RANK_OK(r) true
#endif
// Host side (api.cu): publish the running search's limits / fill and check the guard regions (no-ops in release builds).
int debug_begin_search(const Index &ix, const Params &p, const Layout &L, void *workspace, cudaStream_t st);

// ---------------------------------------------------------------------------------------------------------------
// Device helpers.
// ---------------------------------------------------------------------------------------------------------------
__device__ __forceinline__ int warp_sum(int v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ unsigned long long warp_max(unsigned long long v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        unsigned long long w = __shfl_xor_sync(0xffffffffu, v, o);
        v = w > v ? w : v;
    }
    return v;
}

// Order-preserving key of (score desc, id asc): a larger key is a better entry.
__device__ __forceinline__ unsigned long long key_int(int32_t score, int32_t id)
{
    return ((unsigned long long)((uint32_t)score ^ 0x80000000u) << 32) | (uint32_t)(0xFFFFFFFFu - (uint32_t)id);
}
__device__ __forceinline__ int32_t key_id(unsigned long long key) { return (int32_t)(0xFFFFFFFFu - (uint32_t)key); }

}  // namespace chimera
