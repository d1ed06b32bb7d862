// C ABI of libchimera: argument checks, workspace layout, stage sequencing, taps, status and profiling.
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <atomic>
#include <new>

#include "common.cuh"

namespace chimera {

// ------------------------------------------------------------------------------------------------ errors ---------
static thread_local char g_err[512] = "";

int fail(int code, const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return code;
}

// ------------------------------------------------------------------------------------------------ wait limit -----
static std::atomic<long long> g_wait_cycles{100000000LL};      // = UMMA_WAIT_CYCLES (umma.cuh)
static std::atomic<int> g_skip_tma{0};
long long wait_limit_cycles() { return g_wait_cycles.load(std::memory_order_relaxed); }
int fault_skip_tma_loads() { return g_skip_tma.load(std::memory_order_relaxed); }

// ------------------------------------------------------------------------------------------------ profiling ------
constexpr int PROF_MARKS = 16;
struct ProfCall {
    cudaEvent_t ev[PROF_MARKS];
    int slot[PROF_MARKS];     // slot[i] = stage that ran between ev[i-1] and ev[i]
    int n = 0;
    bool created = false;
};
static bool g_prof_on = false;
static ProfCall g_calls[CHIMERA_PROFILE_MAX_CALLS];
static int g_n_calls = 0;
// launch counters are bumped by every search, from whichever host thread calls it; the per-call timing marks below
// belong to one profiling thread (chimera_profile_enable's caller)
static std::atomic<int64_t> g_launches[CHIMERA_PROFILE_SLOTS];
static ProfCall *g_cur = nullptr;

void count_launch(int slot, int n) { g_launches[slot].fetch_add(n, std::memory_order_relaxed); }

static void prof_begin(cudaStream_t st)
{
    g_cur = nullptr;
    if (!g_prof_on || g_n_calls >= CHIMERA_PROFILE_MAX_CALLS) return;
    ProfCall *c = &g_calls[g_n_calls];
    if (!c->created) {
        for (int i = 0; i < PROF_MARKS; ++i)
            if (cudaEventCreate(&c->ev[i]) != cudaSuccess) return;
        c->created = true;
    }
    c->n = 0;
    if (cudaEventRecord(c->ev[0], st) != cudaSuccess) return;
    c->slot[0] = -1;
    c->n = 1;
    g_cur = c;
    ++g_n_calls;
}
static void prof_mark(int slot, cudaStream_t st)
{
    if (!g_cur || g_cur->n >= PROF_MARKS) return;
    if (cudaEventRecord(g_cur->ev[g_cur->n], st) != cudaSuccess) return;
    g_cur->slot[g_cur->n] = slot;
    ++g_cur->n;
}

// ------------------------------------------------------------------------------------------------ layout ---------
static size_t align_up(size_t x) { return (x + 255) & ~(size_t)255; }

Layout make_layout(const Index &ix, const Params &p)
{
    Layout L;
    memset(&L, 0, sizeof(L));
    // probe stage: about four blocks per SM over the whole batch, at most 512 per query, at least ~256 rows each;
    // every block leaves one partial list per query token
    int64_t blocks = (4LL * ix.sm_count + p.B - 1) / p.B;
    int64_t by_rows = (ix.K + 255) / 256;
    if (blocks > by_rows) blocks = by_rows;
    if (blocks > 512) blocks = 512;
    if (blocks < 1) blocks = 1;
    L.probe_blocks = (int32_t)blocks;
    L.n_part = L.probe_blocks;
    L.words = (ix.N + 31) / 32;
    L.n_chunks = (int32_t)((L.words + BITMAP_CHUNK_WORDS - 1) / BITMAP_CHUNK_WORDS);

    size_t o = 0;
#ifdef CHIMERA_DEBUG
    // a 256-byte guard region behind every region: a kernel that writes past its array damages the pattern there
    auto take = [&](size_t bytes) {
        size_t at = o;
        o = align_up(o + bytes);
        if (L.n_guards < MAX_GUARDS) L.guards[L.n_guards++] = o;
        o += 256;
        return at;
    };
#else
    auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes); return at; };
#endif
    const size_t B = (size_t)p.B, nq = (size_t)p.nq;
    L.status = take(64 * sizeof(uint32_t));
    L.q_stage = take(B * nq * ix.D * sizeof(float));
    L.out_ids = take(B * p.k * sizeof(int32_t));
    L.out_scores = take(B * p.k * sizeof(float));
    L.qdig = take(3 * B * nq * 128);
    L.table = take(B * (size_t)ix.K * nq * sizeof(int32_t));
    L.table8 = take(coarse_supported(p.nq) ? B * (size_t)ix.K * nq : 0);
    L.pq_stride = probe_queue_stride(ix, p);
    L.pq_groups = L.pq_stride ? probe_sample_groups(ix, L.pq_stride) : 0;
    L.part = take(B * L.n_part * p.P * nq * sizeof(unsigned long long));
    L.probes = take(B * nq * p.P * sizeof(int32_t));
    L.pq_cap = L.pq_stride ? probe_queue_cap() : 0;
    L.pq_gmax = take(L.pq_stride ? B * (size_t)L.pq_groups * nq * sizeof(int32_t) : 0);
    L.pq_thr = take(L.pq_stride ? B * nq * sizeof(int32_t) : 0);
    L.pq_cnt = take(L.pq_stride ? B * nq * sizeof(int32_t) : 0);
    L.pq_keys = take(L.pq_stride ? B * nq * (size_t)L.pq_cap * sizeof(unsigned long long) : 0);
    L.pq_ovf = take(L.pq_stride ? B * sizeof(int32_t) : 0);
    L.bitmap = take(B * (size_t)L.words * sizeof(uint32_t));
    L.chunk_cnt = take(B * (size_t)(L.n_chunks + 1) * sizeof(int32_t));
    L.cand = take(B * (size_t)p.maxc * sizeof(int32_t));
    L.n_cand = take(B * sizeof(int32_t));
    L.ci = take(B * (size_t)p.maxc * sizeof(int32_t));
    const size_t two_phase = coarse_supported(p.nq) ? B * (size_t)p.maxc * sizeof(int32_t) : 0;
    L.lo = take(two_phase);
    L.hi = take(two_phase);
    L.cont = take(two_phase);
    L.cand_rng = take(2 * two_phase);
    L.cont_rng = take(2 * two_phase);
    L.n_cont = take(B * sizeof(int32_t));
    L.pruned = take(B * p.n_prune * sizeof(int32_t));
    L.word_rank = take(B * (size_t)L.words * sizeof(int32_t));
    // partial-score table: dense rows per candidate (always for the RaBitQ refinement), or the hashed form
    L.hash_slots = partial_hash_slots(ix, p);
    {
        const size_t dense = B * (size_t)p.maxc * nq * sizeof(int32_t);
        const size_t hashed = B * (size_t)L.hash_slots * sizeof(unsigned long long);
        size_t bytes = 0;
        if (ix.tok_id) bytes = L.hash_slots ? hashed : dense;
        if (ix.rot_t && bytes < dense) bytes = dense;
        L.partial_m = take(bytes);
    }
    L.graph_vis = take(ix.graph ? graph_scratch_bytes(ix, (int64_t)p.B * p.nq) : 0);
    L.q_rot = take(ix.rot_t ? B * nq * ix.D * sizeof(float) : 0);
    L.qdig_rot = take(ix.rot_t ? 3 * B * nq * 128 : 0);
    L.n_pruned = take(B * sizeof(int32_t));
    L.pruned_ci = take(B * p.n_prune * sizeof(int32_t));
    L.sel_scratch = take(select_split_scratch_bytes(ix, p));
    L.score4 = take(B * p.n_prune * sizeof(float));
    L.total = o;
    return L;
}

// ------------------------------------------------------------------------------------------------ debug build ----
#ifdef CHIMERA_DEBUG
__device__ DbgLimits chimera_dbg;

struct GuardList { size_t off[MAX_GUARDS]; int n; };
constexpr uint32_t GUARD_PATTERN = 0xC0FFEE00u;
// grid (n guards), 64 threads: guard g holds 64 words GUARD_PATTERN | g.
__global__ void guard_fill_kernel(char *ws, GuardList g)
{
    reinterpret_cast<uint32_t *>(ws + g.off[blockIdx.x])[threadIdx.x] = GUARD_PATTERN | blockIdx.x;
}
// the lowest damaged guard goes to status[STATUS_WORD_CANARY] (preset to 0xffffffff)
__global__ void guard_check_kernel(const char *ws, GuardList g, uint32_t *status)
{
    if (reinterpret_cast<const uint32_t *>(ws + g.off[blockIdx.x])[threadIdx.x] != (GUARD_PATTERN | blockIdx.x))
        atomicMin(&status[STATUS_WORD_CANARY], (uint32_t)blockIdx.x);
}

int debug_begin_search(const Index &ix, const Params &p, const Layout &L, void *workspace, cudaStream_t st)
{
    DbgLimits lim;
    lim.status = reinterpret_cast<uint32_t *>((char *)workspace + L.status);
    lim.K = ix.K; lim.N = ix.N; lim.T = ix.T; lim.maxc = p.maxc;
    CHIMERA_CUDA(cudaMemcpyToSymbolAsync(chimera_dbg, &lim, sizeof(lim), 0, cudaMemcpyHostToDevice, st));
    GuardList g;
    g.n = L.n_guards;
    for (int i = 0; i < L.n_guards; ++i) g.off[i] = L.guards[i];
    if (g.n > 0) guard_fill_kernel<<<g.n, 64, 0, st>>>((char *)workspace, g);
    CHIMERA_CUDA(cudaGetLastError());
    return CHIMERA_OK;
}
#else
int debug_begin_search(const Index &, const Params &, const Layout &, void *, cudaStream_t) { return CHIMERA_OK; }
#endif

static int check_params(const Index *ix, int32_t B, int32_t nq, int32_t P, int32_t n_prune, int32_t k,
                        int64_t max_candidates, Params *out)
{
    if (!ix) return fail(CHIMERA_INVALID_ARG, "index is NULL");
    if (B < 1 || B > 65535) return fail(CHIMERA_INVALID_ARG, "n_queries must be in [1, 65535], got %d", B);
    if (nq < 1 || nq > CHIMERA_MAX_QLEN) return fail(CHIMERA_INVALID_ARG, "q_len must be in [1, %d], got %d", CHIMERA_MAX_QLEN, nq);
    if (P < 1 || P > CHIMERA_MAX_NPROBE || P > ix->K)
        return fail(CHIMERA_INVALID_ARG, "nprobe must be in [1, min(n_centroids, %d)], got %d", CHIMERA_MAX_NPROBE, P);
    if (n_prune < 1 || n_prune > CHIMERA_MAX_NPRUNE)
        return fail(CHIMERA_INVALID_ARG, "n_prune must be in [1, %d], got %d", CHIMERA_MAX_NPRUNE, n_prune);
    if (k < 1 || k > CHIMERA_MAX_K) return fail(CHIMERA_INVALID_ARG, "k must be in [1, %d], got %d", CHIMERA_MAX_K, k);
    if (max_candidates < 0) return fail(CHIMERA_INVALID_ARG, "max_candidates must be >= 0");
    out->B = B; out->nq = nq; out->P = P; out->n_prune = n_prune; out->k = k;
    out->maxc = (max_candidates == 0 || max_candidates > ix->N) ? ix->N : max_candidates;
    return CHIMERA_OK;
}

// ------------------------------------------------------------------------------------------------ pipeline -------
static int copy_d2d(void *dst, const void *src, size_t bytes, cudaStream_t st)
{
    if (bytes == 0) return CHIMERA_OK;
    CHIMERA_CUDA(cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToDevice, st));
    return CHIMERA_OK;
}

static int run(const Index &ix, const Params &p, int first, int last, const float *queries, void *workspace,
               size_t workspace_bytes, cudaStream_t st, const chimera_taps *taps, int32_t *out_ids, float *out_scores,
               bool partial = false, bool rabitq = false, bool resume = false, const GraphSearch *graph = nullptr)
{
    // graph: the probes come from a search of the centroid graph; stage 1 and stage 2a do not run (only the RaBitQ
    // pipeline can do without the score table)
    if (graph && (!rabitq || first > 1)) return fail(CHIMERA_INVALID_ARG, "graph probes are for the RaBitQ pipeline");
    if (graph) {
        const int grc = check_graph_params(ix, *graph, p.P);
        if (grc) return grc;
    }
    // resume: stages before `first` ran in an earlier call on this workspace with the same parameters and their
    // results are still there (document-sharded search: the exchange happens between the two calls)
    if (partial && !ix.tok_id)
        return fail(CHIMERA_INVALID_ARG, "partial-score refinement needs chimera_index_enable_partial first");
    if (rabitq && (!ix.rot_t || !residual_umma_supported(p.nq)))
        return fail(CHIMERA_INVALID_ARG, "the RaBitQ pipeline needs chimera_index_attach_rabitq and q_len <= 64");
    if (!workspace || ((uintptr_t)workspace & 255)) return fail(CHIMERA_INVALID_ARG, "workspace is NULL or not 256-byte aligned");
    const Layout L = make_layout(ix, p);
    if (workspace_bytes < L.total)
        return fail(CHIMERA_WORKSPACE_TOO_SMALL, "workspace has %zu bytes, %zu needed", workspace_bytes, L.total);
    if ((first <= 1 || (first <= 4 && last >= 4)) && (!queries || ((uintptr_t)queries & 15)))
        return fail(CHIMERA_INVALID_ARG, "queries is NULL or not 16-byte aligned");
    if (last >= 5 && (!out_ids || !out_scores)) return fail(CHIMERA_INVALID_ARG, "out_ids / out_scores is NULL");

    char *ws = (char *)workspace;
    uint32_t *status = (uint32_t *)(ws + L.status);
    int8_t *qdig = (int8_t *)(ws + L.qdig);
    int32_t *table = (int32_t *)(ws + L.table);
    unsigned long long *part = (unsigned long long *)(ws + L.part);
    int32_t *probes = (int32_t *)(ws + L.probes);
    uint32_t *bitmap = (uint32_t *)(ws + L.bitmap);
    int32_t *chunk_cnt = (int32_t *)(ws + L.chunk_cnt);
    int32_t *cand = (int32_t *)(ws + L.cand);
    int32_t *n_cand = (int32_t *)(ws + L.n_cand);
    int32_t *ci = (int32_t *)(ws + L.ci);
    const bool two_phase = coarse_supported(p.nq) && !partial && !rabitq;
    uint8_t *table8 = two_phase ? (uint8_t *)(ws + L.table8) : nullptr;
    int32_t *lo = (int32_t *)(ws + L.lo);
    int32_t *hi = (int32_t *)(ws + L.hi);
    int32_t *cont = (int32_t *)(ws + L.cont);
    int32_t *n_cont = (int32_t *)(ws + L.n_cont);
    int32_t *pruned = (int32_t *)(ws + L.pruned);
    int32_t *n_pruned = (int32_t *)(ws + L.n_pruned);
    int32_t *pruned_ci = (int32_t *)(ws + L.pruned_ci);
    int32_t *sel_scratch = select_split_used(ix, p) ? (int32_t *)(ws + L.sel_scratch) : nullptr;
    int32_t *word_rank = (int32_t *)(ws + L.word_rank);
    int32_t *partial_m = (int32_t *)(ws + L.partial_m);
    float *q_rot = (float *)(ws + L.q_rot);
    int8_t *qdig_rot = (int8_t *)(ws + L.qdig_rot);
    float *score4 = (float *)(ws + L.score4);

    const size_t B = (size_t)p.B;
    const size_t table_bytes = B * (size_t)ix.K * p.nq * sizeof(int32_t);
    const size_t cand_bytes = B * (size_t)p.maxc * sizeof(int32_t);
    const size_t pruned_bytes = B * p.n_prune * sizeof(int32_t);
    int rc;

    prof_begin(st);
    // a resumed call continues an earlier one: the status bits that one set stay, new ones are OR-ed in
    if (!resume) CHIMERA_CUDA(cudaMemsetAsync(status, 0, 64 * sizeof(uint32_t), st));
    if (!resume && (rc = debug_begin_search(ix, p, L, workspace, st))) return rc;      // debug builds only

    // results of the stages that do not run come from the caller
    if (first > 1 && !resume) {
        if (!taps) return fail(CHIMERA_INVALID_ARG, "taps are required when first_stage > 1");
        if (first <= 4) {       // stages 2-4 read the score table
            if (!taps->score_table) return fail(CHIMERA_INVALID_ARG, "taps->score_table is required");
            if ((rc = copy_d2d(table, taps->score_table, table_bytes, st))) return rc;
        }
        if (first == 3) {
            if (!taps->cand || !taps->n_cand) return fail(CHIMERA_INVALID_ARG, "taps->cand / n_cand are required");
            if ((rc = copy_d2d(cand, taps->cand, cand_bytes, st))) return rc;
            if ((rc = copy_d2d(n_cand, taps->n_cand, B * sizeof(int32_t), st))) return rc;
        }
        if (first >= 4) {
            if (!taps->pruned || !taps->n_pruned) return fail(CHIMERA_INVALID_ARG, "taps->pruned / n_pruned are required");
            if ((rc = copy_d2d(pruned, taps->pruned, pruned_bytes, st))) return rc;
            if ((rc = copy_d2d(n_pruned, taps->n_pruned, B * sizeof(int32_t), st))) return rc;
        }
        if (first == 5) {
            if (!taps->score4) return fail(CHIMERA_INVALID_ARG, "taps->score4 is required");
            if ((rc = copy_d2d(score4, taps->score4, B * p.n_prune * sizeof(float), st))) return rc;
        }
    }
    prof_mark(SLOT_MISC, st);

    // stages 1 and 2a of one call run together when the layout provides for it: the probes come out of the score
    // table's epilogue and the table is not read again
    const bool together = first <= 1 && last >= 2 && !graph && L.pq_stride > 0;
    if (first <= 1 && last >= 1 && !graph) {
        if (together)
            rc = launch_score_table_probes(ix, p, L, queries, qdig, table, table8, ws, status, st);
        else
            rc = launch_score_table(ix, p, queries, qdig, table, table8, status, st);
        if (rc) return rc;
        prof_mark(SLOT_G1, st);
    }
    if (first <= 2 && last >= 2) {
        if (graph) {
            if ((rc = launch_graph_probes(ix, queries, (int64_t)p.B * p.nq, p.P, *graph, (uint32_t *)(ws + L.graph_vis),
                                          probes, nullptr, nullptr, st)))
                return rc;
        } else if (together) {
            if ((rc = launch_probe_merge(ix, p, L, table, ws, st))) return rc;
        } else if ((rc = launch_probes(ix, p, L, table, part, probes, st))) {
            return rc;
        }
        prof_mark(SLOT_PROBE, st);
        if ((rc = launch_gather(ix, p, L, probes, bitmap, chunk_cnt, cand, n_cand, word_rank, status, st))) return rc;
        prof_mark(SLOT_GATHER, st);
    }
    if (first <= 3 && last >= 3) {
        if (rabitq) {
            // the paper's pipeline on its own codec: rotate the queries, refine by partial 1-bit scores
            if ((rc = launch_rotate(ix, p, queries, q_rot, st))) return rc;
            if ((rc = launch_digits(q_rot, (int64_t)p.B * p.nq, ix.D, qdig_rot, status, st))) return rc;
            count_launch(SLOT_G1);
            prof_mark(SLOT_G1, st);
            if ((rc = launch_rabitq_partial(ix, p, L, q_rot, probes, bitmap, word_rank, n_cand, partial_m, ci, st)))
                return rc;
            prof_mark(SLOT_CI, st);
            if ((rc = launch_select(ix, p, cand, n_cand, ci, pruned, n_pruned, pruned_ci, sel_scratch, st))) return rc;
            prof_mark(SLOT_SELECT, st);
        } else if (partial) {
            // the paper's candidate refinement: partial scores from the retrieved tokens only, then the same selection
            if ((rc = launch_partial_scores(ix, p, L, queries, table, probes, bitmap, word_rank, n_cand, partial_m, ci,
                                            status, st)))
                return rc;
            prof_mark(SLOT_CI, st);
            if ((rc = launch_select(ix, p, cand, n_cand, ci, pruned, n_pruned, pruned_ci, sel_scratch, st))) return rc;
            prof_mark(SLOT_SELECT, st);
        } else if (two_phase) {
            if (first > 1) {                       // the table came from the caller: derive its coarse copy
                if ((rc = launch_coarse_table(ix, p, table, table8, st))) return rc;
                prof_mark(SLOT_MISC, st);
            }
            // bounds for every candidate, contenders for the top n_prune, exact CI and selection among those
            if ((rc = launch_coarse_bounds(ix, p, table8, cand, n_cand, lo, hi, (int2 *)(ws + L.cand_rng), st))) return rc;
            prof_mark(SLOT_CI, st);
            if ((rc = launch_contenders(ix, p, cand, n_cand, lo, hi, cont, n_cont, ci, (const int2 *)(ws + L.cand_rng),
                                        (int2 *)(ws + L.cont_rng), st))) return rc;
            prof_mark(SLOT_SELECT, st);
            // blocks per query for the few contenders (typically two to three times n_prune documents): one per SM
            // in a large batch, more when n_prune is large (about one block per eight survivors wanted; Large,
            // n_prune 4096: 2.75 ms with 444-592 blocks against 3.26 ms with 148, Mid unchanged), four per SM when a
            // single query has the GPU to itself
            int exact_blocks = (4 * ix.sm_count + p.B - 1) / p.B;
            if (exact_blocks < ix.sm_count) exact_blocks = ix.sm_count;
            if (exact_blocks < p.n_prune / 8) exact_blocks = p.n_prune / 8;
            if ((rc = launch_centroid_interaction(ix, p, table, cont, n_cont, ci, exact_blocks, SLOT_CI_EXACT,
                                                  ix.T < 0x7fffffffLL ? (const int2 *)(ws + L.cont_rng) : nullptr, st)))
                return rc;
            prof_mark(SLOT_CI_EXACT, st);
            if ((rc = launch_select(ix, p, cont, n_cont, ci, pruned, n_pruned, pruned_ci, nullptr, st))) return rc;
            prof_mark(SLOT_SELECT, st);
        } else {
            if ((rc = launch_centroid_interaction(ix, p, table, cand, n_cand, ci, 0, SLOT_CI, nullptr, st))) return rc;
            prof_mark(SLOT_CI, st);
            if ((rc = launch_select(ix, p, cand, n_cand, ci, pruned, n_pruned, pruned_ci, sel_scratch, st))) return rc;
            prof_mark(SLOT_SELECT, st);
        }
    }
    if (first <= 4 && last >= 4) {
        if (rabitq) {
            if ((rc = launch_rabitq_scores_umma(ix, p, q_rot, qdig_rot, pruned, score4, status, st))) return rc;
        } else if (residual_umma_supported(p.nq)) {
            if (first > 1) {                       // stage 1 did not run in this call: build the query digit planes
                if ((rc = launch_digits(queries, (int64_t)p.B * p.nq, ix.D, qdig, status, st))) return rc;
                count_launch(SLOT_G4);
            }
            if ((rc = launch_residual_scores_umma(ix, p, queries, qdig, table, pruned, score4, status, st))) return rc;
        } else if ((rc = launch_residual_scores(ix, p, queries, table, pruned, score4, st))) {
            return rc;
        }
        prof_mark(SLOT_G4, st);
    }
    if (last >= 5) {
        if ((rc = launch_topk(ix, p, pruned, score4, out_ids, out_scores, st))) return rc;
        prof_mark(SLOT_TOPK, st);
    }

    if (taps) {
        if (taps->score_table && first <= 1 && last >= 1 && !graph &&
            (rc = copy_d2d(taps->score_table, table, table_bytes, st)))
            return rc;
        if (first <= 2 && last >= 2) {
            if (taps->probes && (rc = copy_d2d(taps->probes, probes, B * p.nq * p.P * sizeof(int32_t), st))) return rc;
            if (taps->cand && (rc = copy_d2d(taps->cand, cand, cand_bytes, st))) return rc;
            if (taps->n_cand && (rc = copy_d2d(taps->n_cand, n_cand, B * sizeof(int32_t), st))) return rc;
        }
        if (first <= 3 && last >= 3) {
            if (taps->ci) {
                if (two_phase) {                   // the search only needed exact CI for the contenders: the tap asks
                                                   // for every candidate, so the exact kernel runs over all of them
                    if ((rc = launch_centroid_interaction(ix, p, table, cand, n_cand, taps->ci, 0, SLOT_MISC, nullptr, st)))
                        return rc;
                } else if ((rc = copy_d2d(taps->ci, ci, cand_bytes, st))) return rc;
            }
            if (taps->n_contenders &&
                (rc = copy_d2d(taps->n_contenders, two_phase ? n_cont : n_cand, B * sizeof(int32_t), st)))
                return rc;
            if (taps->pruned && (rc = copy_d2d(taps->pruned, pruned, pruned_bytes, st))) return rc;
            if (taps->n_pruned && (rc = copy_d2d(taps->n_pruned, n_pruned, B * sizeof(int32_t), st))) return rc;
        }
        if (first <= 4 && last >= 4 && taps->score4 &&
            (rc = copy_d2d(taps->score4, score4, B * p.n_prune * sizeof(float), st)))
            return rc;
        prof_mark(SLOT_MISC, st);
    }
    return CHIMERA_OK;
}

}  // namespace chimera

using namespace chimera;

// ================================================================================================ C ABI ==========
extern "C" {

int chimera_version(void) { return 100; }

const char *chimera_last_error(void) { return g_err; }

int chimera_build_index(const chimera_index_desc *desc, const float *centroids, const int32_t *cids,
                        const uint8_t *codes, const int32_t *doclens, void *stream, chimera_index **out)
{
    if (out) *out = nullptr;
    if (!desc || !centroids || !cids || !codes || !doclens || !out) return fail(CHIMERA_INVALID_ARG, "NULL argument");
    if (desc->n_centroids < 1 || desc->n_docs < 1 || desc->n_tokens < 1)
        return fail(CHIMERA_INVALID_ARG, "n_centroids, n_docs and n_tokens must be >= 1");
    if (desc->n_centroids > 0x7fffffffLL || desc->n_docs > 0x7fffffffLL)
        return fail(CHIMERA_UNSUPPORTED, "n_centroids and n_docs must fit int32");
    if (desc->dim < 32 || desc->dim > 128 || desc->dim % 32) return fail(CHIMERA_UNSUPPORTED, "dim must be 32, 64, 96 or 128, got %d", desc->dim);
    if (desc->nbits != 1 && desc->nbits != 2) return fail(CHIMERA_UNSUPPORTED, "nbits must be 1 or 2, got %d", desc->nbits);
    if (!(desc->res_hi > desc->res_lo)) return fail(CHIMERA_INVALID_ARG, "res_hi must exceed res_lo");
    if (((uintptr_t)cids & 3) || ((uintptr_t)codes & 31) || ((uintptr_t)centroids & 15))
        return fail(CHIMERA_INVALID_ARG, "centroids must be 16-byte aligned and codes 32-byte aligned");

    Index *ix = new (std::nothrow) Index();
    if (!ix) return fail(CHIMERA_CUDA_ERROR, "out of host memory");
    cudaError_t e = cudaGetDevice(&ix->device);
    cudaDeviceProp prop;
    if (e == cudaSuccess) e = cudaGetDeviceProperties(&prop, ix->device);
    if (e != cudaSuccess) {
        delete ix;
        return fail(CHIMERA_CUDA_ERROR, "no usable CUDA device: %s", cudaGetErrorString(e));
    }
    if (prop.major != 10) {
        delete ix;
        return fail(CHIMERA_UNSUPPORTED, "device is sm_%d%d; this library is built for sm_100a only", prop.major, prop.minor);
    }
    ix->sm_count = prop.multiProcessorCount;
    ix->D = desc->dim;
    ix->nbits = desc->nbits;
    ix->CB = desc->dim * desc->nbits / 8;
    ix->K = desc->n_centroids;
    ix->N = desc->n_docs;
    ix->T = desc->n_tokens;
    ix->res_lo = desc->res_lo;
    ix->res_hi = desc->res_hi;
    ix->cids = cids;
    ix->codes = codes;
    int rc = build_index_device(*ix, centroids, doclens, (cudaStream_t)stream);
    if (rc) {
        chimera_destroy_index(reinterpret_cast<chimera_index *>(ix));
        return rc;
    }
    *out = reinterpret_cast<chimera_index *>(ix);
    return CHIMERA_OK;
}

int chimera_index_enable_partial(chimera_index *index, void *stream)
{
    Index *ix = reinterpret_cast<Index *>(index);
    if (!ix) return fail(CHIMERA_INVALID_ARG, "index is NULL");
    return build_token_lists(*ix, (cudaStream_t)stream);
}

int chimera_search_partial(const chimera_index *index, const float *queries, int32_t n_queries, int32_t q_len,
                           int32_t nprobe, int32_t n_prune, int32_t k, int64_t max_candidates, void *workspace,
                           size_t workspace_bytes, void *stream, int32_t *out_ids, float *out_scores,
                           const chimera_taps *taps)
{
    const Index *ix = reinterpret_cast<const Index *>(index);
    Params p;
    int rc = check_params(ix, n_queries, q_len, nprobe, n_prune, k, max_candidates, &p);
    if (rc) return rc;
    return run(*ix, p, 1, 5, queries, workspace, workspace_bytes, (cudaStream_t)stream, taps, out_ids, out_scores,
               true);
}

int chimera_index_attach_rabitq(chimera_index *index, const float *rotation, const uint8_t *bits,
                                const float *inv_dot, void *stream)
{
    Index *ix = reinterpret_cast<Index *>(index);
    if (!ix || !rotation || !bits || !inv_dot) return fail(CHIMERA_INVALID_ARG, "NULL argument");
    if (((uintptr_t)bits & 15) || ((uintptr_t)inv_dot & 3)) return fail(CHIMERA_INVALID_ARG, "bits must be 16-byte aligned");
    int rc = build_token_lists(*ix, (cudaStream_t)stream);
    if (rc) return rc;
    rc = attach_rabitq(*ix, rotation, (cudaStream_t)stream);
    if (rc) return rc;
    ix->rq_bits = bits;
    ix->rq_inv = inv_dot;
    return CHIMERA_OK;
}

int chimera_search_rabitq(const chimera_index *index, const float *queries, int32_t n_queries, int32_t q_len,
                          int32_t nprobe, int32_t k_refine, int32_t k, int64_t max_candidates, void *workspace,
                          size_t workspace_bytes, void *stream, int32_t *out_ids, float *out_scores,
                          const chimera_taps *taps)
{
    const Index *ix = reinterpret_cast<const Index *>(index);
    Params p;
    int rc = check_params(ix, n_queries, q_len, nprobe, k_refine, k, max_candidates, &p);
    if (rc) return rc;
    return run(*ix, p, 1, 5, queries, workspace, workspace_bytes, (cudaStream_t)stream, taps, out_ids, out_scores,
               false, true);
}

// ---- centroid graph ---------------------------------------------------------------------------------------------
int chimera_index_build_graph(chimera_index *index, const float *centroids, int32_t degree, void *stream)
{
    Index *ix = reinterpret_cast<Index *>(index);
    if (!ix || !centroids) return fail(CHIMERA_INVALID_ARG, "NULL argument");
    if ((uintptr_t)centroids & 15) return fail(CHIMERA_INVALID_ARG, "centroids must be 16-byte aligned");
    return build_graph(*ix, centroids, degree, (cudaStream_t)stream);
}

int chimera_index_copy_graph(const chimera_index *index, int32_t *out_graph, int32_t *out_degree, void *stream)
{
    const Index *ix = reinterpret_cast<const Index *>(index);
    if (!ix || !out_degree) return fail(CHIMERA_INVALID_ARG, "NULL argument");
    *out_degree = ix->graph_deg;
    if (out_graph && ix->graph)
        CHIMERA_CUDA(cudaMemcpyAsync(out_graph, ix->graph, sizeof(int32_t) * (size_t)ix->K * ix->graph_deg,
                                     cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
    return CHIMERA_OK;
}

int chimera_graph_scratch_bytes(const chimera_index *index, int32_t n_queries, int32_t q_len, size_t *out)
{
    const Index *ix = reinterpret_cast<const Index *>(index);
    if (!ix || !out) return fail(CHIMERA_INVALID_ARG, "NULL argument");
    if (n_queries < 1 || q_len < 1 || q_len > CHIMERA_MAX_QLEN) return fail(CHIMERA_INVALID_ARG, "n_queries or q_len out of range");
    *out = graph_scratch_bytes(*ix, (int64_t)n_queries * q_len);
    return CHIMERA_OK;
}

int chimera_graph_probes(const chimera_index *index, const float *queries, int32_t n_queries, int32_t q_len,
                         int32_t nprobe, int32_t beam, int32_t n_entries, int32_t max_expansions, void *scratch,
                         size_t scratch_bytes, void *stream, int32_t *out_probes, int32_t *out_scores,
                         int32_t *out_n_visited)
{
    const Index *ix = reinterpret_cast<const Index *>(index);
    if (!ix || !queries || !scratch || !out_probes) return fail(CHIMERA_INVALID_ARG, "NULL argument");
    if ((uintptr_t)queries & 15) return fail(CHIMERA_INVALID_ARG, "queries must be 16-byte aligned");
    if (n_queries < 1 || q_len < 1 || q_len > CHIMERA_MAX_QLEN || nprobe < 1 || nprobe > CHIMERA_MAX_NPROBE)
        return fail(CHIMERA_INVALID_ARG, "n_queries, q_len or nprobe out of range");
    GraphSearch g;
    g.beam = beam; g.n_entries = n_entries; g.max_expansions = max_expansions;
    int rc = check_graph_params(*ix, g, nprobe);
    if (rc) return rc;
    const int64_t tokens = (int64_t)n_queries * q_len;
    if (scratch_bytes < graph_scratch_bytes(*ix, tokens))
        return fail(CHIMERA_WORKSPACE_TOO_SMALL, "scratch has %zu bytes, %zu needed", scratch_bytes, graph_scratch_bytes(*ix, tokens));
    return launch_graph_probes(*ix, queries, tokens, nprobe, g, (uint32_t *)scratch, out_probes, out_scores, out_n_visited,
                               (cudaStream_t)stream);
}

int chimera_search_rabitq_graph(const chimera_index *index, const float *queries, int32_t n_queries, int32_t q_len,
                                int32_t nprobe, int32_t k_refine, int32_t k, int64_t max_candidates, int32_t beam,
                                int32_t n_entries, int32_t max_expansions, void *workspace, size_t workspace_bytes,
                                void *stream, int32_t *out_ids, float *out_scores, const chimera_taps *taps)
{
    const Index *ix = reinterpret_cast<const Index *>(index);
    Params p;
    int rc = check_params(ix, n_queries, q_len, nprobe, k_refine, k, max_candidates, &p);
    if (rc) return rc;
    GraphSearch g;
    g.beam = beam; g.n_entries = n_entries; g.max_expansions = max_expansions;
    return run(*ix, p, 1, 5, queries, workspace, workspace_bytes, (cudaStream_t)stream, taps, out_ids, out_scores,
               false, true, false, &g);
}

// ---- document-sharded search ------------------------------------------------------------------------------------
static int shard_mode(int32_t mode, bool *partial, bool *rabitq)
{
    if (mode < 0 || mode > 2) return fail(CHIMERA_INVALID_ARG, "mode must be 0 (centroid interaction), 1 (partial scores) or 2 (RaBitQ)");
    *partial = mode == 1;
    *rabitq = mode == 2;
    return CHIMERA_OK;
}

int chimera_shard_local(const chimera_index *index, const float *queries, int32_t n_queries, int32_t q_len,
                        int32_t nprobe, int32_t n_prune, int32_t k, int64_t max_candidates, int32_t mode,
                        int64_t doc_base, void *workspace, size_t workspace_bytes, void *stream, int32_t *out_ids,
                        int32_t *out_scores3)
{
    const Index *ix = reinterpret_cast<const Index *>(index);
    Params p;
    bool partial = false, rabitq = false;
    int rc = check_params(ix, n_queries, q_len, nprobe, n_prune, k, max_candidates, &p);
    if (rc || (rc = shard_mode(mode, &partial, &rabitq))) return rc;
    if (!out_ids || !out_scores3) return fail(CHIMERA_INVALID_ARG, "out_ids / out_scores3 is NULL");
    if (doc_base < 0 || doc_base + ix->N > 0x7fffffffLL) return fail(CHIMERA_INVALID_ARG, "global document ids must fit int32");
    cudaStream_t st = (cudaStream_t)stream;
    if ((rc = run(*ix, p, 1, 3, queries, workspace, workspace_bytes, st, nullptr, nullptr, nullptr, partial, rabitq)))
        return rc;
    const Layout L = make_layout(*ix, p);
    char *ws = (char *)workspace;
    return launch_shard_export(p, (const int32_t *)(ws + L.pruned), (const int32_t *)(ws + L.pruned_ci), doc_base,
                               out_ids, out_scores3, st);
}

int chimera_shard_finish(const chimera_index *index, const float *queries, int32_t n_queries, int32_t q_len,
                         int32_t nprobe, int32_t n_prune, int32_t k, int64_t max_candidates, int32_t mode,
                         int64_t doc_base, int32_t world, const int32_t *all_ids, const int32_t *all_scores3,
                         void *workspace, size_t workspace_bytes, void *stream, int32_t *out_ids, float *out_scores)
{
    const Index *ix = reinterpret_cast<const Index *>(index);
    Params p;
    bool partial = false, rabitq = false;
    int rc = check_params(ix, n_queries, q_len, nprobe, n_prune, k, max_candidates, &p);
    if (rc || (rc = shard_mode(mode, &partial, &rabitq))) return rc;
    if (world < 1 || (int64_t)world * n_prune > 0x7fffffffLL) return fail(CHIMERA_INVALID_ARG, "world out of range");
    if (!all_ids || !all_scores3 || !out_ids || !out_scores) return fail(CHIMERA_INVALID_ARG, "NULL argument");
    if (!workspace || ((uintptr_t)workspace & 255)) return fail(CHIMERA_INVALID_ARG, "workspace is NULL or not 256-byte aligned");
    const Layout L = make_layout(*ix, p);
    if (workspace_bytes < L.total)
        return fail(CHIMERA_WORKSPACE_TOO_SMALL, "workspace has %zu bytes, %zu needed", workspace_bytes, L.total);
    cudaStream_t st = (cudaStream_t)stream;
    char *ws = (char *)workspace;
    if ((rc = launch_shard_select(p, all_ids, all_scores3, world, doc_base, ix->N, (int32_t *)(ws + L.pruned),
                                  (int32_t *)(ws + L.n_pruned), st)))
        return rc;
    if ((rc = run(*ix, p, 4, 5, queries, workspace, workspace_bytes, st, nullptr, out_ids, out_scores, partial, rabitq,
                  true)))
        return rc;
    return launch_add_base(out_ids, (int64_t)p.B * p.k, doc_base, st);
}

int chimera_shard_merge_topk(const int32_t *all_ids, const float *all_scores, int32_t world, int32_t n_queries,
                             int32_t k, void *stream, int32_t *out_ids, float *out_scores)
{
    if (!all_ids || !all_scores || !out_ids || !out_scores) return fail(CHIMERA_INVALID_ARG, "NULL argument");
    if (world < 1 || n_queries < 1 || n_queries > 65535 || k < 1 || k > CHIMERA_MAX_K)
        return fail(CHIMERA_INVALID_ARG, "world, n_queries or k out of range");
    if ((int64_t)world * k > 16384)
        return fail(CHIMERA_UNSUPPORTED, "world * k = %lld entries per query exceed the 16384 the merge holds",
                    (long long)world * k);
    return launch_shard_merge_topk(all_ids, all_scores, world, n_queries, k, out_ids, out_scores, (cudaStream_t)stream);
}

int chimera_destroy_index(chimera_index *index)
{
    Index *ix = reinterpret_cast<Index *>(index);
    if (!ix) return CHIMERA_OK;
    cudaFree(ix->graph);
    cudaFree(ix->xc);
    cudaFree(ix->rot_t);
    cudaFree(ix->tok_off);
    cudaFree(ix->tok_id);
    cudaFree(ix->tok_doc);
    cudaFree(ix->doc_off);
    cudaFree(ix->cdig);
    cudaFree(ix->ivf_off);
    cudaFree(ix->ivf_doc);
    delete ix;
    return CHIMERA_OK;
}

int chimera_index_info(const chimera_index *index, chimera_index_desc *desc, int64_t *posting_entries,
                       int32_t *max_doclen)
{
    const Index *ix = reinterpret_cast<const Index *>(index);
    if (!ix) return fail(CHIMERA_INVALID_ARG, "index is NULL");
    if (desc) {
        desc->dim = ix->D; desc->nbits = ix->nbits; desc->res_lo = ix->res_lo; desc->res_hi = ix->res_hi;
        desc->n_centroids = ix->K; desc->n_docs = ix->N; desc->n_tokens = ix->T;
    }
    if (posting_entries) *posting_entries = ix->ivf_len;
    if (max_doclen) *max_doclen = ix->max_doclen;
    return CHIMERA_OK;
}

int chimera_workspace_bytes(const chimera_index *index, int32_t n_queries, int32_t q_len, int32_t nprobe,
                            int32_t n_prune, int32_t k, int64_t max_candidates, size_t *out)
{
    const Index *ix = reinterpret_cast<const Index *>(index);
    Params p;
    int rc = check_params(ix, n_queries, q_len, nprobe, n_prune, k, max_candidates, &p);
    if (rc) return rc;
    if (!out) return fail(CHIMERA_INVALID_ARG, "out is NULL");
    *out = make_layout(*ix, p).total;
    return CHIMERA_OK;
}

int chimera_search_tapped(const chimera_index *index, const float *queries, int32_t n_queries, int32_t q_len,
                          int32_t nprobe, int32_t n_prune, int32_t k, int64_t max_candidates, void *workspace,
                          size_t workspace_bytes, void *stream, int32_t *out_ids, float *out_scores,
                          const chimera_taps *taps)
{
    const Index *ix = reinterpret_cast<const Index *>(index);
    Params p;
    int rc = check_params(ix, n_queries, q_len, nprobe, n_prune, k, max_candidates, &p);
    if (rc) return rc;
    return run(*ix, p, 1, 5, queries, workspace, workspace_bytes, (cudaStream_t)stream, taps, out_ids, out_scores);
}

int chimera_search(const chimera_index *index, const float *queries, int32_t n_queries, int32_t q_len,
                   int32_t nprobe, int32_t n_prune, int32_t k, int64_t max_candidates, void *workspace,
                   size_t workspace_bytes, void *stream, int32_t *out_ids, float *out_scores)
{
    return chimera_search_tapped(index, queries, n_queries, q_len, nprobe, n_prune, k, max_candidates, workspace,
                                 workspace_bytes, stream, out_ids, out_scores, nullptr);
}

int chimera_search_host(const chimera_index *index, const float *queries_host, int32_t n_queries, int32_t q_len,
                        int32_t nprobe, int32_t n_prune, int32_t k, int64_t max_candidates, void *workspace,
                        size_t workspace_bytes, void *stream, int32_t *out_ids_host, float *out_scores_host)
{
    const Index *ix = reinterpret_cast<const Index *>(index);
    Params p;
    int rc = check_params(ix, n_queries, q_len, nprobe, n_prune, k, max_candidates, &p);
    if (rc) return rc;
    if (!queries_host || !out_ids_host || !out_scores_host) return fail(CHIMERA_INVALID_ARG, "NULL host buffer");
    if (!workspace || ((uintptr_t)workspace & 255)) return fail(CHIMERA_INVALID_ARG, "workspace is NULL or not 256-byte aligned");
    const Layout L = make_layout(*ix, p);
    if (workspace_bytes < L.total)
        return fail(CHIMERA_WORKSPACE_TOO_SMALL, "workspace has %zu bytes, %zu needed", workspace_bytes, L.total);
    cudaStream_t st = (cudaStream_t)stream;
    char *ws = (char *)workspace;
    float *dq = (float *)(ws + L.q_stage);
    int32_t *dids = (int32_t *)(ws + L.out_ids);
    float *dsc = (float *)(ws + L.out_scores);
    const size_t qbytes = (size_t)p.B * p.nq * ix->D * sizeof(float);
    CHIMERA_CUDA(cudaMemcpyAsync(dq, queries_host, qbytes, cudaMemcpyHostToDevice, st));
    rc = run(*ix, p, 1, 5, dq, workspace, workspace_bytes, st, nullptr, dids, dsc);
    if (rc) return rc;
    CHIMERA_CUDA(cudaMemcpyAsync(out_ids_host, dids, (size_t)p.B * p.k * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    CHIMERA_CUDA(cudaMemcpyAsync(out_scores_host, dsc, (size_t)p.B * p.k * sizeof(float), cudaMemcpyDeviceToHost, st));
    CHIMERA_CUDA(cudaStreamSynchronize(st));
    return CHIMERA_OK;
}

int chimera_run_stages(const chimera_index *index, int32_t first_stage, int32_t last_stage, const float *queries,
                       int32_t n_queries, int32_t q_len, int32_t nprobe, int32_t n_prune, int32_t k,
                       int64_t max_candidates, void *workspace, size_t workspace_bytes, void *stream,
                       const chimera_taps *inout, int32_t *out_ids, float *out_scores)
{
    const Index *ix = reinterpret_cast<const Index *>(index);
    Params p;
    int rc = check_params(ix, n_queries, q_len, nprobe, n_prune, k, max_candidates, &p);
    if (rc) return rc;
    if (first_stage < 1 || last_stage > 5 || first_stage > last_stage)
        return fail(CHIMERA_INVALID_ARG, "stages must satisfy 1 <= first <= last <= 5");
    return run(*ix, p, first_stage, last_stage, queries, workspace, workspace_bytes, (cudaStream_t)stream, inout,
               out_ids, out_scores);
}

int chimera_workspace_status(const void *workspace, void *stream, int32_t *status)
{
    if (!workspace || !status) return fail(CHIMERA_INVALID_ARG, "NULL argument");
    uint32_t bits = 0;
    CHIMERA_CUDA(cudaMemcpyAsync(&bits, workspace, sizeof(bits), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    CHIMERA_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
    if (bits & ST_BAD_INDEX) *status = CHIMERA_DEBUG_CHECK_FAILED;
    else if (bits & ST_TIMEOUT) *status = CHIMERA_TIMEOUT;
    else if (bits & ST_BAD_QUERY) *status = CHIMERA_INVALID_ARG;
    else if (bits & ST_OVERFLOW) *status = CHIMERA_CAPACITY_OVERFLOW;
    else *status = CHIMERA_OK;
    return CHIMERA_OK;
}

int chimera_probe_plan(const chimera_index *index, int32_t n_queries, int32_t q_len, int32_t nprobe,
                       int32_t *sample_stride)
{
    const Index *ix = reinterpret_cast<const Index *>(index);
    Params p;
    int rc = check_params(ix, n_queries, q_len, nprobe, 1, 1, 0, &p);
    if (rc) return rc;
    if (!sample_stride) return fail(CHIMERA_INVALID_ARG, "NULL argument");
    *sample_stride = probe_queue_stride(*ix, p);
    return CHIMERA_OK;
}

int chimera_is_debug_build(void)
{
#ifdef CHIMERA_DEBUG
    return 1;
#else
    return 0;
#endif
}

int chimera_workspace_check(const chimera_index *index, int32_t n_queries, int32_t q_len, int32_t nprobe,
                            int32_t n_prune, int32_t k, int64_t max_candidates, const void *workspace, void *stream,
                            int32_t *damaged_region)
{
    const Index *ix = reinterpret_cast<const Index *>(index);
    Params p;
    int rc = check_params(ix, n_queries, q_len, nprobe, n_prune, k, max_candidates, &p);
    if (rc) return rc;
    if (!workspace || !damaged_region) return fail(CHIMERA_INVALID_ARG, "NULL argument");
#ifdef CHIMERA_DEBUG
    const Layout L = make_layout(*ix, p);
    cudaStream_t st = (cudaStream_t)stream;
    uint32_t *status = reinterpret_cast<uint32_t *>((char *)workspace + L.status);
    GuardList g;
    g.n = L.n_guards;
    for (int i = 0; i < L.n_guards; ++i) g.off[i] = L.guards[i];
    CHIMERA_CUDA(cudaMemsetAsync(status + STATUS_WORD_CANARY, 0xff, sizeof(uint32_t), st));
    if (g.n > 0) guard_check_kernel<<<g.n, 64, 0, st>>>((const char *)workspace, g, status);
    CHIMERA_CUDA(cudaGetLastError());
    uint32_t first = 0xffffffffu;
    CHIMERA_CUDA(cudaMemcpyAsync(&first, status + STATUS_WORD_CANARY, sizeof(first), cudaMemcpyDeviceToHost, st));
    CHIMERA_CUDA(cudaStreamSynchronize(st));
    *damaged_region = first == 0xffffffffu ? -1 : (int32_t)first;
    return CHIMERA_OK;
#else
    (void)stream;
    *damaged_region = -1;
    return fail(CHIMERA_UNSUPPORTED, "this library was built without CHIMERA_DEBUG: the workspace has no guard regions");
#endif
}

int chimera_test_wait_fault(int32_t skip_loads, int64_t wait_cycles)
{
    g_skip_tma.store(skip_loads ? 1 : 0, std::memory_order_relaxed);
    g_wait_cycles.store(wait_cycles > 0 ? (long long)wait_cycles : 100000000LL, std::memory_order_relaxed);
    return CHIMERA_OK;
}

int chimera_profile_enable(int32_t on)
{
    g_prof_on = on != 0;
    return CHIMERA_OK;
}

int chimera_profile_read(float *ms, int64_t *launches)
{
    if (!ms || !launches) return fail(CHIMERA_INVALID_ARG, "NULL argument");
    for (int s = 0; s < CHIMERA_PROFILE_SLOTS; ++s) { ms[s] = 0.f; launches[s] = g_launches[s].exchange(0, std::memory_order_relaxed); }
    for (int c = 0; c < g_n_calls; ++c) {
        ProfCall &pc = g_calls[c];
        if (pc.n < 2) continue;
        CHIMERA_CUDA(cudaEventSynchronize(pc.ev[pc.n - 1]));
        for (int i = 1; i < pc.n; ++i) {
            float t = 0.f;
            CHIMERA_CUDA(cudaEventElapsedTime(&t, pc.ev[i - 1], pc.ev[i]));
            if (pc.slot[i] >= 0 && pc.slot[i] < CHIMERA_PROFILE_SLOTS) ms[pc.slot[i]] += t;
        }
        pc.n = 0;
    }
    g_n_calls = 0;
    g_cur = nullptr;
    return CHIMERA_OK;
}

}  // extern "C"
