/*
 * libchimera — GPU-resident late-interaction (MaxSim) retrieval over centroid + residual codes, for NVIDIA B200
 * (sm_100a).  C ABI: plain pointers and sizes, no C++ or framework types.
 *
 * Pipeline run by every search call, all on the device, on the caller's stream, with no host round trip between
 * stages (paper: Algorithm 1 skeleton "generate -> refine -> score -> top-k"; Definition 1 for every score):
 *   stage 1  score table      S[c,i] = <q_i, centroid_c> for all query tokens x all centroids, in exact Q.24
 *                             fixed point (Definition 1's inner product; integer so that later discrete choices do
 *                             not depend on summation order)
 *   stage 2  candidates       per query token the nprobe best centroids; union of their posting lists; the set of
 *                             documents owning at least one such token (Sec. 3.2 step 1, sets L_q and S)
 *   stage 3  pruning          CI(d) = sum_i max_{t in d} S[cid_t, i] (Chamfer aggregation rule of Sec. 4.2 applied
 *                             to centroid scores); keep the n_prune candidates with the largest CI
 *   stage 4  residual scores  score(d) = sum_i max_{t in d} <q_i, centroid_{cid_t} + residual(code_t)>
 *                             (Definition 1 on the decoded tokens)
 *   stage 5  top-k            the k best scores, best first (Definition 2, Eq. 1)
 * Ties are always broken towards the smaller id.
 *
 * Conventions
 *   - "device" pointers are CUDA global-memory addresses valid on the index's device; "host" pointers are ordinary
 *     process memory.  The caller owns every buffer it passes and keeps it alive until the work enqueued on the
 *     stream has finished.  The library owns only what chimera_build_index allocates inside the index.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *   - Every function returns a chimera_status; chimera_last_error() gives a text for the calling thread's last
 *     failure.  No function throws, traps the device, or leaves a kernel waiting on anything.
 *   - Search calls only enqueue work (they are asynchronous to the host) unless stated otherwise.
 *   - Searches on one index from several host threads are safe when each uses its own workspace and stream (the
 *     index is read-only after its build / enable / attach calls, which must not overlap a search); the profiling
 *     calls are for one thread.
 */
#ifndef CHIMERA_H
#define CHIMERA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    CHIMERA_OK = 0,
    CHIMERA_INVALID_ARG = 1,        /* bad pointer, size or parameter; nothing was enqueued */
    CHIMERA_CUDA_ERROR = 2,         /* a CUDA runtime call failed; text in chimera_last_error() */
    CHIMERA_WORKSPACE_TOO_SMALL = 3,
    CHIMERA_CAPACITY_OVERFLOW = 4,  /* a query produced more candidates than max_candidates (reported by status) */
    CHIMERA_TIMEOUT = 5,            /* a bounded device-side wait gave up after ~50 ms (reported by status) */
    CHIMERA_UNSUPPORTED = 6,        /* dim, nbits or a size outside the supported set */
    CHIMERA_DEBUG_CHECK_FAILED = 7  /* debug build only: a kernel met an index out of range and skipped it (reported
                                       by status) */
} chimera_status;

#define CHIMERA_MAX_NPROBE 64       /* nprobe per query token */
#define CHIMERA_MAX_QLEN 127        /* tokens per query (keeps sum_i max S[., i] inside int32) */
#define CHIMERA_MAX_NPRUNE 16384    /* n_prune */
#define CHIMERA_MAX_K 16384         /* k */

typedef struct chimera_index chimera_index; /* opaque */

/* Index-time description.  Residual codes are uniform `nbits`-bit bucket indices per dimension over
 * [res_lo, res_hi): value u decodes to res_lo + (u + 0.5) * (res_hi - res_lo) / 2^nbits.  Packing is little-endian
 * within a byte: 2-bit codes put dimension 4g+t in bits [2t, 2t+1] of byte g; 1-bit codes put dimension 8g+t in bit
 * t of byte g. */
typedef struct {
    int32_t dim;         /* multiple of 32, <= 128 (96 and 128 are the tuned cases) */
    int32_t nbits;       /* 1 or 2 */
    float res_lo;        /* e.g. -0.25f */
    float res_hi;        /* e.g. +0.25f */
    int64_t n_centroids; /* K >= 1 */
    int64_t n_docs;      /* N >= 1 */
    int64_t n_tokens;    /* T = sum of doclens */
} chimera_index_desc;

/* Library version as major*10000 + minor*100 + patch. */
int chimera_version(void);

/* Text of the calling thread's most recent failure ("" if none).  The pointer stays valid until that thread's next
 * failing call. */
const char *chimera_last_error(void);

/* Build the device-resident index (offline step; Sec. 3.1: centroids, posting lists, per-token codes).
 *   desc       host pointer.
 *   centroids  device, 16-byte aligned, [K, dim] float32 row-major, unit-norm rows (every |element| <= 1 and norm <= 1 + 2^-10:
 *              checked, INVALID_ARG otherwise).  Copied (as fixed-point
 *              digits); may be freed after the call returns.
 *   cids       device, [T] int32 in [0, K), document-major (document 0's tokens first).  REFERENCED, not copied:
 *              must outlive the index.
 *   codes      device, 32-byte aligned, [T, dim*nbits/8] uint8, document-major.  REFERENCED, not copied: must outlive
 *              the index.
 *   doclens    device, [N] int32, each >= 1, summing to T.  Copied (as prefix sums).
 *   stream     work is enqueued on it and the call synchronises it before returning.
 *   out        host pointer receiving the handle.
 * Allocates (cudaMalloc) prefix sums, centroid digits and an inverted file: for each centroid the unique ids of the
 * documents owning a token assigned to it, in unspecified order.
 * Errors: INVALID_ARG (null or misaligned pointer, sizes < 1, a cid outside [0,K), a doclen < 1, lengths not summing to T),
 * UNSUPPORTED (dim / nbits), CUDA_ERROR.  On error nothing stays allocated and *out is NULL. */
int chimera_build_index(const chimera_index_desc *desc, const float *centroids, const int32_t *cids,
                        const uint8_t *codes, const int32_t *doclens, void *stream, chimera_index **out);

/* Free everything the index owns (not the referenced cids / codes).  NULL is accepted. */
int chimera_destroy_index(chimera_index *index);

/* Bytes of device workspace a search call with these parameters needs.  max_candidates bounds the candidate list of
 * one query (0 = n_docs, which can never overflow).  out: host pointer.
 * Errors: INVALID_ARG / UNSUPPORTED for parameters outside: 1 <= q_len <= CHIMERA_MAX_QLEN,
 * 1 <= nprobe <= min(K, CHIMERA_MAX_NPROBE), 1 <= n_prune <= CHIMERA_MAX_NPRUNE, 1 <= k <= CHIMERA_MAX_K,
 * n_queries >= 1. */
int chimera_workspace_bytes(const chimera_index *index, int32_t n_queries, int32_t q_len, int32_t nprobe,
                            int32_t n_prune, int32_t k, int64_t max_candidates, size_t *out);

/* Stages 1-5 for a batch of queries (Algorithm 1 with the stage list at the top of this file).
 *   queries     device, 16-byte aligned, [n_queries, q_len, dim] float32, unit-norm rows (the library does not
 *               normalise; an element outside [-1, 1] or a row longer than 1 + 2^-10 is reported by
 *               chimera_workspace_status as CHIMERA_INVALID_ARG and the results are then unspecified).
 *   workspace   device, 256-byte aligned, at least chimera_workspace_bytes(...) bytes; contents are scratch.  Two
 *               calls that may overlap on the device need distinct workspaces.
 *   out_ids     device, [n_queries, k] int32: best first; -1 where fewer than k documents survive.
 *   out_scores  device, [n_queries, k] float32: -inf beside every -1.
 * Results do not depend on n_queries (a batch equals the same queries run one by one).
 * Errors: INVALID_ARG, UNSUPPORTED, WORKSPACE_TOO_SMALL (nothing enqueued), CUDA_ERROR (launch failure). */
int chimera_search(const chimera_index *index, const float *queries, int32_t n_queries, int32_t q_len,
                   int32_t nprobe, int32_t n_prune, int32_t k, int64_t max_candidates, void *workspace,
                   size_t workspace_bytes, void *stream, int32_t *out_ids, float *out_scores);

/* The same search with HOST query and result buffers: copies the queries to the device (into the workspace), runs
 * chimera_search, copies ids and scores back and synchronises the stream before returning.  Pinned host memory makes
 * the copies asynchronous to each other but is not required.  The workspace must be
 * chimera_workspace_bytes(...) bytes as for chimera_search (the staging areas are included in that figure). */
int chimera_search_host(const chimera_index *index, const float *queries_host, int32_t n_queries, int32_t q_len,
                        int32_t nprobe, int32_t n_prune, int32_t k, int64_t max_candidates, void *workspace,
                        size_t workspace_bytes, void *stream, int32_t *out_ids_host, float *out_scores_host);

/* Intermediate results ("taps") of a search: caller-owned device buffers, each optional (NULL = skip).
 * They are copies of what the stages hand to each other, never a different computation. */
typedef struct {
    int32_t *score_table; /* [n_queries, K, q_len]  Q.24 fixed-point <q_i, c>, centroid-major                  */
    int32_t *probes;      /* [n_queries, q_len, nprobe] best first (score desc, id asc)                         */
    int32_t *cand;        /* [n_queries, max_candidates] ascending document ids; entries past n_cand undefined  */
    int32_t *n_cand;      /* [n_queries]                                                                        */
    int32_t *ci;          /* [n_queries, max_candidates] exact centroid-interaction score of cand[...] (Q.24
                             sum); the search itself needs it only for documents that can reach the top n_prune,
                             so asking for this tap runs the exact kernel over every candidate as well          */
    int32_t *pruned;      /* [n_queries, n_prune] ascending document ids, -1 padded                             */
    int32_t *n_pruned;    /* [n_queries]                                                                        */
    float *score4;        /* [n_queries, n_prune] stage-4 score of pruned[...], -inf beside -1                  */
    int32_t *n_contenders;/* [n_queries] documents whose CI upper bound reached the pruning threshold and got an
                             exact CI (q_len 32 or 64); n_cand for other q_len                                  */
} chimera_taps;

/* chimera_search that also copies the intermediates out (same kernels, same order).  taps: host pointer to a struct
 * of device pointers; max_candidates = 0 means n_docs here as well. */
int chimera_search_tapped(const chimera_index *index, const float *queries, int32_t n_queries, int32_t q_len,
                          int32_t nprobe, int32_t n_prune, int32_t k, int64_t max_candidates, void *workspace,
                          size_t workspace_bytes, void *stream, int32_t *out_ids, float *out_scores,
                          const chimera_taps *taps);

/* Run only stages first_stage..last_stage (1..5, first <= last).  Results of the stages before first_stage are read
 * from `inout`, which must then hold: first_stage 2, 3 or 4: score_table; first_stage 3: also cand and n_cand;
 * first_stage 4 or 5: pruned and n_pruned; first_stage 5: also score4.  Results of the stages that ran are written
 * to the other non-NULL members of `inout`.  out_ids / out_scores may be NULL unless last_stage is 5.  For tests that feed one stage with
 * another implementation's output. */
int chimera_run_stages(const chimera_index *index, int32_t first_stage, int32_t last_stage, const float *queries,
                       int32_t n_queries, int32_t q_len, int32_t nprobe, int32_t n_prune, int32_t k,
                       int64_t max_candidates, void *workspace, size_t workspace_bytes, void *stream,
                       const chimera_taps *inout, int32_t *out_ids, float *out_scores);

/* Build the token-level posting lists (per centroid: its tokens and their documents; Sec. 3.2 step 1 keeps posting
 * lists at token level) that chimera_search_partial needs.  Allocates 8 bytes per token plus 8 per centroid inside the
 * index (cudaMalloc), synchronises the stream.  Idempotent.  Workspace sizes grow afterwards (a score table of
 * n_queries x max_candidates x q_len int32), so query chimera_workspace_bytes again.
 * Errors: INVALID_ARG, UNSUPPORTED (more than 2^31 - 1 tokens), CUDA_ERROR (nothing stays allocated). */
int chimera_index_enable_partial(chimera_index *index, void *stream);

/* The search with the paper's own candidate refinement in place of stage 3 (Sec. 3.2 step 2, Algorithm 2; aggregation
 * as in Algorithm 4): only the tokens retrieved in candidate generation are scored.  For query token i every token t of
 * its nprobe probed posting lists raises score[doc(t), i] (initially 0) to
 *     dist(i, t) = S[cid_t, i] + llrint(delta*4*T + kappa*4*SQ_i)          (Q.24 fixed point)
 * with T = sum_x Xq_i[x] u_t[x], SQ_i = sum_x Xq_i[x], Xq = rint(q * 2^22), delta = (res_hi - res_lo) / 2^nbits and
 * kappa = res_lo + delta / 2 in float, products and sum in double; F'(d) = sum_i score[d, i]; the n_prune candidates
 * with the largest F' (ties: smaller id) go on to stages 4 and 5 unchanged.  It touches sum_i |L_i| tokens instead of
 * every token of every candidate, and prunes by a different (cheaper, coarser) score than chimera_search, so results
 * differ from chimera_search; they are exactly reproducible.
 * Arguments as chimera_search_tapped (taps may be NULL); taps->ci receives F' of every candidate, taps->n_contenders
 * the candidate counts.  Requires chimera_index_enable_partial. */
int chimera_search_partial(const chimera_index *index, const float *queries, int32_t n_queries, int32_t q_len,
                           int32_t nprobe, int32_t n_prune, int32_t k, int64_t max_candidates, void *workspace,
                           size_t workspace_bytes, void *stream, int32_t *out_ids, float *out_scores,
                           const chimera_taps *taps);

/* Attach RaBitQ 1-bit codes of the corpus tokens (Sec. 2.2: unit-norm token o, o_p = P o, code bit x = (o_p[x] > 0),
 * nearest codeword o_p-bar = sign(o_p) / sqrt(dim)) so that chimera_search_rabitq can run the paper's own GPU pipeline.
 *   rotation  device, [dim, dim] float32 row-major orthonormal matrix P.  Copied (transposed).
 *   bits      device, [T, dim/8] uint8, document-major: bit t of byte g is dimension 8g+t.  REFERENCED, not copied.
 *   inv_dot   device, [T] float32, 1 / <o_p, o_p-bar> = sqrt(dim) / sum_x |o_p[x]|.  REFERENCED, not copied.
 * Also builds the token-level posting lists (as chimera_index_enable_partial).  Synchronises the stream.
 * Errors: INVALID_ARG, CUDA_ERROR. */
int chimera_index_attach_rabitq(chimera_index *index, const float *rotation, const uint8_t *bits,
                                const float *inv_dot, void *stream);

/* The paper's GPU-resident pipeline on its own codec (Algorithm 1 without the CPU half): stage 1 and 2 as in
 * chimera_search (centroid probes, candidate set); queries rotated (q_p = P q, one fp32 fma chain per output);
 * candidate refinement by partial 1-bit scores (Algorithm 2: score[doc, i] starts at 0 and is raised by every
 * retrieved token's estimate; F' = sum over i in increasing i, fp32) keeping k_refine documents; document scoring =
 * the complete 1-bit Chamfer score sum_i max_t est(i, t) of the survivors; top-k.  The estimate (Sec. 2.2) is
 *     est(i, t) = <q_p, o_p-bar> / <o_p, o_p-bar> = inv_dot_t * (c * (float)(2 T - SQ_i)),   c = 1 / (sqrt(dim) 2^22),
 * T = sum_x Xq_i[x] bit_t[x], SQ_i = sum_x Xq_i[x], Xq = rint(q_p * 2^22): reproducible bit for bit.
 * Arguments as chimera_search_tapped with k_refine in the place of n_prune (taps may be NULL); taps->ci receives the
 * bit patterns of the float F' of every candidate, taps->score4 the complete 1-bit scores.  q_len <= 64.
 * Requires chimera_index_attach_rabitq; query chimera_workspace_bytes after attaching. */
int chimera_search_rabitq(const chimera_index *index, const float *queries, int32_t n_queries, int32_t q_len,
                          int32_t nprobe, int32_t k_refine, int32_t k, int64_t max_candidates, void *workspace,
                          size_t workspace_bytes, void *stream, int32_t *out_ids, float *out_scores,
                          const chimera_taps *taps);

/* ---- Proximity graph over the centroids (Sec. 3.1; Algorithm 1, line searchCAGRA; Sec. 2.3) -----------------------
 * The paper finds each query token's n_probe centroids by searching a proximity graph built over the IVF centroids
 * instead of scoring all of them.  Here:
 *   graph   node c is linked to the `degree` other centroids with the largest fixed-point inner product S_fx(c, c')
 *           (ties: smaller id), best first;
 *   search  per query token a best-first search with a bounded list: the entry points floor(j K / n_entries),
 *           j < n_entries, are visited (scored, marked, offered to the list); then, repeatedly, the first list member not
 *           yet expanded is expanded -- each of its neighbours that was never visited is visited -- until every member
 *           is expanded or max_expansions expansions are done; the list keeps the best `beam` visited centroids by
 *           (S_fx descending, id ascending); the probes are its first nprobe members.
 * Scores are the exact S_fx of stage 1, so probes, their scores and the set of visited centroids are reproducible bit
 * for bit; whether the probes are the exhaustive top nprobe depends on the data and on (degree, n_entries, beam).
 *
 * chimera_index_build_graph: builds the graph inside the index (cudaMalloc of K * degree * 4 + K * dim * 4 bytes, plus
 *   about 0.7 GB of temporary memory freed before returning); synchronises the stream.  centroids: device, the same
 *   [K, dim] float32 array the index was built from.  1 <= degree <= min(63, K - 1).  Query chimera_workspace_bytes
 *   again afterwards.  Errors: INVALID_ARG, CUDA_ERROR (nothing stays allocated).
 * chimera_graph_probes: the search alone.  queries: device [n_queries, q_len, dim].  scratch: device,
 *   chimera_graph_scratch_bytes(...) bytes (one bit per centroid and query token: afterwards the visited sets, row
 *   t = query * q_len + token, bit c & 31 of word c / 32).  out_probes: device [n_queries, q_len, nprobe] int32 (-1 if
 *   fewer were visited); out_scores (optional): their S_fx; out_n_visited (optional): [n_queries, q_len] counts.
 *   nprobe <= beam <= 64, nprobe <= n_entries <= K, max_expansions >= 0.
 * chimera_search_rabitq_graph: chimera_search_rabitq with these probes in place of stage 1 and stage 2a -- the
 *   paper's GPU pipeline as Algorithm 1 states it (no score table is built; taps->score_table is not written). */
int chimera_index_build_graph(chimera_index *index, const float *centroids, int32_t degree, void *stream);
/* Degree of the index's graph (0 = none) to *out_degree (host); with out_graph non-NULL also a copy of the graph,
 * [K, degree] int32 row-major, to that device buffer (enqueued on `stream`). */
int chimera_index_copy_graph(const chimera_index *index, int32_t *out_graph, int32_t *out_degree, void *stream);
int chimera_graph_scratch_bytes(const chimera_index *index, int32_t n_queries, int32_t q_len, size_t *out);
int chimera_graph_probes(const chimera_index *index, const float *queries, int32_t n_queries, int32_t q_len,
                         int32_t nprobe, int32_t beam, int32_t n_entries, int32_t max_expansions, void *scratch,
                         size_t scratch_bytes, void *stream, int32_t *out_probes, int32_t *out_scores,
                         int32_t *out_n_visited);
int chimera_search_rabitq_graph(const chimera_index *index, const float *queries, int32_t n_queries, int32_t q_len,
                                int32_t nprobe, int32_t k_refine, int32_t k, int64_t max_candidates, int32_t beam,
                                int32_t n_entries, int32_t max_expansions, void *workspace, size_t workspace_bytes,
                                void *stream, int32_t *out_ids, float *out_scores, const chimera_taps *taps);

/* Device-side status of the last search that used this workspace: synchronises the stream, then writes CHIMERA_OK,
 * CHIMERA_CAPACITY_OVERFLOW (some query had more than max_candidates candidates; its results are computed on the
 * first max_candidates of them and are not the specified output), CHIMERA_INVALID_ARG (a query element outside
 * [-1, 1]), CHIMERA_TIMEOUT or (debug build) CHIMERA_DEBUG_CHECK_FAILED to *status (host pointer). */
int chimera_workspace_status(const void *workspace, void *stream, int32_t *status);

/* How a search with these parameters finds its probes (Sec. 3.2 step 1, the top-n_probe centroids of each query
 * token).  Writes to *sample_stride (host pointer) 0 when stage 2a is a scan of the finished score table, or s > 1
 * when stages 1 and 2a run together in calls that cover both: every s-th tile of 128 centroids is scored first, a
 * lower bound on each query token's nprobe-th best score is taken from that sample, and the score-table kernel queues
 * every score at or above the bound while it writes the rest of the table, so the table is not read again (a query
 * whose queue overflows is redone by the scan; the result is the same exact top n_probe either way).  The joint form
 * needs nprobe <= 32, q_len a multiple of 4 and at least 8 sample tiles. */
int chimera_probe_plan(const chimera_index *index, int32_t n_queries, int32_t q_len, int32_t nprobe,
                       int32_t *sample_stride);
/* The same rule as plain arithmetic on the sizes (no index, no device): the sampling stride for n_centroids centroids,
 * queries of q_len tokens and nprobe probes per token, or 0 for the table scan. */
int32_t chimera_probe_sample_stride(int64_t n_centroids, int32_t q_len, int32_t nprobe);

/* Debug build (the paper has no counterpart).  libchimera_debug.so is the same source compiled with -DCHIMERA_DEBUG:
 * every kernel checks each centroid id, document id, token position and candidate rank before it gathers through it
 * (an index out of range is not dereferenced; chimera_workspace_status then reports CHIMERA_DEBUG_CHECK_FAILED), and
 * every workspace region is followed by a 256-byte guard pattern, so chimera_workspace_bytes is larger.  It stands in
 * for a memory checker where none can be run; it is several times slower and serves one search at a time per process.
 * chimera_is_debug_build: 1 in that library, 0 otherwise.
 * chimera_workspace_check: after a search with the same parameters on `workspace`, verifies the guard patterns
 * (synchronises the stream) and writes the index of the first damaged region to *damaged_region (host pointer), -1 if
 * all are intact.  Returns CHIMERA_UNSUPPORTED in a release build. */
int chimera_is_debug_build(void);
int chimera_workspace_check(const chimera_index *index, int32_t n_queries, int32_t q_len, int32_t nprobe,
                            int32_t n_prune, int32_t k, int64_t max_candidates, const void *workspace, void *stream,
                            int32_t *damaged_region);

/* Test hook for the give-up path of the bounded device-side waits (the paper has no counterpart).  The two tensor-core
 * kernels (stage 1, stage 4) wait on mbarriers for their TMA loads and MMAs; each wait gives up after a limit (default
 * 100,000,000 SM cycles, about 50 ms), sets the TIMEOUT status bit, and the block frees its tensor memory and returns.
 * skip_loads != 0 makes every later search of this process issue NO TMA load in those kernels, so their waits run
 * into the limit with nothing in flight; wait_cycles > 0 sets the limit (<= 0 restores the default).  The searches
 * still return CHIMERA_OK (they only enqueue); chimera_workspace_status then reports CHIMERA_TIMEOUT and the results
 * are undefined.  Call it again with (0, 0) to restore normal operation; the device context stays usable.
 * Process-wide; not for production use. */
int chimera_test_wait_fault(int32_t skip_loads, int64_t wait_cycles);

/* Sizes held by an index (host pointers, each optional). */
int chimera_index_info(const chimera_index *index, chimera_index_desc *desc, int64_t *posting_entries,
                       int32_t *max_doclen);

/* Per-stage device timing.  After chimera_profile_enable(1) every search records CUDA events around its stages on
 * the search's stream; chimera_profile_read synchronises those events and returns, per stage slot, the summed
 * milliseconds and the number of kernels launched since the last read, then resets both.  Slots:
 * 0 score table, 1 probes, 2 candidate gather, 3 centroid-interaction bounds over every candidate (or the exact scan
 * when q_len is not 32/64), 4 selections (contenders, top n_prune), 5 residual scores, 6 top-k, 7 copies/clears,
 * 8 exact centroid interaction of the contenders.  ms and launches: host arrays of CHIMERA_PROFILE_SLOTS entries.  At most
 * CHIMERA_PROFILE_MAX_CALLS searches are kept between reads (later ones are not timed).  Not thread-safe. */
#define CHIMERA_PROFILE_SLOTS 9
#define CHIMERA_PROFILE_MAX_CALLS 256
int chimera_profile_enable(int32_t on);
int chimera_profile_read(float *ms, int64_t *launches);

/* Top-nprobe centroids per query token WITHOUT any device allocation and without a workspace (the paper has no
 * counterpart: this is a packaging variant of stage 2a for callers that cannot allocate).
 *
 * Who needs it: callers that may not call cudaMalloc (or any allocating routine) at query time -- serving loops that
 * fix all memory at start-up, or processes where another component owns the device memory pool.  The stage's scratch
 * (partial top-nprobe lists) lives in a 4 MiB array built into the library image; every GPU that loads the library
 * holds those 4 MiB until the process exits.
 *
 *   score_table  device, [n_queries, n_centroids, q_len] int32, centroid-major (stage 1's output layout).
 *   out_probes   device, [n_queries, q_len, nprobe] int32, best first (score descending, centroid id ascending):
 *                identical to the probes of chimera_search / chimera_run_stages for the same table.
 *   stream       cudaStream_t as void*; the two kernels are enqueued on it, the call does not synchronise.
 *
 * Limits: n_queries * lists * nprobe * q_len * 8 bytes must fit the 4 MiB array, where lists = min(512,
 * ceil(4 * SM count / n_queries), ceil(n_centroids / 256)); e.g. one query of 32 tokens with nprobe 4 against 65,536
 * centroids needs 256 KiB, a batch of 64 such queries 640 KiB.  Larger calls return CHIMERA_WORKSPACE_TOO_SMALL and
 * enqueue nothing (use chimera_search with a workspace).  Other argument limits are those of chimera_search.
 *
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress, with that device current)
 * and caches it; under lazy module loading that first call may also make the CUDA runtime load the library's kernels
 * and place the array, so make it once at start-up, before any stream capture and before memory is frozen.  After
 * that a call allocates and frees nothing.  A cached address does not survive cudaDeviceReset.  All calls share the one array per device and it keeps the previous call's contents: the kernels overwrite
 * every entry they later read, so no clearing is needed, but two calls whose kernels may overlap on the same device
 * (different streams, or concurrent host threads) race on it -- serialise them. */
int chimera_probes_static(const int32_t *score_table, int64_t n_centroids, int32_t n_queries, int32_t q_len,
                          int32_t nprobe, void *stream, int32_t *out_probes);

/* ---- Document-sharded search over several GPUs (the scaling sketch of Sec. 3.3) -----------------------------------
 * The documents are partitioned into `world` contiguous id ranges in rank order; rank r builds an index of its own
 * documents (local ids 0 .. n_local-1 = global ids doc_base .. doc_base+n_local-1) and of ALL centroids.  Queries are
 * the same on every rank.  Only ids and scores cross GPUs (the caller moves them, e.g. with an all-gather):
 *   1. chimera_shard_local   stages 1-3 on the local shard; exports the local top n_prune (global ids ascending,
 *                            -1 padded) and their stage-3 scores (INT_MIN padded): int32 [n_queries, n_prune] each.
 *   2. all-gather both arrays over the ranks, in rank order: [world, n_queries, n_prune].
 *   3. chimera_shard_finish  the global top n_prune of the gathered lists by (score descending, global id ascending)
 *                            -- the set a single index of all documents prunes to, because stage-3 scores are
 *                            integers that do not depend on the shard --, of which this rank keeps its own documents,
 *                            scores them (stage 4) and emits its local top-k with GLOBAL ids: [n_queries, k].
 *   4. all-gather ids and scores: [world, n_queries, k].
 *   5. chimera_shard_merge_topk  the best k of the union, (score descending, id ascending): equal to the single-index
 *                            result (a document's stage-4 score does not depend on the shard it is scored in).
 * mode: 0 = stage 3 by centroid interaction, 1 = by partial scores (needs chimera_index_enable_partial), 2 = the
 * RaBitQ pipeline (needs chimera_index_attach_rabitq).  Steps 1 and 3 must use the same workspace and the same
 * parameters, with no other call on that workspace in between (step 3 continues from what step 1 left there, and
 * keeps the status bits step 1 set: one chimera_workspace_status after step 3 covers both).  In a multi-process run
 * exchange the status with the other ranks before acting on it: a rank that stops between the collectives leaves the
 * others waiting in theirs.  All pointers device; everything is enqueued on `stream`.
 * world * k <= 16384 in step 5 (CHIMERA_UNSUPPORTED otherwise). */
int chimera_shard_local(const chimera_index *index, const float *queries, int32_t n_queries, int32_t q_len,
                        int32_t nprobe, int32_t n_prune, int32_t k, int64_t max_candidates, int32_t mode,
                        int64_t doc_base, void *workspace, size_t workspace_bytes, void *stream, int32_t *out_ids,
                        int32_t *out_scores3);
int chimera_shard_finish(const chimera_index *index, const float *queries, int32_t n_queries, int32_t q_len,
                         int32_t nprobe, int32_t n_prune, int32_t k, int64_t max_candidates, int32_t mode,
                         int64_t doc_base, int32_t world, const int32_t *all_ids, const int32_t *all_scores3,
                         void *workspace, size_t workspace_bytes, void *stream, int32_t *out_ids, float *out_scores);
int chimera_shard_merge_topk(const int32_t *all_ids, const float *all_scores, int32_t world, int32_t n_queries,
                             int32_t k, void *stream, int32_t *out_ids, float *out_scores);

#ifdef __cplusplus
}
#endif
#endif /* CHIMERA_H */
