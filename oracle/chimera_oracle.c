/*
 * CPU oracle for late-interaction (MaxSim / Chamfer) retrieval over centroid + residual codes.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, single-threaded, obviously-correct statement of
 * what the retrieval pipeline computes.  It shares no code, header, table or constant with the CUDA
 * library and is never linked into or called from it.  Only the test-suite, the smoke check and the
 * benchmark's CPU-baseline leg may call it.
 *
 * Every function takes host pointers; nothing is blocked, fused, vectorised or reordered beyond the
 * definition it states.  Floating-point sums are accumulated in double.
 *
 * Stages (each function cites the passage of the paper it follows):
 *   O-1 oracle_score_table   fixed-point <q_i, c_c>                        (Def. 1, inner product)
 *   O-2 oracle_probes        top-nprobe centroids per query token          (Sec. 3.2 step 1)
 *   O-3 oracle_candidates    S = { V : some v in V lies in a probed list } (Sec. 3.2 step 1, set S)
 *   O-4 oracle_ci / oracle_prune   centroid-interaction max-then-sum, keep top n'   (Sec. 4.2 rule)
 *   O-5 oracle_score_docs    Chamfer similarity on decoded tokens          (Def. 1)
 *   O-6 oracle_topk          top-k by score                                (Def. 2, Eq. 1)
 *   O-7 oracle_chamfer       Def. 1 on raw vectors;  oracle_recall  Def. 3
 *   O-8 oracle_partial_scores  candidate refinement with partial scores F'(Q,V)  (Sec. 3.2 step 2, Algorithm 2)
 *   O-9 oracle_rotate, oracle_rabitq_score_docs, oracle_rabitq_partial   the same two steps on RaBitQ 1-bit codes
 *       (Sec. 2.2: rotation, 1-bit code, estimator <q_p, o_p-bar> / <o_p, o_p-bar>, code form of <q_p, o_p-bar>)
 *   O-10 oracle_knn_graph, oracle_graph_probes   proximity graph over the centroids and the search that replaces the
 *       exhaustive centroid scan (Sec. 2.3 "Proximity graph", Sec. 3.1, Algorithm 1 line searchCAGRA)
 *
 * Pins: every function above is pinned by tests that do not call it to produce their expectation
 * (closed forms, library routines on special cases, set identities, hand-worked values).  Unpinned:
 * absolute recall values on the synthetic corpora (nothing in the paper fixes them).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define Q22 4194304.0 /* 2^22 */

/* ---------------------------------------------------------------- O-1 ------------------------------------------ */
/* Def. 1 uses the inner product <q, v>.  For the centroid table it is evaluated in exact integer arithmetic so that
 * every later discrete decision (probe lists, candidate sets, pruned ids) is independent of summation order:
 *   Xq = rint(q * 2^22), Xc = rint(c * 2^22)  (round-half-even),  T = sum_d Xq[d]*Xc[d]  (int64, exact),
 *   S_fx = floor((T + 2^19) / 2^20)           (a Q.24 fixed-point value; the real score is S_fx * 2^-24).
 * Output layout is centroid-major: S[c*nq + i]. */
void oracle_score_table(const float *q, int32_t nq, const float *cent, int64_t K, int32_t D, int32_t *S)
{
    int64_t *xq = (int64_t *)malloc(sizeof(int64_t) * (size_t)nq * D);
    int64_t *xc = (int64_t *)malloc(sizeof(int64_t) * (size_t)D);
    for (int64_t e = 0; e < (int64_t)nq * D; ++e) xq[e] = (int64_t)rint((double)q[e] * Q22);
    for (int64_t c = 0; c < K; ++c) {
        for (int d = 0; d < D; ++d) xc[d] = (int64_t)rint((double)cent[c * D + d] * Q22);
        for (int i = 0; i < nq; ++i) {
            int64_t t = 0;
            for (int d = 0; d < D; ++d) t += xq[(int64_t)i * D + d] * xc[d];
            int64_t u = t + (1LL << 19);
            int64_t f = u / (1LL << 20); /* floor division */
            if ((u % (1LL << 20)) < 0) f -= 1;
            S[c * nq + i] = (int32_t)f;
        }
    }
    free(xq);
    free(xc);
}

/* ---------------------------------------------------------------- O-2 ------------------------------------------ */
/* Sec. 3.2 step 1: for each query token the nprobe best-ranked centroids.  All vectors are unit-norm, so ranking by
 * distance ascending is ranking by inner product descending.  Ties: smaller centroid id first.
 * probes[i*nprobe + p] = p-th best centroid of query token i. */
typedef struct { int32_t s; int32_t id; } si_pair;
static int cmp_si_desc(const void *a, const void *b)
{
    const si_pair *x = (const si_pair *)a, *y = (const si_pair *)b;
    if (x->s != y->s) return (x->s > y->s) ? -1 : 1;
    if (x->id != y->id) return (x->id < y->id) ? -1 : 1;
    return 0;
}
void oracle_probes(const int32_t *S, int32_t nq, int64_t K, int32_t nprobe, int32_t *probes)
{
    si_pair *v = (si_pair *)malloc(sizeof(si_pair) * (size_t)K);
    for (int i = 0; i < nq; ++i) {
        for (int64_t c = 0; c < K; ++c) { v[c].s = S[c * nq + i]; v[c].id = (int32_t)c; }
        qsort(v, (size_t)K, sizeof(si_pair), cmp_si_desc);
        for (int p = 0; p < nprobe; ++p) probes[i * nprobe + p] = v[p].id;
    }
    free(v);
}

/* ---------------------------------------------------------------- O-3 ------------------------------------------ */
/* Sec. 3.2 step 1: L_q is the union of the probed posting lists (a posting list holds the tokens assigned to one
 * centroid), and the candidate set S holds every document with at least one token in the union over all query
 * tokens.  Written as a plain scan of every token of every document (no inverted file).  Returns |S|; cand gets the
 * ids in ascending order (cand must have room for N ids). */
int64_t oracle_candidates(const int32_t *probes, int32_t n_probes_total, int64_t K, const int32_t *cids,
                          const int32_t *doclens, int64_t N, int32_t *cand)
{
    uint8_t *probed = (uint8_t *)calloc((size_t)K, 1);
    for (int e = 0; e < n_probes_total; ++e) probed[probes[e]] = 1;
    int64_t t = 0, n = 0;
    for (int64_t d = 0; d < N; ++d) {
        int hit = 0;
        for (int j = 0; j < doclens[d]; ++j, ++t)
            if (probed[cids[t]]) hit = 1;
        if (hit) cand[n++] = (int32_t)d;
    }
    free(probed);
    return n;
}

/* ---------------------------------------------------------------- O-4 ------------------------------------------ */
/* Chamfer aggregation rule (Sec. 4.2: per query token the maximum over the document's tokens, then the sum over query
 * tokens) applied to the centroid scores: CI(d) = sum_i max_{t in d} S[cid_t, i].  Integer arithmetic, order-free.
 * doc_off[d] = index of the first token of document d (doc_off has N+1 entries). */
void oracle_ci(const int32_t *S, int32_t nq, const int32_t *cand, int64_t n_cand, const int32_t *cids,
               const int64_t *doc_off, int32_t *ci)
{
    for (int64_t j = 0; j < n_cand; ++j) {
        int64_t d = cand[j];
        int64_t sum = 0;
        for (int i = 0; i < nq; ++i) {
            int32_t m = INT32_MIN;
            for (int64_t t = doc_off[d]; t < doc_off[d + 1]; ++t) {
                int32_t s = S[(int64_t)cids[t] * nq + i];
                if (s > m) m = s;
            }
            sum += m;
        }
        ci[j] = (int32_t)sum;
    }
}

/* Keep the n' candidates with the largest CI (ties: smaller document id first); all of them if fewer exist.
 * pruned gets the kept ids in ascending id order.  Returns how many were kept. */
static int cmp_i32_asc(const void *a, const void *b)
{
    int32_t x = *(const int32_t *)a, y = *(const int32_t *)b;
    return (x > y) - (x < y);
}
int64_t oracle_prune(const int32_t *cand, const int32_t *ci, int64_t n_cand, int64_t n_prune, int32_t *pruned)
{
    si_pair *v = (si_pair *)malloc(sizeof(si_pair) * (size_t)(n_cand > 0 ? n_cand : 1));
    for (int64_t j = 0; j < n_cand; ++j) { v[j].s = ci[j]; v[j].id = cand[j]; }
    qsort(v, (size_t)n_cand, sizeof(si_pair), cmp_si_desc);
    int64_t keep = n_cand < n_prune ? n_cand : n_prune;
    for (int64_t j = 0; j < keep; ++j) pruned[j] = v[j].id;
    qsort(pruned, (size_t)keep, sizeof(int32_t), cmp_i32_asc);
    free(v);
    return keep;
}

/* ---------------------------------------------------------------- O-8 ------------------------------------------ */
/* Candidate refinement (Sec. 3.2 step 2, Algorithm 2): only the tokens retrieved in candidate generation contribute.
 * For each query token i, L_i = the tokens assigned to one of its nprobe probed centroids; every document score
 * starts at 0 per query token, each retrieved token raises doc.score[i] to max(score, dist(i, token)), and the
 * partial score is F'(d) = sum_i doc.score[i]  (a query token that retrieved nothing of d contributes 0).
 *
 * dist(i, t) is the low-bit score <q_i, c_cid + r^(code_t)> in Q.24 fixed point, so that the refinement is exactly
 * reproducible:  dist = S[cid_t, i] + llrint(delta*4*T + kappa*4*SQ_i),  T = sum_x Xq_i[x] u_t[x],
 * SQ_i = sum_x Xq_i[x],  Xq = rint(q * 2^22),  delta = (hi - lo) / 2^b and kappa = lo + delta/2 evaluated in float,
 * the two products and their sum in double (each exact or correctly rounded, no fused operations).
 *
 * cand: ascending candidate ids (O-3); fprime[j] = F' of cand[j].  Written as Algorithm 2's loops over a dense
 * n_cand x nq score table. */
void oracle_partial_scores(const int32_t *S, const float *q, int32_t nq, int32_t D, int32_t nbits, float lo, float hi,
                           const int32_t *probes, int32_t nprobe, const int32_t *cids, const uint8_t *codes,
                           const int32_t *doclens, int64_t N, const int32_t *cand, int64_t n_cand, int32_t *fprime)
{
    const int per_byte = 8 / nbits, mask = (1 << nbits) - 1;
    const int64_t cb = (int64_t)D * nbits / 8;
    const float delta = (hi - lo) / (float)(1 << nbits);
    const float kappa = lo + 0.5f * delta;
    int64_t *slot = (int64_t *)malloc(sizeof(int64_t) * (size_t)N);   /* document -> row of the score table, or -1 */
    for (int64_t d = 0; d < N; ++d) slot[d] = -1;
    for (int64_t j = 0; j < n_cand; ++j) slot[cand[j]] = j;
    int32_t *score = (int32_t *)calloc((size_t)(n_cand > 0 ? n_cand : 1) * nq, sizeof(int32_t));   /* init 0 */
    int64_t *xq = (int64_t *)malloc(sizeof(int64_t) * (size_t)D);
    int64_t K = 0;                                        /* centroid ids are < K = 1 + the largest id in use */
    for (int64_t d = 0, t = 0; d < N; ++d)
        for (int j = 0; j < doclens[d]; ++j, ++t)
            if (cids[t] >= K) K = (int64_t)cids[t] + 1;
    for (int e = 0; e < nq * nprobe; ++e)
        if (probes[e] >= K) K = (int64_t)probes[e] + 1;
    uint8_t *probed = (uint8_t *)malloc((size_t)K);       /* is this centroid probed by query token i? */
    for (int i = 0; i < nq; ++i) {
        int64_t sq = 0;
        for (int x = 0; x < D; ++x) { xq[x] = (int64_t)rint((double)q[(int64_t)i * D + x] * Q22); sq += xq[x]; }
        memset(probed, 0, (size_t)K);
        for (int p = 0; p < nprobe; ++p) probed[probes[i * nprobe + p]] = 1;
        int64_t t = 0;
        for (int64_t d = 0; d < N; ++d) {
            for (int j = 0; j < doclens[d]; ++j, ++t) {
                if (!probed[cids[t]]) continue;           /* token t is in L_i iff its centroid is probed by i */
                int64_t T = 0;
                for (int x = 0; x < D; ++x) {
                    int u = (codes[t * cb + x / per_byte] >> ((x % per_byte) * nbits)) & mask;
                    T += xq[x] * u;
                }
                double r = (double)delta * 4.0 * (double)T + (double)kappa * 4.0 * (double)sq;
                int64_t dist = (int64_t)S[(int64_t)cids[t] * nq + i] + (int64_t)llrint(r);
                int32_t *cell = &score[slot[d] * nq + i];
                if (dist > *cell) *cell = (int32_t)dist;
            }
        }
    }
    for (int64_t j = 0; j < n_cand; ++j) {
        int64_t sum = 0;
        for (int i = 0; i < nq; ++i) sum += score[j * nq + i];
        fprime[j] = (int32_t)sum;
    }
    free(slot);
    free(score);
    free(xq);
    free(probed);
}

/* ---------------------------------------------------------------- O-9 ------------------------------------------ */
/* Sec. 2.2: vectors are rotated by a random orthonormal matrix P before quantisation; inner products are preserved.
 * q_p = P q, evaluated as one fp32 fused-multiply-add chain per output in increasing x, so that every implementation
 * that follows this order gets the same bits.  P is [D][D] row-major, q is [n][D]. */
void oracle_rotate(const float *P, const float *q, int64_t n, int32_t D, float *out)
{
    for (int64_t i = 0; i < n; ++i)
        for (int r = 0; r < D; ++r) {
            float acc = 0.0f;
            for (int x = 0; x < D; ++x) acc = fmaf(P[(int64_t)r * D + x], q[i * D + x], acc);
            out[i * D + r] = acc;
        }
}

/* Estimator of Sec. 2.2 with B = 1:  <q, o> ~ <q_p, o_p-bar> / <o_p, o_p-bar>, and by the code equation
 * <q_p, o_p-bar> = (1 / |y-bar|) (<q_p, o_b> - 1/2 sum q_p), |y-bar| = sqrt(D) / 2, o_b the 0/1 code.
 * With Xq = rint(q_p * 2^22):  T = sum_x Xq[x] o_b[x],  A = 2 T - sum_x Xq[x]  (integers),
 * est = inv_dot * (c * (float)A),  c = (float)(1 / (sqrt(D) * 2^22)),  two fp32 multiplications in that order.
 * bits: bit t of byte g holds dimension 8g+t. */
static float rabitq_est(const int64_t *xq, int64_t sq, const uint8_t *bits, int64_t t, int32_t D, float inv_dot)
{
    const int64_t cb = D / 8;
    int64_t T = 0;
    for (int x = 0; x < D; ++x)
        if ((bits[t * cb + x / 8] >> (x % 8)) & 1) T += xq[x];
    const float c = (float)(1.0 / (sqrt((double)D) * Q22));
    const float a = (float)(2 * T - sq);
    const float ca = c * a;
    return inv_dot * ca;
}

/* Document scoring on the 1-bit codes (Sec. 3.2 step 3, GPU half): the complete 1-bit Chamfer score
 * sum_i max_{t in d} est(i, t), query tokens summed in increasing i in fp32.  qp: rotated query [nq][D]. */
void oracle_rabitq_score_docs(const float *qp, int32_t nq, int32_t D, const uint8_t *bits, const float *inv_dot,
                              const int64_t *doc_off, const int32_t *docs, int64_t n_listed, float *scores)
{
    int64_t *xq = (int64_t *)malloc(sizeof(int64_t) * (size_t)nq * D);
    int64_t *sq = (int64_t *)calloc((size_t)nq, sizeof(int64_t));
    for (int i = 0; i < nq; ++i)
        for (int x = 0; x < D; ++x) {
            xq[(int64_t)i * D + x] = (int64_t)rint((double)qp[(int64_t)i * D + x] * Q22);
            sq[i] += xq[(int64_t)i * D + x];
        }
    for (int64_t j = 0; j < n_listed; ++j) {
        const int64_t d = docs[j];
        if (d < 0) { scores[j] = -INFINITY; continue; }
        float total = 0.0f;
        for (int i = 0; i < nq; ++i) {
            float best = -INFINITY;
            for (int64_t t = doc_off[d]; t < doc_off[d + 1]; ++t) {
                float e = rabitq_est(xq + (int64_t)i * D, sq[i], bits, t, D, inv_dot[t]);
                if (e > best) best = e;
            }
            total = total + best;
        }
        scores[j] = total;
    }
    free(xq);
    free(sq);
}

/* Candidate refinement (Algorithm 2) with the 1-bit estimate as the distance: doc.score[i] starts at 0 and is raised
 * by every retrieved token; F' = sum_i doc.score[i] in increasing i in fp32.  fprime[j] belongs to cand[j]. */
void oracle_rabitq_partial(const float *qp, int32_t nq, int32_t D, const uint8_t *bits, const float *inv_dot,
                           const int32_t *probes, int32_t nprobe, const int32_t *cids, const int32_t *doclens,
                           int64_t N, int64_t K, const int32_t *cand, int64_t n_cand, float *fprime)
{
    int64_t *slot = (int64_t *)malloc(sizeof(int64_t) * (size_t)N);
    for (int64_t d = 0; d < N; ++d) slot[d] = -1;
    for (int64_t j = 0; j < n_cand; ++j) slot[cand[j]] = j;
    float *score = (float *)calloc((size_t)(n_cand > 0 ? n_cand : 1) * nq, sizeof(float));   /* init 0 */
    int64_t *xq = (int64_t *)malloc(sizeof(int64_t) * (size_t)D);
    uint8_t *probed = (uint8_t *)malloc((size_t)K);
    for (int i = 0; i < nq; ++i) {
        int64_t sq = 0;
        for (int x = 0; x < D; ++x) { xq[x] = (int64_t)rint((double)qp[(int64_t)i * D + x] * Q22); sq += xq[x]; }
        memset(probed, 0, (size_t)K);
        for (int p = 0; p < nprobe; ++p) probed[probes[i * nprobe + p]] = 1;
        int64_t t = 0;
        for (int64_t d = 0; d < N; ++d)
            for (int j = 0; j < doclens[d]; ++j, ++t) {
                if (!probed[cids[t]]) continue;
                float e = rabitq_est(xq, sq, bits, t, D, inv_dot[t]);
                float *cell = &score[slot[d] * nq + i];
                if (e > *cell) *cell = e;
            }
    }
    for (int64_t j = 0; j < n_cand; ++j) {
        float sum = 0.0f;
        for (int i = 0; i < nq; ++i) sum = sum + score[j * nq + i];
        fprime[j] = sum;
    }
    free(slot);
    free(score);
    free(xq);
    free(probed);
}

/* ---------------------------------------------------------------- O-10 ----------------------------------------- */
/* Exact fixed-point score of one query token against one centroid (the O-1 formula for a single pair). */
static int32_t fx_score(const int64_t *xq, const float *c, int32_t D)
{
    int64_t t = 0;
    for (int d = 0; d < D; ++d) t += xq[d] * (int64_t)rint((double)c[d] * Q22);
    int64_t u = t + (1LL << 19);
    int64_t f = u / (1LL << 20);
    if ((u % (1LL << 20)) < 0) f -= 1;
    return (int32_t)f;
}

/* Sec. 2.3 / Sec. 3.1: a proximity graph over the IVF centroids, "constructed by linking each node to a limited number
 * of nearest neighbors".  Here: node c is linked to the R other centroids with the largest fixed-point inner product
 * S_fx(c, c') (all centroids are unit vectors, so this is nearest first), ties towards the smaller id, listed best
 * first.  No pruning or diversification.  graph[c*R + r] = r-th neighbour of c.  Requires 1 <= R <= K - 1. */
void oracle_knn_graph(const float *cent, int64_t K, int32_t D, int32_t R, int32_t *graph)
{
    si_pair *v = (si_pair *)malloc(sizeof(si_pair) * (size_t)K);
    int64_t *xq = (int64_t *)malloc(sizeof(int64_t) * (size_t)D);
    for (int64_t c = 0; c < K; ++c) {
        for (int d = 0; d < D; ++d) xq[d] = (int64_t)rint((double)cent[c * D + d] * Q22);
        int64_t n = 0;
        for (int64_t o = 0; o < K; ++o) {
            if (o == c) continue;
            v[n].s = fx_score(xq, cent + o * D, D);
            v[n].id = (int32_t)o;
            ++n;
        }
        qsort(v, (size_t)n, sizeof(si_pair), cmp_si_desc);
        for (int r = 0; r < R; ++r) graph[c * R + r] = v[r].id;
    }
    free(v);
    free(xq);
}

/* Sec. 2.3: "the search starts from one or a few entry points and iteratively moves to neighboring nodes that are
 * closer to the query until convergence"; Algorithm 1 uses it to get each query token's n_probe centroids.  Stated
 * here as a best-first search with a bounded result list:
 *   - entry points: the n_entries centroids floor(j K / n_entries), j = 0 .. n_entries - 1 (the same for every query);
 *   - a list of at most `beam` visited centroids, ordered by (score descending, id ascending);
 *   - every entry point is visited (scored, marked, offered to the list);
 *   - repeat: take the first list member that has not been expanded, mark it expanded, and visit each of its graph
 *     neighbours that has not been visited before; stop when every list member is expanded, or after
 *     max_expansions expansions;
 *   - a visited centroid enters the list if the list is not full or it ranks before the last member, which is then
 *     dropped (a dropped centroid stays visited and is never scored again).
 * The score is the exact fixed-point S_fx(q, c), so the outcome does not depend on evaluation order.
 * Outputs: probes / scores = the first nprobe list members (requires nprobe <= beam and nprobe <= n_entries <= K);
 * visited[c] = 1 for every scored centroid.  Returns the number of visited centroids. */
int64_t oracle_graph_probes(const float *q, const float *cent, int64_t K, int32_t D, const int32_t *graph, int32_t R,
                            int32_t n_entries, int32_t beam, int64_t max_expansions, int32_t nprobe, int32_t *probes,
                            int32_t *scores, uint8_t *visited)
{
    int64_t *xq = (int64_t *)malloc(sizeof(int64_t) * (size_t)D);
    for (int d = 0; d < D; ++d) xq[d] = (int64_t)rint((double)q[d] * Q22);
    si_pair *list = (si_pair *)malloc(sizeof(si_pair) * (size_t)(beam + 1));
    uint8_t *expanded = (uint8_t *)malloc((size_t)(beam + 1));
    int32_t size = 0;
    int64_t n_visited = 0, expansions = 0;
    memset(visited, 0, (size_t)K);
    for (int64_t step = -n_entries;; ++step) {
        /* the centroids to visit in this step: one entry point, or the neighbours of the member to expand */
        int32_t one, count;
        const int32_t *todo;
        if (step < 0) {
            one = (int32_t)(((int64_t)(step + n_entries) * K) / n_entries);
            todo = &one;
            count = 1;
        } else {
            int32_t p = -1;
            for (int32_t m = 0; m < size; ++m)
                if (!expanded[m]) { p = m; break; }
            if (p < 0 || expansions == max_expansions) break;
            expanded[p] = 1;
            ++expansions;
            todo = graph + (int64_t)list[p].id * R;
            count = R;
        }
        for (int32_t r = 0; r < count; ++r) {
            const int32_t n = todo[r];
            if (visited[n]) continue;
            visited[n] = 1;
            ++n_visited;
            si_pair x;
            x.s = fx_score(xq, cent + (int64_t)n * D, D);
            x.id = n;
            int32_t pos = size;                           /* position of x in the ordered list */
            while (pos > 0 && cmp_si_desc(&x, &list[pos - 1]) < 0) --pos;
            if (pos >= beam) continue;                    /* ranks behind a full list */
            for (int32_t m = size; m > pos; --m) { list[m] = list[m - 1]; expanded[m] = expanded[m - 1]; }
            list[pos] = x;
            expanded[pos] = 0;
            if (size < beam) ++size;                      /* else the former last member fell off */
        }
    }
    for (int32_t r = 0; r < nprobe; ++r) {
        probes[r] = r < size ? list[r].id : -1;
        scores[r] = r < size ? list[r].s : INT32_MIN;
    }
    free(xq);
    free(list);
    free(expanded);
    return n_visited;
}

/* ---------------------------------------------------------------- O-5 ------------------------------------------ */
/* Decode one token: d^[x] = c[cid][x] + r^(u_x), r^(u) = lo + (u + 0.5) * delta, delta = (hi - lo) / 2^b, in fp32.
 * Packing: 2-bit codes put dimension 4g+t into bits [2t, 2t+1] of byte g; 1-bit codes put dimension 8g+t into bit t
 * of byte g.  No re-normalisation. */
static void decode_token(const float *cent, const int32_t *cids, const uint8_t *codes, int64_t t, int32_t D,
                         int32_t nbits, float lo, float hi, float *out)
{
    const int per_byte = 8 / nbits;
    const int mask = (1 << nbits) - 1;
    const float delta = (hi - lo) / (float)(1 << nbits);
    const int64_t cb = (int64_t)D * nbits / 8;
    const float *c = cent + (int64_t)cids[t] * D;
    for (int x = 0; x < D; ++x) {
        int u = (codes[t * cb + x / per_byte] >> ((x % per_byte) * nbits)) & mask;
        float r = lo + ((float)u + 0.5f) * delta;
        out[x] = c[x] + r;
    }
}

/* Def. 1: F(Q, V) = sum_{q in Q} max_{v in V} <q, v>, on raw fp32 vectors, accumulated in double. */
double oracle_chamfer(const float *q, int32_t nq, const float *v, int64_t nv, int32_t D)
{
    double total = 0.0;
    for (int i = 0; i < nq; ++i) {
        double best = -INFINITY;
        for (int64_t j = 0; j < nv; ++j) {
            double s = 0.0;
            for (int x = 0; x < D; ++x) s += (double)q[(int64_t)i * D + x] * (double)v[j * D + x];
            if (s > best) best = s;
        }
        total += best;
    }
    return total;
}

/* score(q, d) = F(Q, decoded tokens of d) for each listed document; ids < 0 (padding) score -inf. */
void oracle_score_docs(const float *q, int32_t nq, int32_t D, int32_t nbits, float lo, float hi, const float *cent,
                       const int32_t *cids, const uint8_t *codes, const int64_t *doc_off, const int32_t *docs,
                       int64_t n_docs_listed, float *scores)
{
    float *buf = NULL;
    int64_t cap = 0;
    for (int64_t j = 0; j < n_docs_listed; ++j) {
        int64_t d = docs[j];
        if (d < 0) { scores[j] = -INFINITY; continue; }
        int64_t len = doc_off[d + 1] - doc_off[d];
        if (len > cap) { cap = len; buf = (float *)realloc(buf, sizeof(float) * (size_t)cap * D); }
        for (int64_t t = 0; t < len; ++t)
            decode_token(cent, cids, codes, doc_off[d] + t, D, nbits, lo, hi, buf + t * D);
        scores[j] = (float)oracle_chamfer(q, nq, buf, len, D);
    }
    free(buf);
}

/* ---------------------------------------------------------------- O-6 ------------------------------------------ */
/* Def. 2 / Eq. 1: the k documents with the largest score, best first (ties: smaller id first).  Entries with id < 0
 * are ignored.  Missing results are padded with id -1 and score -inf. */
typedef struct { float s; int32_t id; } fi_pair;
static int cmp_fi_desc(const void *a, const void *b)
{
    const fi_pair *x = (const fi_pair *)a, *y = (const fi_pair *)b;
    if (x->s != y->s) return (x->s > y->s) ? -1 : 1;
    if (x->id != y->id) return (x->id < y->id) ? -1 : 1;
    return 0;
}
void oracle_topk(const int32_t *docs, const float *scores, int64_t n, int32_t k, int32_t *out_ids, float *out_scores)
{
    fi_pair *v = (fi_pair *)malloc(sizeof(fi_pair) * (size_t)(n > 0 ? n : 1));
    int64_t m = 0;
    for (int64_t j = 0; j < n; ++j)
        if (docs[j] >= 0) { v[m].s = scores[j]; v[m].id = docs[j]; ++m; }
    qsort(v, (size_t)m, sizeof(fi_pair), cmp_fi_desc);
    for (int32_t r = 0; r < k; ++r) {
        if (r < m) { out_ids[r] = v[r].id; out_scores[r] = v[r].s; }
        else { out_ids[r] = -1; out_scores[r] = -INFINITY; }
    }
    free(v);
}

/* ---------------------------------------------------------------- O-7 ------------------------------------------ */
/* Def. 3: Recall@k = |R intersect R'| / k, R = ground-truth top-k ids, R' = returned ids (negative ids ignored). */
double oracle_recall(const int32_t *truth, const int32_t *got, int32_t k)
{
    int hit = 0;
    for (int a = 0; a < k; ++a) {
        if (truth[a] < 0) continue;
        for (int b = 0; b < k; ++b)
            if (got[b] == truth[a]) { ++hit; break; }
    }
    return (double)hit / (double)k;
}
