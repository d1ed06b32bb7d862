"""Pins of the CPU oracle against what the paper and the mathematics fix.

No expectation in this file is produced by calling the oracle function under test: each comes from a closed form, a
hand-worked value under tests/golden/, a numpy library routine on a special case, a set identity, or a brute-force
enumeration written straight from the definition.
"""
import os

import numpy as np
import pytest

import oracle
from helpers import levels, random_corpus, unit_rows, unpack_codes

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden_rows(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return [ln.strip() for ln in f if ln.strip() and not ln.startswith("#")]


# ------------------------------------------------------------------ O-1 score table ------------------------------

def test_score_table_handworked_fixed_point():
    for row in _golden_rows("fixed_point_handworked.txt"):
        q, c, want = row.split()
        S = oracle.score_table(np.array([[float(q)]], np.float32), np.array([[float(c)]], np.float32))
        assert S.shape == (1, 1) and int(S[0, 0]) == int(want), row


def test_score_table_within_error_bound_of_exact_inner_product():
    # |S_fx - 2^24 <q,c>| <= 2 (|q|_1 + |c|_1) + D 2^-22 + 1/2  (rounding each input to 2^-22, then the result to 2^-24)
    rng = np.random.default_rng(1)
    for nq, K, D in [(5, 7, 128), (3, 11, 96), (32, 40, 128), (1, 1, 8)]:
        q, c = unit_rows(rng, nq, D), unit_rows(rng, K, D)
        S = oracle.score_table(q, c)
        assert S.shape == (K, nq) and S.dtype == np.int32      # centroid-major
        exact = (c.astype(np.float64) @ q.astype(np.float64).T) * 2.0 ** 24
        bound = 2.0 * (np.abs(c).sum(1)[:, None] + np.abs(q).sum(1)[None, :]) + 1.0
        assert np.all(np.abs(S - exact) <= bound)
        assert np.abs(S - exact).max() <= 47.0                 # 2*2*sqrt(128) + 1 for unit vectors


def test_score_table_unit_vector_with_itself_is_one():
    rng = np.random.default_rng(2)
    q = unit_rows(rng, 16, 128)
    S = oracle.score_table(q, q)
    assert np.all(np.abs(np.diag(S).astype(np.int64) - (1 << 24)) <= 50)
    assert np.array_equal(S, S.T)                              # <q_i,q_j> is symmetric, exactly so in integers


def test_score_table_matches_python_big_integers():
    rng = np.random.default_rng(3)
    q, c = unit_rows(rng, 2, 8), unit_rows(rng, 3, 8)
    S = oracle.score_table(q, c)
    for ci in range(3):
        for qi in range(2):
            t = sum(int(round(float(q[qi, d]) * 2 ** 22)) * int(round(float(c[ci, d]) * 2 ** 22)) for d in range(8))
            assert int(S[ci, qi]) == (t + 2 ** 19) // 2 ** 20  # python // floors


# ------------------------------------------------------------------ O-2 probes ------------------------------------

def test_probes_match_numpy_lexsort_with_ties():
    rng = np.random.default_rng(4)
    S = rng.integers(-5, 6, size=(50, 7)).astype(np.int32)    # many equal scores -> exercises the id tie-break
    for P in (1, 3, 50):
        got = oracle.probes(S, P)
        for i in range(7):
            order = np.lexsort((np.arange(50), -S[:, i].astype(np.int64)))
            assert np.array_equal(got[i], order[:P])


def test_probes_are_nested_in_nprobe():
    rng = np.random.default_rng(5)
    S = rng.integers(-2 ** 24, 2 ** 24, size=(64, 9)).astype(np.int32)
    prev = oracle.probes(S, 1)
    for P in range(2, 20):
        cur = oracle.probes(S, P)
        assert np.array_equal(cur[:, :P - 1], prev)
        prev = cur


# ------------------------------------------------------------------ O-3 candidates --------------------------------

def _index(seed, N=40, K=12, D=8, nbits=2, **kw):
    cent, cids, codes, doclens = random_corpus(seed, N, K, D, nbits, **kw)
    return oracle.make_index(cent, cids, codes, doclens, nbits)


def test_candidates_all_centroids_probed_gives_every_document():
    ix = _index(6)
    pr = np.arange(ix.K, dtype=np.int32).reshape(1, -1)
    assert np.array_equal(oracle.candidates(pr, ix), np.arange(ix.N))


def test_candidates_equal_set_definition():
    ix = _index(7, N=60, K=20)
    rng = np.random.default_rng(7)
    for _ in range(5):
        pr = rng.integers(0, ix.K, size=(3, 2)).astype(np.int32)
        probed = set(pr.ravel().tolist())
        want = [d for d in range(ix.N)
                if any(int(c) in probed for c in ix.cids[ix.doc_off[d]:ix.doc_off[d + 1]])]
        assert oracle.candidates(pr, ix).tolist() == want
    assert oracle.candidates(np.zeros((0,), np.int32), ix).size == 0


def test_candidates_grow_with_more_probes():
    ix = _index(8, N=80, K=30)
    prev = set()
    for m in range(1, 30):
        cur = set(oracle.candidates(np.arange(m, dtype=np.int32), ix).tolist())
        assert prev <= cur
        prev = cur


# ------------------------------------------------------------------ O-4 centroid interaction ----------------------

def test_ci_one_token_documents_is_a_column_sum():
    rng = np.random.default_rng(9)
    K, nq, N = 9, 5, 30
    S = rng.integers(-2 ** 24, 2 ** 24, size=(K, nq)).astype(np.int32)
    cids = rng.integers(0, K, size=N).astype(np.int32)
    ix = oracle.make_index(unit_rows(rng, K, 8), cids, np.zeros((N, 2), np.uint8), np.ones(N, np.int32), 2)
    cand = np.arange(N, dtype=np.int32)
    assert np.array_equal(oracle.ci_scores(S, cand, ix), S[cids].astype(np.int64).sum(1))


def test_ci_is_max_over_tokens_then_sum_over_query_tokens():
    rng = np.random.default_rng(10)
    ix = _index(10, N=25, K=10)
    S = rng.integers(-2 ** 24, 2 ** 24, size=(ix.K, 6)).astype(np.int32)
    cand = np.array([0, 3, 4, 11, 24], np.int32)
    want = [int(S[ix.cids[ix.doc_off[d]:ix.doc_off[d + 1]]].max(axis=0).astype(np.int64).sum()) for d in cand]
    assert oracle.ci_scores(S, cand, ix).tolist() == want


def test_ci_single_centroid_is_constant():
    rng = np.random.default_rng(11)
    S = rng.integers(-100, 100, size=(1, 4)).astype(np.int32)
    ix = oracle.make_index(unit_rows(rng, 1, 8), np.zeros(17, np.int32), np.zeros((17, 2), np.uint8),
                           np.array([5, 1, 11], np.int32), 2)
    assert oracle.ci_scores(S, np.arange(3, dtype=np.int32), ix).tolist() == [int(S.sum())] * 3


def test_ci_invariant_to_token_order_and_query_token_order():
    rng = np.random.default_rng(12)
    cent, cids, codes, doclens = random_corpus(12, 30, 10, 8, 2)
    ix = oracle.make_index(cent, cids, codes, doclens, 2)
    S = rng.integers(-2 ** 24, 2 ** 24, size=(10, 6)).astype(np.int32)
    cand = np.arange(30, dtype=np.int32)
    base = oracle.ci_scores(S, cand, ix)
    cids2 = cids.copy()
    for d in range(30):
        seg = slice(ix.doc_off[d], ix.doc_off[d + 1])
        cids2[seg] = rng.permutation(cids2[seg])
    ix2 = oracle.make_index(cent, cids2, codes, doclens, 2)
    assert np.array_equal(oracle.ci_scores(S, cand, ix2), base)
    assert np.array_equal(oracle.ci_scores(S[:, rng.permutation(6)].copy(), cand, ix), base)


def test_prune_matches_numpy_lexsort_and_is_nested():
    rng = np.random.default_rng(13)
    cand = np.sort(rng.choice(1000, size=200, replace=False)).astype(np.int32)
    ci = rng.integers(-4, 5, size=200).astype(np.int32)       # many ties
    order = np.lexsort((cand, -ci.astype(np.int64)))
    prev = set()
    for n in [0, 1, 2, 17, 199, 200, 500]:
        got = oracle.prune(cand, ci, n)
        want = np.sort(cand[order[:n]])
        assert np.array_equal(got, want)
        assert prev <= set(got.tolist())
        prev = set(got.tolist())


# ------------------------------------------------------------------ O-5 / O-7 scores ------------------------------

def test_chamfer_handworked():
    for row in _golden_rows("chamfer_handworked.txt"):
        shape, qs, vs, want = [p.split() for p in row.split("|")]
        nq, nv, D = map(int, shape)
        q = np.array(list(map(float, qs)), np.float32).reshape(nq, D)
        v = np.array(list(map(float, vs)), np.float32).reshape(nv, D)
        assert oracle.chamfer(q, v) == pytest.approx(float(want[0]), abs=1e-6)


def test_chamfer_of_unit_set_with_itself_is_its_size():
    rng = np.random.default_rng(14)
    for n, D in [(1, 8), (32, 128), (64, 96)]:
        q = unit_rows(rng, n, D)
        assert oracle.chamfer(q, q) == pytest.approx(float(n), abs=1e-5)


def test_chamfer_matches_numpy_and_is_not_symmetric():
    rng = np.random.default_rng(15)
    q, v = unit_rows(rng, 7, 16), unit_rows(rng, 13, 16)
    want = (q.astype(np.float64) @ v.astype(np.float64).T).max(axis=1).sum()
    assert oracle.chamfer(q, v) == pytest.approx(want, abs=1e-9)
    other = (v.astype(np.float64) @ q.astype(np.float64).T).max(axis=1).sum()
    assert oracle.chamfer(v, q) == pytest.approx(other, abs=1e-9)


def test_decode_handworked_packing():
    # one-token document, zero centroid, query = unit basis vector e_x  =>  score = reconstructed residual of dim x
    for row in _golden_rows("code_packing_handworked.txt"):
        head, vals = row.split("|")
        nbits, byte = map(int, head.split())
        want = list(map(float, vals.split()))
        D = 8                                  # one byte of 1-bit codes, two bytes of 2-bit codes
        nbytes = D * nbits // 8
        for pos in range(nbytes):
            codes = np.zeros((1, nbytes), np.uint8)
            codes[0, pos] = byte
            ix = oracle.make_index(np.zeros((1, D), np.float32), np.zeros(1, np.int32), codes, np.ones(1, np.int32),
                                   nbits)
            per_byte = 8 // nbits
            for t in range(per_byte):
                e = np.zeros((1, D), np.float32)
                e[0, pos * per_byte + t] = 1.0
                got = oracle.score_docs(e, np.array([0], np.int32), ix)
                assert got[0] == pytest.approx(want[t], abs=1e-7), (row, pos, t)


@pytest.mark.parametrize("D,nbits", [(128, 2), (128, 1), (96, 2), (96, 1), (8, 2)])
def test_score_docs_equals_chamfer_on_explicitly_decoded_vectors(D, nbits):
    rng = np.random.default_rng(16)
    cent, cids, codes, doclens = random_corpus(16, 12, 6, D, nbits, len_lo=1, len_hi=9)
    ix = oracle.make_index(cent, cids, codes, doclens, nbits)
    q = unit_rows(rng, 5, D)
    dec = cent[cids].astype(np.float32) + levels(nbits)[unpack_codes(codes, D, nbits)].astype(np.float32)
    docs = np.arange(12, dtype=np.int32)
    got = oracle.score_docs(q, docs, ix)
    for d in range(12):
        v = dec[ix.doc_off[d]:ix.doc_off[d + 1]].astype(np.float64)
        want = (q.astype(np.float64) @ v.T).max(axis=1).sum()
        assert got[d] == pytest.approx(want, rel=2e-7, abs=1e-6)
    assert oracle.score_docs(q, np.array([-1, 3], np.int32), ix)[0] == -np.inf


def test_score_docs_linear_decomposition_two_bit():
    # <q, c + r^> = <q,c> + delta * sum_x q_x u_x + (lo + delta/2) * sum_x q_x
    rng = np.random.default_rng(17)
    D = 128
    cent, cids, codes, doclens = random_corpus(17, 20, 5, D, 2, len_lo=1, len_hi=1)
    ix = oracle.make_index(cent, cids, codes, doclens, 2)
    q = unit_rows(rng, 1, D).astype(np.float64)
    u = unpack_codes(codes, D, 2).astype(np.float64)
    want = cent[cids].astype(np.float64) @ q[0] + 0.125 * (u @ q[0]) + (-0.25 + 0.0625) * q[0].sum()
    got = oracle.score_docs(q.astype(np.float32), np.arange(20, dtype=np.int32), ix)
    assert np.allclose(got, want, rtol=0, atol=2e-6)


def test_score_docs_one_bit_lookup_table_identity():
    # Sec. 4.1: <q,b> = sum_j T_q[j, b^(j)], T_q[j,u] = sum_{t<4} u_t q_{4j+t}.  With 1-bit codes over [-0.25, 0.25)
    # the residual is 0.25*b - 0.125, so score = <q,c> + 0.25 * <q,b> - 0.125 * sum(q).
    rng = np.random.default_rng(18)
    D = 128
    cent, cids, codes, doclens = random_corpus(18, 16, 4, D, 1, len_lo=1, len_hi=1)
    ix = oracle.make_index(cent, cids, codes, doclens, 1)
    q = unit_rows(rng, 1, D)[0].astype(np.float64)
    T = np.zeros((D // 4, 16))
    for j in range(D // 4):
        for uu in range(16):
            T[j, uu] = sum(((uu >> t) & 1) * q[4 * j + t] for t in range(4))
    assert T.size * 4 * 32 == 64 * 1024        # 64 KB of fp32 tables for 32 query tokens, as the paper states
    got = oracle.score_docs(q[None].astype(np.float32), np.arange(16, dtype=np.int32), ix)
    for d in range(16):
        nibbles = []
        for byte in codes[d]:
            nibbles += [int(byte) & 15, int(byte) >> 4]
        qb = sum(T[j, nibbles[j]] for j in range(D // 4))
        want = float(cent[cids[d]].astype(np.float64) @ q) + 0.25 * qb - 0.125 * q.sum()
        assert got[d] == pytest.approx(want, abs=2e-6)


# ------------------------------------------------------------------ O-6 top-k, Def. 3 recall ----------------------

def test_topk_matches_numpy_lexsort_ties_and_padding():
    rng = np.random.default_rng(19)
    docs = rng.permutation(300)[:100].astype(np.int32)
    docs[[5, 50]] = -1
    sc = rng.integers(0, 6, size=100).astype(np.float32) * 0.5
    valid = docs >= 0
    order = np.lexsort((docs[valid], -sc[valid].astype(np.float64)))
    for k in (1, 10, 98, 120):
        ids, top = oracle.topk(docs, sc, k)
        m = min(k, int(valid.sum()))
        assert np.array_equal(ids[:m], docs[valid][order[:m]])
        assert np.array_equal(top[:m], sc[valid][order[:m]])
        assert np.all(ids[m:] == -1) and np.all(np.isneginf(top[m:]))


def test_recall_handworked():
    # Def. 3: |R n R'| / k
    assert oracle.recall(np.array([1, 2, 3, 4]), np.array([4, 9, 1, 7])) == 0.5
    assert oracle.recall(np.array([1, 2, 3, 4]), np.array([1, 2, 3, 4])) == 1.0
    assert oracle.recall(np.array([1, 2, 3, 4]), np.array([5, 6, 7, 8])) == 0.0
    assert oracle.recall(np.array([7, -1]), np.array([-1, 7])) == 0.5


# ------------------------------------------------------------------ whole pipeline ---------------------------------

def _small_case(seed, N=120, K=24, D=16, nbits=2, nq=6):
    rng = np.random.default_rng(seed)
    cent, cids, codes, doclens = random_corpus(seed, N, K, D, nbits, len_lo=1, len_hi=10)
    return oracle.make_index(cent, cids, codes, doclens, nbits), unit_rows(rng, nq, D)


def test_pipeline_with_everything_probed_and_no_pruning_is_exhaustive_search():
    for seed, nbits in [(20, 2), (21, 1)]:
        ix, q = _small_case(seed, nbits=nbits)
        r = oracle.pipeline(q, ix, nprobe=ix.K, n_prune=ix.N, k=10)
        assert np.array_equal(r.cand, np.arange(ix.N))
        assert np.array_equal(r.pruned, np.arange(ix.N))
        # ground truth from the definition with numpy (explicit decode, Def. 1, Def. 2)
        dec = ix.centroids[ix.cids] + levels(nbits)[unpack_codes(ix.codes, ix.dim, nbits)].astype(np.float32)
        full = np.array([(q.astype(np.float64) @ dec[ix.doc_off[d]:ix.doc_off[d + 1]].astype(np.float64).T)
                         .max(axis=1).sum() for d in range(ix.N)])
        want = np.lexsort((np.arange(ix.N), -full))[:10]
        gaps = np.diff(-np.sort(-full)[:11])
        if np.all(np.abs(gaps) > 1e-5):                       # no near-ties: order is decided
            assert np.array_equal(r.ids, want)
        assert np.allclose(r.scores, full[r.ids], rtol=1e-6)
        ids, top, _ = oracle.exhaustive(q, ix, 10)
        assert np.array_equal(ids, r.ids) and np.array_equal(top, r.scores)


def test_pipeline_brute_force_from_definitions():
    ix, q = _small_case(22, N=50, K=16, D=8)
    nprobe, n_prune, k = 2, 7, 3
    r = oracle.pipeline(q, ix, nprobe, n_prune, k)
    # exact integer table from Python integers
    X = lambda a: int(round(float(a) * 2 ** 22))
    S = [[(sum(X(q[i, d]) * X(ix.centroids[c, d]) for d in range(8)) + 2 ** 19) // 2 ** 20 for i in range(len(q))]
         for c in range(ix.K)]
    assert r.S.tolist() == S
    probed = set()
    for i in range(len(q)):
        ranked = sorted(range(ix.K), key=lambda c: (-S[c][i], c))
        assert r.probes[i].tolist() == ranked[:nprobe]
        probed |= set(ranked[:nprobe])
    toks = lambda d: range(int(ix.doc_off[d]), int(ix.doc_off[d + 1]))
    cand = [d for d in range(ix.N) if any(int(ix.cids[t]) in probed for t in toks(d))]
    assert r.cand.tolist() == cand
    ci = [sum(max(S[int(ix.cids[t])][i] for t in toks(d)) for i in range(len(q))) for d in cand]
    assert r.ci.tolist() == ci
    keep = sorted(sorted(range(len(cand)), key=lambda j: (-ci[j], cand[j]))[:n_prune])
    assert r.pruned.tolist() == [cand[j] for j in keep]
    lv = levels(2)
    sc = []
    for d in r.pruned:
        tot = 0.0
        for i in range(len(q)):
            tot += max(sum(float(q[i, x]) * (float(np.float32(ix.centroids[ix.cids[t], x]
                                                             + np.float32(lv[(ix.codes[t, x // 4] >> (2 * (x % 4))) & 3]))))
                           for x in range(8)) for t in toks(d))
        sc.append(tot)
    assert np.allclose(r.score4, sc, rtol=1e-6)
    best = sorted(range(len(sc)), key=lambda j: (-r.score4[j], r.pruned[j]))[:k]
    assert r.ids.tolist() == [int(r.pruned[j]) for j in best]


def test_pipeline_nestedness_and_recall_monotone_in_n_prune():
    ix, q = _small_case(23, N=300, K=48, D=16, nq=8)
    k = 10
    truth, _, _ = oracle.exhaustive(q, ix, k)
    prev_c = set()
    for P in (1, 2, 4, 8, 48):
        r = oracle.pipeline(q, ix, P, 40, k)
        cur = set(r.cand.tolist())
        assert prev_c <= cur                                   # cand(P) subset of cand(P+1)
        prev_c = cur
    cand_recall = [len(set(truth.tolist()) & set(oracle.pipeline(q, ix, P, 40, k).cand.tolist())) / k
                   for P in (1, 2, 4, 8, 48)]
    assert cand_recall == sorted(cand_recall) and cand_recall[-1] == 1.0
    prev_p, prev_rec = set(), -1.0
    for n_prune in (10, 20, 40, 80, 160, 300):
        r = oracle.pipeline(q, ix, 4, n_prune, k)
        cur = set(r.pruned.tolist())
        assert prev_p <= cur                                   # pruned(n') subset of pruned(n'+1)
        rec = oracle.recall(truth, r.ids)
        assert rec >= prev_rec                                 # the final score is the ground-truth score
        assert rec == pytest.approx(len(set(truth.tolist()) & cur) / k)
        prev_p, prev_rec = cur, rec


def test_pipeline_invariant_to_query_token_order():
    ix, q = _small_case(24, N=200, K=32, D=16, nq=8)
    a = oracle.pipeline(q, ix, 3, 25, 5)
    perm = np.random.default_rng(24).permutation(8)
    b = oracle.pipeline(q[perm].copy(), ix, 3, 25, 5)
    assert np.array_equal(a.cand, b.cand) and np.array_equal(a.ci, b.ci) and np.array_equal(a.pruned, b.pruned)
    assert np.array_equal(a.probes[perm], b.probes)
    assert np.array_equal(a.ids, b.ids)


def test_tiny_config_candidate_count_matches_closed_form():
    # E|cand| = sum_d [1 - (1 - m/K)^len_d], m = number of distinct probed centroids (uniform component draws)
    import torch  # noqa: F401  (the generator is torch based)
    from synth import CONFIGS, make_corpus, make_queries
    cfg = CONFIGS["tiny"]
    corp = make_corpus(cfg)
    ix = oracle.make_index(corp.centroids, corp.cids, corp.codes, corp.doclens, cfg.nbits, cfg.res_lo, cfg.res_hi)
    q = make_queries(cfg, 2).numpy()
    assert 620_000 < corp.n_tokens < 660_000 and ix.N == 10_000
    for b in range(2):
        r = oracle.pipeline(q[b], ix, cfg.nprobe, cfg.n_prune, cfg.k)
        m = len(set(r.probes.ravel().tolist()))
        expect = float((1.0 - (1.0 - m / ix.K) ** ix.doclens.astype(np.float64)).sum())
        sd = np.sqrt(expect * (1 - expect / ix.N)) + 1
        assert abs(len(r.cand) - expect) < 6 * sd + 0.01 * expect
        assert len(r.pruned) == cfg.n_prune and np.all(np.diff(r.pruned) > 0)
        # the generating component is the nearest centroid: probe 0 of a query token scores ~ cos(noise angle)
        assert np.all(r.S[r.probes[:, 0], np.arange(cfg.q_len)] > 0.8 * 2 ** 24)


# ------------------------------------------------------------------ O-8 candidate refinement (Algorithm 2) --------

def test_partial_scores_handworked():
    D = 8
    cent = np.zeros((2, D), np.float32)
    cent[0, 0] = 1.0
    cent[1, 1] = 1.0
    q = cent.copy()
    cids = np.array([0, 0, 0, 0, 1, 1], np.int32)
    codes = np.array([[1], [0], [1], [0], [2], [0]], np.uint8)
    doclens = np.array([1, 2, 2, 1], np.int32)
    ix = oracle.make_index(cent, cids, codes, doclens, 1)
    S = oracle.score_table(q, cent)
    pr = oracle.probes(S, 1)
    assert pr.tolist() == [[0], [1]]
    cand = oracle.candidates(pr, ix)
    assert cand.tolist() == [0, 1, 2, 3]
    want = [int(r.split()[1]) for r in _golden_rows("partial_score_handworked.txt")]
    assert oracle.partial_scores(S, q, pr, cand, ix).tolist() == want


def test_partial_scores_with_every_list_probed_equal_the_full_low_bit_maxsim():
    # Sec. 3.2: F' only drops the tokens that were not retrieved; with every cluster probed V n L_q = V, so F' is the
    # full score of the decoded document (here every per-query-token maximum is positive, so the 0 floor is inactive)
    for nbits in (2, 1):
        ix, q = _small_case(30 + nbits, N=60, K=8, D=32, nbits=nbits, nq=5)
        S = oracle.score_table(q, ix.centroids)
        pr = oracle.probes(S, ix.K)
        cand = oracle.candidates(pr, ix)
        fp = oracle.partial_scores(S, q, pr, cand, ix)
        full = oracle.score_docs(q, cand, ix).astype(np.float64)
        dec = ix.centroids[ix.cids] + levels(nbits)[unpack_codes(ix.codes, ix.dim, nbits)].astype(np.float32)
        for j, d in enumerate(cand):
            per_q = (q.astype(np.float64) @ dec[ix.doc_off[d]:ix.doc_off[d + 1]].astype(np.float64).T).max(axis=1)
            if np.all(per_q > 1e-3):
                assert fp[j] * 2.0 ** -24 == pytest.approx(full[j], abs=5e-6)
            else:                                        # floor at 0 for query tokens whose best token is negative
                assert fp[j] * 2.0 ** -24 == pytest.approx(np.maximum(per_q, 0).sum(), abs=5e-6)


def test_partial_scores_brute_force_and_monotone_in_nprobe():
    ix, q = _small_case(33, N=80, K=16, D=16, nbits=2, nq=6)
    S = oracle.score_table(q, ix.centroids)
    X = lambda a: int(round(float(a) * 2 ** 22))
    delta = np.float32(0.5) / np.float32(4)
    kappa = np.float32(-0.25) + np.float32(0.5) * delta
    prev = None
    for P in (1, 2, 5, 16):
        pr = oracle.probes(S, P)
        cand = oracle.candidates(pr, ix)
        fp = oracle.partial_scores(S, q, pr, cand, ix)
        # Algorithm 2 from Python dictionaries, integers and one rounding per token
        score = {}
        for i in range(len(q)):
            xq = [X(v) for v in q[i]]
            for d in range(ix.N):
                for t in range(int(ix.doc_off[d]), int(ix.doc_off[d + 1])):
                    if int(ix.cids[t]) not in pr[i].tolist():
                        continue
                    T = sum(xq[x] * ((int(ix.codes[t, x // 4]) >> (2 * (x % 4))) & 3) for x in range(16))
                    r = float(delta) * 4.0 * float(T) + float(kappa) * 4.0 * float(sum(xq))
                    dist = int(S[ix.cids[t], i]) + int(np.rint(r))
                    score[(d, i)] = max(score.get((d, i), 0), dist)
        want = [sum(score.get((int(d), i), 0) for i in range(len(q))) for d in cand]
        assert fp.tolist() == want
        cur = dict(zip(cand.tolist(), fp.tolist()))
        if prev is not None:                                      # more retrieved tokens can only raise a maximum
            assert all(cur[d] >= v for d, v in prev.items())
        prev = cur


def test_pipeline_with_partial_scores_prunes_by_f_prime():
    ix, q = _small_case(34, N=150, K=24, D=16, nq=6)
    r = oracle.pipeline(q, ix, 3, 20, 5, partial=True)
    order = np.lexsort((r.cand, -r.ci.astype(np.int64)))[:20]
    assert np.array_equal(r.pruned, np.sort(r.cand[order]))
    assert np.array_equal(r.score4, oracle.score_docs(q, r.pruned, ix))


# ------------------------------------------------------------------ O-9 RaBitQ 1-bit codes (Sec. 2.2) --------------

def _rabitq_case(seed, N=40, K=8, D=64, nq=5):
    import torch
    from synth import CONFIGS, encode_rabitq_1bit, random_rotation
    rng = np.random.default_rng(seed)
    cent, cids, codes, doclens = random_corpus(seed, N, K, D, 1, len_lo=1, len_hi=8)
    raw = unit_rows(rng, len(cids), D)
    P = random_rotation(CONFIGS["tiny"].replace(dim=D, seed=seed))
    bits, inv = encode_rabitq_1bit(torch.from_numpy(raw), P)
    ix = oracle.make_index(cent, cids, codes, doclens, 1)
    rq = oracle.make_rabitq(P, bits, inv)
    return ix, rq, raw, unit_rows(rng, nq, D)


def test_rotation_is_orthonormal_and_rotate_matches_numpy():
    ix, rq, raw, q = _rabitq_case(40)
    P = rq.rotation.astype(np.float64)
    assert np.allclose(P @ P.T, np.eye(P.shape[0]), atol=1e-6)
    qp = oracle.rotate(rq.rotation, q)
    assert np.allclose(qp, q.astype(np.float64) @ P.T, atol=1e-6)
    assert np.allclose(np.linalg.norm(qp, axis=1), 1.0, atol=1e-6)
    # inner products are preserved by the rotation (Sec. 2.2)
    rp = oracle.rotate(rq.rotation, raw[:7])
    assert np.allclose(qp.astype(np.float64) @ rp.astype(np.float64).T, q.astype(np.float64) @ raw[:7].T.astype(np.float64),
                       atol=1e-6)


def test_rabitq_estimate_equals_codeword_formula_and_is_exact_on_codewords():
    ix, rq, raw, q = _rabitq_case(41, N=30, D=64)
    D = ix.dim
    qp = oracle.rotate(rq.rotation, q).astype(np.float64)
    # one-token documents: the score of document d for a single query token is est(q, token d)
    one = oracle.make_index(ix.centroids, ix.cids, ix.codes, np.ones(len(ix.cids), np.int32), 1)
    op = raw.astype(np.float64) @ rq.rotation.astype(np.float64).T
    obar = np.sign(op) / np.sqrt(D)                      # nearest codeword of G_r for B = 1
    want = (qp[:1] @ obar.T)[0] / np.einsum("td,td->t", op, obar)      # <q_p, o-bar> / <o_p, o-bar>
    got = oracle.rabitq_score_docs(qp[:1].astype(np.float32), np.arange(len(raw), dtype=np.int32), one, rq)
    assert np.allclose(got, want, atol=3e-6)
    # a token that IS a codeword is estimated exactly: est = <q, o>
    signs = np.where(np.random.default_rng(1).random((5, D)) > 0.5, 1.0, -1.0) / np.sqrt(D)
    tok = (signs @ rq.rotation.astype(np.float64)).astype(np.float32)          # o = P^T o_p
    import torch
    from synth import encode_rabitq_1bit
    bits, inv = encode_rabitq_1bit(torch.from_numpy(tok), torch.from_numpy(rq.rotation))
    rq2 = oracle.make_rabitq(rq.rotation, bits, inv)
    one2 = oracle.make_index(ix.centroids, np.zeros(5, np.int32), np.zeros((5, D // 8), np.uint8), np.ones(5, np.int32), 1)
    got2 = oracle.rabitq_score_docs(qp[:1].astype(np.float32), np.arange(5, dtype=np.int32), one2, rq2)
    assert np.allclose(got2, (q[:1].astype(np.float64) @ tok.astype(np.float64).T)[0], atol=5e-6)


def test_rabitq_estimator_is_unbiased_with_error_of_order_one_over_sqrt_d():
    # Sec. 2.2: the estimator is unbiased with a tight error bound; over many random unit vectors the mean error is
    # zero within its standard error and the error spread is a small multiple of 1/sqrt(D)
    import torch
    from synth import CONFIGS, encode_rabitq_1bit, random_rotation
    D, n = 128, 4000
    rng = np.random.default_rng(42)
    raw = unit_rows(rng, n, D)
    q = unit_rows(rng, 1, D)
    P = random_rotation(CONFIGS["tiny"].replace(seed=5))
    bits, inv = encode_rabitq_1bit(torch.from_numpy(raw), P)
    rq = oracle.make_rabitq(P, bits, inv)
    one = oracle.make_index(unit_rows(rng, 1, D), np.zeros(n, np.int32), np.zeros((n, D // 8), np.uint8),
                            np.ones(n, np.int32), 1)
    est = oracle.rabitq_score_docs(oracle.rotate(P.numpy(), q), np.arange(n, dtype=np.int32), one, rq).astype(np.float64)
    err = est - (raw.astype(np.float64) @ q[0].astype(np.float64))
    assert abs(err.mean()) < 4 * err.std() / np.sqrt(n)
    assert 0.2 / np.sqrt(D) < err.std() < 1.5 / np.sqrt(D)


def test_rabitq_lookup_table_identity():
    # Sec. 4.1: <q, b> = sum_j T_q[j, b^(j)] with 4-bit chunks; it is the integer T of the estimate
    ix, rq, raw, q = _rabitq_case(43, N=12, D=64)
    D = ix.dim
    qp = oracle.rotate(rq.rotation, q[:1])
    xq = np.rint(qp[0].astype(np.float64) * 2 ** 22)
    Tq = np.array([[sum(((u >> t) & 1) * xq[4 * j + t] for t in range(4)) for u in range(16)] for j in range(D // 4)])
    one = oracle.make_index(ix.centroids, ix.cids, ix.codes, np.ones(len(ix.cids), np.int32), 1)
    got = oracle.rabitq_score_docs(qp, np.arange(len(raw), dtype=np.int32), one, rq)
    c = np.float32(1.0 / (np.sqrt(float(D)) * 2.0 ** 22))
    for t in range(len(raw)):
        nib = []
        for byte in rq.bits[t]:
            nib += [int(byte) & 15, int(byte) >> 4]
        T = sum(Tq[j, nib[j]] for j in range(D // 4))
        want = rq.inv_dot[t] * np.float32(c * np.float32(2 * T - xq.sum()))
        assert got[t] == np.float32(want)


def test_rabitq_partial_with_every_list_probed_is_the_complete_one_bit_score():
    ix, rq, raw, q = _rabitq_case(44, N=50, K=8, D=64, nq=6)
    S = oracle.score_table(q, ix.centroids)
    pr = oracle.probes(S, ix.K)
    cand = oracle.candidates(pr, ix)
    qp = oracle.rotate(rq.rotation, q)
    fp = oracle.rabitq_partial(qp, pr, cand, ix, rq)
    # per query token max(0, max_t est), summed in fp32 in increasing i -- from one-token scores
    one = oracle.make_index(ix.centroids, ix.cids, ix.codes, np.ones(len(ix.cids), np.int32), 1)
    per_tok = np.stack([oracle.rabitq_score_docs(qp[i:i + 1], np.arange(len(ix.cids), dtype=np.int32), one, rq)
                        for i in range(len(q))])
    for j, d in enumerate(cand):
        tot = np.float32(0)
        for i in range(len(q)):
            tot = np.float32(tot + max(np.float32(0), per_tok[i, ix.doc_off[d]:ix.doc_off[d + 1]].max()))
        assert fp[j] == tot
    r = oracle.pipeline_rabitq(q, ix, rq, 2, 10, 4)
    assert len(r.pruned) == 10 and np.all(np.diff(r.pruned) > 0) and np.all(np.isin(r.ids, r.pruned))
    assert np.array_equal(r.score4, oracle.rabitq_score_docs(qp, r.pruned, ix, rq))


def test_rabitq_partial_handworked_with_unprobed_lists():
    # golden/rabitq_partial_handworked.txt: nprobe = 1 < K = 3, a query token that retrieves nothing of a document, a
    # token in a list only the OTHER query token probes, and a token in a list nobody probes
    D = 8
    toks = [[(0, 0x01, 1.0)], [(0, 0x00, 2.0), (0, 0x03, 1.0)], [(0, 0x00, 1.0), (1, 0x02, 2.0)],
            [(1, 0x03, 4.0), (2, 0x03, 4.0)], [(1, 0x01, 2.0)], [(2, 0x03, 1.0)]]
    flat = [t for d in toks for t in d]
    cids = np.array([t[0] for t in flat], np.int32)
    bits = np.array([[t[1]] for t in flat], np.uint8)
    inv = np.array([t[2] for t in flat], np.float32)
    ix = oracle.make_index(np.eye(3, D, dtype=np.float32), cids, np.zeros((len(flat), 1), np.uint8),
                           np.array([len(d) for d in toks], np.int32), 1)
    rq = oracle.make_rabitq(np.eye(D, dtype=np.float32), bits, inv)
    q = np.eye(2, D, dtype=np.float32)
    pr = np.array([[0], [1]], np.int32)
    cand = oracle.candidates(pr, ix)
    assert cand.tolist() == [0, 1, 2, 3, 4]
    fp = oracle.rabitq_partial(oracle.rotate(rq.rotation, q), pr, cand, ix, rq)
    rows = [r.split() for r in _golden_rows("rabitq_partial_handworked.txt")]
    assert [int(r[0]) for r in rows] == cand.tolist()
    assert fp.tolist() == [float(np.float32(float(r[1]))) for r in rows]


def test_rabitq_partial_brute_force_below_full_probing():
    # Algorithm 2 from Python dictionaries with the estimate of Sec. 2.2 built from the explicit nearest codeword
    # o_p-bar = sign(o_p) / sqrt(D) in float64 -- no oracle call produces the expectation.  nprobe < K, so which tokens
    # a query token retrieves (those of ITS OWN probed lists) decides the result.
    ix, rq, raw, q = _rabitq_case(45, N=60, K=16, D=64, nq=6)
    D = ix.dim
    S = oracle.score_table(q, ix.centroids)
    P64 = rq.rotation.astype(np.float64)
    qp64 = q.astype(np.float64) @ P64.T
    op = raw.astype(np.float64) @ P64.T
    obar = np.sign(op) / np.sqrt(D)
    est = (qp64 @ obar.T) / np.einsum("td,td->t", op, obar)[None, :]          # [nq, T]
    qp = oracle.rotate(rq.rotation, q)
    seen_partial = False
    for P in (1, 2, 5):
        pr = oracle.probes(S, P)
        cand = oracle.candidates(pr, ix)
        fp = oracle.rabitq_partial(qp, pr, cand, ix, rq)
        score = {}
        for i in range(len(q)):
            mine = set(pr[i].tolist())
            for d in range(ix.N):
                for t in range(int(ix.doc_off[d]), int(ix.doc_off[d + 1])):
                    if int(ix.cids[t]) in mine:
                        score[(d, i)] = max(score.get((d, i), 0.0), est[i, t])
        want = np.array([sum(score.get((int(d), i), 0.0) for i in range(len(q))) for d in cand])
        assert np.allclose(fp, want, atol=2e-5)
        # the case is selective: some candidate has a query token that retrieved none of its tokens
        seen_partial |= any((int(d), i) not in score for d in cand for i in range(len(q)))
        # and differs from probing every list for every query token (what a non-selective filter would compute)
        every = np.array([sum(max(0.0, est[i, ix.doc_off[d]:ix.doc_off[d + 1]].max()) for i in range(len(q)))
                          for d in cand])
        assert np.abs(every - want).max() > 1e-2
    assert seen_partial
