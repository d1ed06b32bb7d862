"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle on the same seeded inputs.

Bit-exact for the score table, probes, candidate sets, centroid-interaction scores and pruned ids; 1e-3 relative for
stage-4 scores; the top-k rule of tests/parity.py for the final ids.
"""
import numpy as np
import pytest
import torch

import oracle
from helpers import random_corpus, unit_rows
from parity import REL_TOL, check_query, check_topk, taps_to_numpy

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def chimera():
    import paper_2608_23553_b200 as pkg
    pkg.lib()
    return pkg


def _gpu_index(pkg, cent, cids, codes, doclens, nbits, lo=-0.25, hi=0.25):
    dev = torch.device("cuda:0")
    return pkg.Index(torch.from_numpy(cent).to(dev), torch.from_numpy(cids).to(dev), torch.from_numpy(codes).to(dev),
                     torch.from_numpy(doclens).to(dev), nbits, lo, hi)


def _run_and_check(pkg, gix, oix, q, nprobe, n_prune, k, table=True):
    """q: [B, nq, D] numpy.  Tapped search of the batch, every query checked against the oracle."""
    B, nq, _ = q.shape
    taps = gix.alloc_taps(B, nq, nprobe, n_prune, table=table)
    ids, sc = gix.search(torch.from_numpy(q).cuda(), nprobe, n_prune, k, taps=taps)
    assert gix.status() == 0
    tn = taps_to_numpy(taps)
    ids, sc = ids.cpu().numpy(), sc.cpu().numpy()
    diffs = 0
    for b in range(B):
        res = oracle.pipeline(q[b], oix, nprobe, n_prune, k)
        diffs += check_query(tn, b, res, ids[b], sc[b], k, n_prune, table=table)
    return diffs, ids, sc


@pytest.mark.parametrize("D,nbits,nq,K,N,nprobe,n_prune,k", [
    (32, 2, 5, 16, 60, 2, 7, 3),          # ragged everything
    (128, 2, 32, 64, 400, 4, 50, 10),
    (128, 1, 32, 64, 400, 4, 50, 10),
    (96, 2, 64, 48, 300, 8, 40, 12),      # two column groups, D = 96
    (96, 1, 40, 48, 300, 3, 33, 5),       # q_len not a multiple of 32
    (64, 2, 100, 32, 200, 5, 64, 64),     # four column groups
    (128, 2, 1, 8, 30, 1, 4, 2),          # single query token
])
def test_small_corpora_all_stages(chimera, D, nbits, nq, K, N, nprobe, n_prune, k):
    cent, cids, codes, doclens = random_corpus(100 + D + nq, N, K, D, nbits, len_lo=1, len_hi=70)
    oix = oracle.make_index(cent, cids, codes, doclens, nbits)
    gix = _gpu_index(chimera, cent, cids, codes, doclens, nbits)
    rng = np.random.default_rng(5)
    q = np.stack([unit_rows(rng, nq, D) for _ in range(3)])
    _run_and_check(chimera, gix, oix, q, nprobe, n_prune, k)
    info = gix.info()
    assert info["max_doclen"] == int(doclens.max()) and info["n_tokens"] == int(doclens.sum())
    # inverted file size = number of distinct (centroid, document) pairs
    doc_of = np.repeat(np.arange(N), doclens)
    assert info["posting_entries"] == len(set(zip(cids.tolist(), doc_of.tolist())))


def test_all_centroids_probed_gives_every_document_and_exhaustive_topk(chimera):
    D, nbits, K, N = 64, 2, 32, 150
    cent, cids, codes, doclens = random_corpus(7, N, K, D, nbits, len_lo=1, len_hi=20)
    oix = oracle.make_index(cent, cids, codes, doclens, nbits)
    gix = _gpu_index(chimera, cent, cids, codes, doclens, nbits)
    q = unit_rows(np.random.default_rng(8), 8, D)[None]
    taps = gix.alloc_taps(1, 8, K, N)
    ids, sc = gix.search(torch.from_numpy(q).cuda(), K, N, 10, taps=taps)
    tn = taps_to_numpy(taps)
    assert int(tn["n_cand"][0]) == N and np.array_equal(tn["cand"][0], np.arange(N))
    assert np.array_equal(tn["pruned"][0], np.arange(N))
    truth_ids, truth_sc, _ = oracle.exhaustive(q[0], oix, 10)
    res = oracle.pipeline(q[0], oix, K, N, 10)
    assert np.array_equal(res.ids, truth_ids)
    check_topk(ids[0].cpu().numpy(), sc[0].cpu().numpy(), res, 10)


def test_ties_are_broken_towards_smaller_ids(chimera):
    # duplicated centroids give equal scores; duplicated documents give equal CI and equal final scores
    D, nbits = 32, 2
    rng = np.random.default_rng(9)
    base = unit_rows(rng, 6, D)
    cent = np.concatenate([base, base, base[:4]])              # 16 centroids, many exact duplicates
    doc_cids = [rng.integers(0, 16, size=rng.integers(1, 9)) for _ in range(20)]
    doc_codes = [rng.integers(0, 256, size=(len(c), D * nbits // 8)) for c in doc_cids]
    order = list(range(20)) * 3                                  # every document three times
    cids = np.concatenate([doc_cids[i] for i in order]).astype(np.int32)
    codes = np.concatenate([doc_codes[i] for i in order]).astype(np.uint8)
    doclens = np.array([len(doc_cids[i]) for i in order], np.int32)
    oix = oracle.make_index(cent, cids, codes, doclens, nbits)
    gix = _gpu_index(chimera, cent, cids, codes, doclens, nbits)
    q = np.stack([unit_rows(rng, 7, D) for _ in range(2)])
    for nprobe, n_prune, k in [(3, 10, 5), (5, 31, 31), (16, 60, 60), (2, 1, 1)]:
        diffs, _, _ = _run_and_check(chimera, gix, oix, q, nprobe, n_prune, k)
        assert diffs == 0                                        # identical scores: order decided by id


def test_padding_when_few_survivors(chimera):
    D, nbits, K, N = 32, 1, 16, 12
    cent, cids, codes, doclens = random_corpus(10, N, K, D, nbits, len_lo=1, len_hi=3)
    oix = oracle.make_index(cent, cids, codes, doclens, nbits)
    gix = _gpu_index(chimera, cent, cids, codes, doclens, nbits)
    q = unit_rows(np.random.default_rng(11), 4, D)[None]
    # k > n_prune > number of candidates
    _, ids, sc = _run_and_check(chimera, gix, oix, q, 1, 50, 100)
    assert (ids[0] == -1).sum() >= 50


def test_candidate_overflow_is_reported(chimera):
    D, nbits, K, N = 32, 2, 8, 200
    cent, cids, codes, doclens = random_corpus(12, N, K, D, nbits, len_lo=2, len_hi=6)
    gix = _gpu_index(chimera, cent, cids, codes, doclens, nbits)
    q = torch.from_numpy(unit_rows(np.random.default_rng(13), 4, D)[None]).cuda()
    gix.search(q, 8, 10, 5, max_candidates=16)
    assert gix.status() == 4
    gix.search(q, 8, 10, 5)
    assert gix.status() == 0
    bad = q.clone()
    bad[0, 0, 0] = 1.5
    gix.search(bad, 8, 10, 5)
    assert gix.status() == 1
    # a query token twice as long as a unit vector (every element inside [-1, 1]): the stage-3 bounds assume unit
    # norms, so it is reported as well
    long_q = q.clone()
    long_q[0, 2] *= 2.0
    assert float(long_q.abs().max()) <= 1.0
    gix.search(long_q, 8, 10, 5)
    assert gix.status() == 1
    gix.search(q, 8, 10, 5)
    assert gix.status() == 0
    # and a centroid that is not unit-norm is rejected when the index is built
    cent2 = cent.copy()
    cent2[5] *= 1.5
    assert np.abs(cent2).max() <= 1.0
    with pytest.raises(chimera.ChimeraError) as e:
        _gpu_index(chimera, cent2, cids, codes, doclens, nbits)
    assert e.value.code == 1


def test_bad_index_arrays_are_rejected(chimera):
    D, nbits, K, N = 32, 2, 8, 20
    cent, cids, codes, doclens = random_corpus(14, N, K, D, nbits)
    bad = cids.copy()
    bad[3] = K
    with pytest.raises(chimera.ChimeraError) as e:
        _gpu_index(chimera, cent, bad, codes, doclens, nbits)
    assert e.value.code == 1
    bad_len = doclens.copy()
    bad_len[0] += 1
    with pytest.raises(chimera.ChimeraError):
        _gpu_index(chimera, cent, cids, codes, bad_len, nbits)


@pytest.fixture(scope="module")
def tiny(chimera):
    from synth import CONFIGS, make_corpus, make_queries
    cfg = CONFIGS["tiny"]
    corp = make_corpus(cfg)
    oix = oracle.make_index(corp.centroids, corp.cids, corp.codes, corp.doclens, cfg.nbits, cfg.res_lo, cfg.res_hi)
    gix = chimera.Index(corp.centroids.cuda(), corp.cids.cuda(), corp.codes.cuda(), corp.doclens.cuda(), cfg.nbits,
                        cfg.res_lo, cfg.res_hi)
    q = make_queries(cfg).numpy()
    return cfg, oix, gix, q


def test_tiny_config_all_queries_all_stages(chimera, tiny):
    cfg, oix, gix, q = tiny
    diffs, ids, sc = _run_and_check(chimera, gix, oix, q, cfg.nprobe, cfg.n_prune, cfg.k)
    assert diffs == 0


def test_tiny_config_batch_invariance_and_host_entry(chimera, tiny):
    cfg, oix, gix, q = tiny
    qd = torch.from_numpy(q).cuda()
    ids16, sc16 = gix.search(qd, cfg.nprobe, cfg.n_prune, cfg.k)
    ids16, sc16 = ids16.clone(), sc16.clone()
    for b in range(q.shape[0]):
        ids1, sc1 = gix.search(qd[b:b + 1].contiguous(), cfg.nprobe, cfg.n_prune, cfg.k)
        assert torch.equal(ids1[0], ids16[b]) and torch.equal(sc1[0], sc16[b])
    hid, hsc = gix.search_host(torch.from_numpy(q).pin_memory(), cfg.nprobe, cfg.n_prune, cfg.k)
    assert torch.equal(hid, ids16.cpu()) and torch.equal(hsc, sc16.cpu())


def test_tiny_config_stage_isolated(chimera, tiny):
    """Each stage fed with the ORACLE's results of the stages before it."""
    cfg, oix, gix, q = tiny
    B = 4
    res = [oracle.pipeline(q[b], oix, cfg.nprobe, cfg.n_prune, cfg.k) for b in range(B)]
    dev = torch.device("cuda:0")
    qd = torch.from_numpy(q[:B]).to(dev)
    N = oix.N

    def fresh():
        return gix.alloc_taps(B, cfg.q_len, cfg.nprobe, cfg.n_prune)

    table = torch.from_numpy(np.stack([r.S for r in res])).to(dev)
    cand = torch.zeros(B, N, dtype=torch.int32, device=dev)
    n_cand = torch.tensor([len(r.cand) for r in res], dtype=torch.int32, device=dev)
    pruned = torch.full((B, cfg.n_prune), -1, dtype=torch.int32, device=dev)
    n_pruned = torch.tensor([len(r.pruned) for r in res], dtype=torch.int32, device=dev)
    score4 = torch.full((B, cfg.n_prune), float("-inf"), device=dev)
    for b, r in enumerate(res):
        cand[b, :len(r.cand)] = torch.from_numpy(r.cand).to(dev)
        pruned[b, :len(r.pruned)] = torch.from_numpy(r.pruned).to(dev)
        score4[b, :len(r.pruned)] = torch.from_numpy(r.score4).to(dev)

    # stage 1 alone
    t = fresh()
    gix.run_stages(1, 1, qd, B, cfg.q_len, cfg.nprobe, cfg.n_prune, cfg.k, t)
    assert torch.equal(t.score_table, table)
    # stage 2 from the oracle's table
    t = fresh()
    t.score_table = table
    gix.run_stages(2, 2, None, B, cfg.q_len, cfg.nprobe, cfg.n_prune, cfg.k, t)
    for b, r in enumerate(res):
        assert np.array_equal(t.probes[b].cpu().numpy(), r.probes)
        assert int(t.n_cand[b]) == len(r.cand) and np.array_equal(t.cand[b, :len(r.cand)].cpu().numpy(), r.cand)
    # stage 3 from the oracle's table and candidates
    t = fresh()
    t.score_table, t.cand, t.n_cand = table, cand, n_cand
    gix.run_stages(3, 3, None, B, cfg.q_len, cfg.nprobe, cfg.n_prune, cfg.k, t)
    for b, r in enumerate(res):
        assert np.array_equal(t.ci[b, :len(r.cand)].cpu().numpy(), r.ci)
        assert np.array_equal(t.pruned[b, :len(r.pruned)].cpu().numpy(), r.pruned)
    # stage 4 from the oracle's table and pruned ids
    t = fresh()
    t.score_table, t.pruned, t.n_pruned = table, pruned, n_pruned
    gix.run_stages(4, 4, qd, B, cfg.q_len, cfg.nprobe, cfg.n_prune, cfg.k, t)
    for b, r in enumerate(res):
        got = t.score4[b, :len(r.pruned)].cpu().numpy()
        assert np.all(np.abs(got - r.score4) <= REL_TOL * np.abs(r.score4))
        assert np.abs(got - r.score4).max() <= 2e-5 * np.abs(r.score4).max()     # what fp32 accumulation gives
    # stage 5 from the oracle's scores: exact
    t = fresh()
    t.pruned, t.n_pruned, t.score4 = pruned, n_pruned, score4
    ids, sc = gix.run_stages(5, 5, None, B, cfg.q_len, cfg.nprobe, cfg.n_prune, cfg.k, t)
    for b, r in enumerate(res):
        assert np.array_equal(ids[b].cpu().numpy(), r.ids) and np.array_equal(sc[b].cpu().numpy(), r.scores)


@pytest.mark.parametrize("n_prune,k", [(17, 17), (100, 128), (128, 100), (129, 64), (1000, 100), (2048, 50),
                                        (4096, 100), (4096, 128), (4097, 100), (5000, 129), (3000, 10), (300, 1000),
                                        (16384, 1000), (16384, 100), (16384, 16384), (9000, 5000), (8193, 129)])
def test_topk_stage_alone_equals_a_plain_sort(chimera, tiny, n_prune, k):
    """Stage 5 on crafted survivors (every kernel variant: k <= 16, k <= 128 over <= 4096 entries, the full network up
    to its 16,384 keys):
    many equal scores, -1 padding inside the valid count's tail, fewer survivors than k.  Expected = Definition 2
    written as a sort by (score descending, id ascending)."""
    cfg, oix, gix, q = tiny
    B = 3
    rng = np.random.default_rng(n_prune * 1000 + k)
    dev = torch.device("cuda:0")
    pruned = np.full((B, n_prune), -1, dtype=np.int32)
    score4 = np.full((B, n_prune), -np.inf, dtype=np.float32)
    n_pruned = np.array([n_prune, max(1, n_prune // 3), min(n_prune, 5)], dtype=np.int32)
    for b in range(B):
        m = int(n_pruned[b])
        pruned[b, :m] = np.sort(rng.choice(max(oix.N, 4 * n_prune), size=m, replace=False)).astype(np.int32)   # stage 5 never looks a document up
        # few distinct values (ties decided by id), both signs, and exact zeros
        score4[b, :m] = rng.choice(np.array([-3.5, -0.0, 0.0, 1.25, 1.25000012, 7.0, 19.75], dtype=np.float32), size=m)
    t = gix.alloc_taps(B, cfg.q_len, cfg.nprobe, n_prune)
    t.pruned, t.n_pruned = torch.from_numpy(pruned).to(dev), torch.from_numpy(n_pruned).to(dev)
    t.score4 = torch.from_numpy(score4).to(dev)
    ids, sc = gix.run_stages(5, 5, None, B, cfg.q_len, cfg.nprobe, n_prune, k, t)
    ids, sc = ids.cpu().numpy(), sc.cpu().numpy()
    for b in range(B):
        m = int(n_pruned[b])
        order = np.lexsort((pruned[b, :m], -score4[b, :m].astype(np.float64)))[:k]
        want_ids = np.full(k, -1, dtype=np.int32)
        want_sc = np.full(k, -np.inf, dtype=np.float32)
        want_ids[:len(order)] = pruned[b, order]
        want_sc[:len(order)] = score4[b, order]
        assert np.array_equal(ids[b], want_ids)
        assert np.array_equal(sc[b], want_sc)


def test_tiny_config_parameter_grid(chimera, tiny):
    cfg, oix, gix, q = tiny
    for nprobe, n_prune, k in [(1, 256, 10), (2, 1024, 100), (8, 64, 10), (32, 4096, 1000), (16, 16384, 10),
                               (4, 2048, 16), (6, 300, 17)]:
        # check_topk (inside) allows position swaps only between scores within the tolerance; with k = 1000 of 4096
        # survivors a few fp32 near-ties are expected
        diffs, _, _ = _run_and_check(chimera, gix, oix, q[:2], nprobe, n_prune, k, table=False)
        assert diffs <= 8


def test_tiny_config_recall_against_exhaustive(chimera, tiny):
    cfg, oix, gix, q = tiny
    qd = torch.from_numpy(q[:3]).cuda()
    ids, _ = gix.search(qd, cfg.nprobe, cfg.n_prune, cfg.k)
    ids = ids.cpu().numpy()
    for b in range(3):
        truth, _, _ = oracle.exhaustive(q[b], oix, cfg.k)
        res = oracle.pipeline(q[b], oix, cfg.nprobe, cfg.n_prune, cfg.k)
        assert oracle.recall(truth, ids[b]) == oracle.recall(truth, res.ids)


def test_sweep_ground_truth_equals_the_oracles_exhaustive_scores(chimera, tiny):
    """The recall sweeps of bench.py take their ground truth from bench.brute_force_maxsim (exhaustive MaxSim written
    from the definition in plain torch; no library call).  Here it is compared with the oracle's exhaustive MaxSim on
    the whole Tiny corpus, all 16 queries: every score, and the top-k set by the usual rule."""
    import bench
    from parity import score_tol
    from synth import CONFIGS, make_corpus
    cfg, oix, gix, q = tiny
    k = 100
    corp = make_corpus(cfg)
    dev = torch.device("cuda:0")
    qd = torch.from_numpy(q).to(dev)
    scores = bench.brute_force_maxsim(corp.centroids.to(dev), corp.cids.to(dev), corp.codes.to(dev),
                                      corp.doclens.to(dev), cfg.nbits, cfg.res_lo, cfg.res_hi, qd, q_group=5,
                                      chunk_tokens=100_000).cpu().numpy()
    # the same through the sweep's own helper (top-k by score)
    class _C:                                          # the corpus fields exhaustive_truth reads, on the device
        centroids, cids, codes, doclens = corp.centroids.to(dev), corp.cids.to(dev), corp.codes.to(dev), corp.doclens.to(dev)
    ids, sc = bench.exhaustive_truth(_C, cfg, qd, k)
    ids, sc = ids.cpu().numpy(), sc.cpu().numpy()
    for b in range(q.shape[0]):
        t_ids, t_sc, all_sc = oracle.exhaustive(q[b], oix, k)
        assert np.all(np.abs(scores[b] - all_sc) <= 1e-5 * np.maximum(1.0, np.abs(all_sc)))
        tau = float(t_sc[-1])
        tol = float(score_tol(tau, cfg.q_len))
        assert len(set(ids[b].tolist())) == k
        assert np.all(all_sc[ids[b]] >= tau - tol)
        assert np.all(np.isin(t_ids[t_sc > tau + tol], ids[b]))
        assert oracle.recall(t_ids, ids[b]) >= 0.99


def test_graphed_search_equals_eager(chimera, tiny):
    cfg, oix, gix, q = tiny
    qd = torch.from_numpy(q).cuda()
    g = chimera.GraphedSearch(gix, 1, cfg.q_len, cfg.nprobe, cfg.n_prune, cfg.k)
    for b in (0, 5, 15):
        ids_e, sc_e = gix.search(qd[b:b + 1].contiguous(), cfg.nprobe, cfg.n_prune, cfg.k)
        ids_e, sc_e = ids_e.clone(), sc_e.clone()
        ids_g, sc_g = g(qd[b:b + 1])
        torch.cuda.synchronize()
        assert torch.equal(ids_g, ids_e) and torch.equal(sc_g, sc_e)


def test_unaligned_queries_are_rejected(chimera, tiny):
    """The query pointer must be 16-byte aligned (the kernels read rows with 16-byte loads)."""
    cfg, oix, gix, q = tiny
    flat = torch.zeros(q[:1].size + 1, dtype=torch.float32, device="cuda")
    shifted = flat[1:].view(1, cfg.q_len, cfg.dim)            # 4 bytes past an aligned address
    shifted.copy_(torch.from_numpy(q[:1]))
    with pytest.raises(chimera.ChimeraError):
        gix.search(shifted, cfg.nprobe, cfg.n_prune, cfg.k)
