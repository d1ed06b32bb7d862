"""GPU parity of the proximity graph over the centroids and its search (the paper's replacement of the exhaustive
centroid scan) against the oracle: the graph, the probes with their scores, the visited sets and the RaBitQ pipeline
that starts from those probes, all bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from helpers import random_corpus, unit_rows

pytestmark = pytest.mark.gpu


def _visited_from_bitmap(bm, K):
    words = bm.cpu().numpy().view(np.uint32)
    bits = (words[:, :, None] >> np.arange(32, dtype=np.uint32)[None, None, :]) & 1
    return bits.reshape(words.shape[0], -1)[:, :K].astype(bool)


@pytest.mark.parametrize("K,D,R", [(2048, 128, 32), (1000, 96, 16), (300, 32, 63), (64, 64, 5)])
def test_graph_equals_oracle_graph(K, D, R):
    import paper_2608_23553_b200 as pkg
    cent, cids, codes, doclens = random_corpus(K + D, 50, K, D, 2)
    dev = torch.device("cuda:0")
    gix = pkg.Index(torch.from_numpy(cent).to(dev), torch.from_numpy(cids).to(dev), torch.from_numpy(codes).to(dev),
                    torch.from_numpy(doclens).to(dev), 2)
    assert gix.graph() is None
    gix.build_graph(R)
    assert np.array_equal(gix.graph().cpu().numpy(), oracle.knn_graph(cent, R))


def test_graph_with_identical_centroids_breaks_ties_towards_smaller_ids():
    import paper_2608_23553_b200 as pkg
    K, D, R = 200, 32, 6
    cent, cids, codes, doclens = random_corpus(77, 20, K, D, 2)
    cent[5] = cent[3]                    # identical twins and a triple: a centroid is not always its own best match
    cent[150] = cent[3]
    cent[199] = cent[198]
    dev = torch.device("cuda:0")
    gix = pkg.Index(torch.from_numpy(cent).to(dev), torch.from_numpy(cids).to(dev), torch.from_numpy(codes).to(dev),
                    torch.from_numpy(doclens).to(dev), 2)
    gix.build_graph(R)
    assert np.array_equal(gix.graph().cpu().numpy(), oracle.knn_graph(cent, R))


@pytest.mark.parametrize("K,D,R,nq,nprobe,beam,E,max_exp", [
    (2048, 128, 32, 32, 4, 32, 64, 1 << 30),
    (2048, 128, 32, 32, 4, 64, 256, 1 << 30),
    (1000, 96, 16, 40, 8, 16, 8, 5),
    (300, 32, 63, 5, 2, 2, 2, 1 << 30),
    (513, 64, 33, 7, 64, 64, 64, 3),
])
def test_graph_probes_scores_and_visited_sets_equal_oracle(K, D, R, nq, nprobe, beam, E, max_exp):
    import paper_2608_23553_b200 as pkg
    cent, cids, codes, doclens = random_corpus(K + nq, 50, K, D, 2)
    dev = torch.device("cuda:0")
    gix = pkg.Index(torch.from_numpy(cent).to(dev), torch.from_numpy(cids).to(dev), torch.from_numpy(codes).to(dev),
                    torch.from_numpy(doclens).to(dev), 2)
    gix.build_graph(R)
    g = oracle.knn_graph(cent, R)
    rng = np.random.default_rng(9)
    # query tokens near centroids (so that the search has something to find) and a few unrelated ones
    B = 3
    q = cent[rng.choice(K, B * nq)] + 0.2 * rng.standard_normal((B * nq, D)).astype(np.float32)
    q[::7] = unit_rows(rng, len(q[::7]), D)
    q /= np.linalg.norm(q, axis=1, keepdims=True)
    q = q.reshape(B, nq, D).astype(np.float32)
    pr, sc, nvis, bm = gix.graph_probes(torch.from_numpy(q).to(dev), nprobe, beam, E, max_exp)
    pr, sc, nvis = pr.cpu().numpy(), sc.cpu().numpy(), nvis.cpu().numpy()
    vis = _visited_from_bitmap(bm, K).reshape(B, nq, K)
    for b in range(B):
        o_pr, o_sc, o_vis = oracle.graph_probes(q[b], cent, g, nprobe, beam, E, max_exp)
        assert np.array_equal(pr[b], o_pr), "probes differ"
        assert np.array_equal(sc[b], o_sc), "probe scores differ"
        assert np.array_equal(vis[b], o_vis), "visited sets differ"
        assert np.array_equal(nvis[b], o_vis.sum(1))


def test_rabitq_pipeline_from_graph_probes_equals_oracle():
    import paper_2608_23553_b200 as pkg
    from synth import CONFIGS, make_corpus, make_queries
    cfg = CONFIGS["tiny"].replace(n_docs=3000, n_queries=4)
    corp = make_corpus(cfg, rabitq=True)
    oix = oracle.make_index(corp.centroids, corp.cids, corp.codes, corp.doclens, cfg.nbits, cfg.res_lo, cfg.res_hi)
    rq = oracle.make_rabitq(corp.rotation, corp.rq_bits, corp.rq_inv_dot)
    gix = pkg.Index(corp.centroids.cuda(), corp.cids.cuda(), corp.codes.cuda(), corp.doclens.cuda(), cfg.nbits,
                    cfg.res_lo, cfg.res_hi)
    gix.attach_rabitq(corp.rotation.cuda(), corp.rq_bits.cuda(), corp.rq_inv_dot.cuda())
    q = make_queries(cfg)
    with pytest.raises(pkg.ChimeraError):                       # no graph yet
        gix.search(q.cuda(), cfg.nprobe, 128, cfg.k, rabitq=True, graph=(32, 128, 1 << 30))
    R, beam, E = 24, 32, 128
    gix.build_graph(R)
    g = oracle.knn_graph(corp.centroids.numpy(), R)
    B, nprobe, k_refine, k = q.shape[0], cfg.nprobe, 128, cfg.k
    taps = gix.alloc_taps(B, cfg.q_len, nprobe, k_refine, table=False)
    ids, sc = gix.search(q.cuda(), nprobe, k_refine, k, taps=taps, rabitq=True, graph=(beam, E, 1 << 30))
    assert gix.status() == 0
    ids, sc = ids.cpu().numpy(), sc.cpu().numpy()
    exact_hits = 0
    for b in range(B):
        o_pr, _, _ = oracle.graph_probes(q[b].numpy(), corp.centroids.numpy(), g, nprobe, beam, E)
        assert np.array_equal(taps.probes[b].cpu().numpy(), o_pr)
        res = oracle.pipeline_rabitq(q[b].numpy(), oix, rq, nprobe, k_refine, k, probes_override=o_pr)
        n = int(taps.n_cand[b])
        assert n == len(res.cand) and np.array_equal(taps.cand[b, :n].cpu().numpy(), res.cand)
        assert np.array_equal(taps.ci[b, :n].cpu().numpy(), res.ci.view(np.int32))
        m = int(taps.n_pruned[b])
        assert np.array_equal(taps.pruned[b, :m].cpu().numpy(), res.pruned)
        assert np.array_equal(taps.score4[b, :m].cpu().numpy(), res.score4)
        assert np.array_equal(ids[b], res.ids) and np.array_equal(sc[b], res.scores)
        exact_hits += int((o_pr[:, 0] == res.probes[:, 0]).sum())          # res.probes = what was passed in
    # the plain RaBitQ search is untouched by the graph
    a = gix.search(q.cuda(), nprobe, k_refine, k, rabitq=True)
    r0 = oracle.pipeline_rabitq(q[0].numpy(), oix, rq, nprobe, k_refine, k)
    assert np.array_equal(a[0][0].cpu().numpy(), r0.ids)
