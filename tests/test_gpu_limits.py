"""Parity at the API's maxima: n_prune = 16384 as a real selection (more than 16,384 candidates), with k = 100 and
k = 1000 behind it (stage 5's sorting network over 16,384 keys in 128 KB of shared memory)."""
import numpy as np
import pytest
import torch

import oracle
from parity import check_query, taps_to_numpy

pytestmark = pytest.mark.gpu


def test_n_prune_16384_is_a_real_selection_and_topk_sorts_16384_keys():
    import paper_2608_23553_b200 as pkg
    from synth import CONFIGS, make_corpus, make_queries
    # Tiny's recipe with four times the documents: nprobe 4 x 32 query tokens of 1,024 centroids reach nearly all of
    # the 40,000 documents, so the selection really drops more than half of the candidates
    cfg = CONFIGS["tiny"].replace(n_docs=40_000, n_queries=3)
    corp = make_corpus(cfg)
    q = make_queries(cfg).numpy()
    oix = oracle.make_index(corp.centroids, corp.cids, corp.codes, corp.doclens, cfg.nbits, cfg.res_lo, cfg.res_hi)
    gix = pkg.Index(corp.centroids.cuda(), corp.cids.cuda(), corp.codes.cuda(), corp.doclens.cuda(), cfg.nbits,
                    cfg.res_lo, cfg.res_hi)
    n_prune, B = 16384, q.shape[0]
    res = [oracle.pipeline(q[b], oix, cfg.nprobe, n_prune, 1000) for b in (0, B - 1)]
    assert all(len(r.cand) > 2 * n_prune and len(r.pruned) == n_prune for r in res)
    for k in (1000, 100):
        taps = gix.alloc_taps(B, cfg.q_len, cfg.nprobe, n_prune, table=False)
        ids, sc = gix.search(torch.from_numpy(q).cuda(), cfg.nprobe, n_prune, k, taps=taps)
        assert gix.status() == 0
        tn = taps_to_numpy(taps)
        ids, sc = ids.cpu().numpy(), sc.cpu().numpy()
        for r, b in zip(res, (0, B - 1)):
            r_k = oracle.Result(r.S, r.probes, r.cand, r.ci, r.pruned, r.score4, *oracle.topk(r.pruned, r.score4, k))
            # swaps are only allowed between scores within the tolerance (rule inside check_query)
            assert check_query(tn, b, r_k, ids[b], sc[b], k, n_prune, table=False) <= 8
    # the same selection through the partial-score refinement (its selection runs over every candidate)
    gix.enable_partial()
    taps = gix.alloc_taps(B, cfg.q_len, cfg.nprobe, n_prune, table=False)
    ids, sc = gix.search(torch.from_numpy(q).cuda(), cfg.nprobe, n_prune, 100, taps=taps, partial=True)
    assert gix.status() == 0
    tn = taps_to_numpy(taps)
    r = oracle.pipeline(q[1], oix, cfg.nprobe, n_prune, 100, partial=True)
    assert check_query(tn, 1, r, ids[1].cpu().numpy(), sc[1].cpu().numpy(), 100, n_prune, table=False) <= 8
