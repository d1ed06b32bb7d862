"""Parity on the other workload shapes: the long-document precision variants (512-token documents, 64-token queries,
dim 96/128, 1/2 residual bits) at reduced document count and one of them at full size (the passage-corpus-shaped
Large corpus has its own file, test_gpu_large.py)."""
import numpy as np
import pytest
import torch

import oracle
from parity import check_query, taps_to_numpy

pytestmark = pytest.mark.gpu


def _properties(tn, ids_np, sc_np, b, cfg, N, k):
    n = int(tn["n_cand"][b])
    cand = tn["cand"][b, :n]
    assert np.all(np.diff(cand) > 0) and cand[0] >= 0 and cand[-1] < N
    m = int(tn["n_pruned"][b])
    pruned = tn["pruned"][b, :m]
    assert m == min(cfg.n_prune, n) and np.all(np.diff(pruned) > 0) and np.all(np.isin(pruned, cand))
    valid = ids_np[b] >= 0
    assert np.all(np.isin(ids_np[b][valid], pruned)) and np.all(np.diff(sc_np[b][valid]) <= 0)
    best = np.lexsort((pruned, -tn["score4"][b, :m].astype(np.float64)))[:k]
    assert np.array_equal(pruned[best], ids_np[b][:len(best)])


@pytest.mark.parametrize("name", ["long_d128_b2", "long_d128_b1", "long_d96_b2", "long_d96_b1"])
def test_long_document_variants_reduced(name):
    import paper_2608_23553_b200 as pkg
    from synth import CONFIGS, make_corpus, make_queries
    cfg = CONFIGS[name].replace(n_docs=4000, n_prune=256, n_queries=4)
    dev = torch.device("cuda:0")
    corp = make_corpus(cfg, device=dev)
    q = make_queries(cfg, device=dev)
    gix = pkg.Index(corp.centroids, corp.cids, corp.codes, corp.doclens, cfg.nbits, cfg.res_lo, cfg.res_hi)
    oix = oracle.make_index(corp.centroids, corp.cids, corp.codes, corp.doclens, cfg.nbits, cfg.res_lo, cfg.res_hi)
    B = q.shape[0]
    taps = gix.alloc_taps(B, cfg.q_len, cfg.nprobe, cfg.n_prune)
    ids, sc = gix.search(q, cfg.nprobe, cfg.n_prune, cfg.k, taps=taps)
    assert gix.status() == 0
    tn = taps_to_numpy(taps)
    ids_np, sc_np, q_np = ids.cpu().numpy(), sc.cpu().numpy(), q.cpu().numpy()
    for b in (0, B - 1):
        res = oracle.pipeline(q_np[b], oix, cfg.nprobe, cfg.n_prune, cfg.k)
        assert check_query(tn, b, res, ids_np[b], sc_np[b], cfg.k, cfg.n_prune) == 0
    for b in range(B):
        _properties(tn, ids_np, sc_np, b, cfg, oix.N, cfg.k)


def test_long_document_corpus_full_size_sampled_query():
    """The long-document workload at full size in the launch configuration the benchmark times (200,000 documents of
    512 tokens, 64-token queries, batch 64, nprobe 8: nearly every document is a candidate): one sampled query against
    the oracle stage by stage, every query for the properties that hold at any size."""
    import psutil
    import paper_2608_23553_b200 as pkg
    from synth import CONFIGS, make_corpus, make_queries
    if psutil.virtual_memory().available < 16e9:
        pytest.skip("needs ~8 GB of host memory for the oracle's copy of the corpus")
    cfg = CONFIGS["long_d128_b2"]
    dev = torch.device("cuda:0")
    corp = make_corpus(cfg, device=dev)
    assert corp.n_tokens == 200_000 * 512
    B = 64
    q = make_queries(cfg, B, device=dev)
    gix = pkg.Index(corp.centroids, corp.cids, corp.codes, corp.doclens, cfg.nbits, cfg.res_lo, cfg.res_hi)
    taps = gix.alloc_taps(B, cfg.q_len, cfg.nprobe, cfg.n_prune, table=False)
    ids, sc = gix.search(q, cfg.nprobe, cfg.n_prune, cfg.k, taps=taps)
    assert gix.status() == 0
    tn = taps_to_numpy(taps)
    ids_np, sc_np, q_np = ids.cpu().numpy(), sc.cpu().numpy(), q.cpu().numpy()
    for b in range(B):
        _properties(tn, ids_np, sc_np, b, cfg, cfg.n_docs, cfg.k)
    oix = oracle.make_index(corp.centroids, corp.cids, corp.codes, corp.doclens, cfg.nbits, cfg.res_lo, cfg.res_hi)
    b = 41
    res = oracle.pipeline(q_np[b], oix, cfg.nprobe, cfg.n_prune, cfg.k)
    assert check_query(tn, b, res, ids_np[b], sc_np[b], cfg.k, cfg.n_prune, table=False) <= 2
    # the same batch through the paper's candidate refinement (partial scores): F' of every candidate of one query,
    # the pruned ids and the later stages against the oracle
    del taps
    gix.enable_partial()
    taps = gix.alloc_taps(B, cfg.q_len, cfg.nprobe, cfg.n_prune, table=False)
    ids, sc = gix.search(q, cfg.nprobe, cfg.n_prune, cfg.k, taps=taps, partial=True)
    assert gix.status() == 0
    tn = taps_to_numpy(taps)
    ids_np, sc_np = ids.cpu().numpy(), sc.cpu().numpy()
    b = 17
    res = oracle.pipeline(q_np[b], oix, cfg.nprobe, cfg.n_prune, cfg.k, partial=True)
    assert check_query(tn, b, res, ids_np[b], sc_np[b], cfg.k, cfg.n_prune, table=False) <= 2
