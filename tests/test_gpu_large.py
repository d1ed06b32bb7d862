"""Parity on the passage-corpus-shaped Large corpus at full size (8.8M documents, ~600M tokens, 262,144 centroids), in
the launch configurations the benchmark and its sweep time: batch 256 at the config's parameters; the sweep's extreme
point (nprobe 32, n_prune 16384, k 1000: ~2M candidates per query, the selection and the top-k at the API's maxima);
and the two paper pipelines (partial-score refinement, RaBitQ 1-bit codes).  Sampled queries are compared with the
oracle stage by stage; every query is checked for the properties that hold at any size."""
import numpy as np
import pytest
import torch

import oracle
from parity import check_query

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def large():
    import psutil
    import paper_2608_23553_b200 as pkg
    from synth import CONFIGS, make_corpus, make_queries
    if psutil.virtual_memory().available < 48e9:
        pytest.skip("needs ~25 GB of host memory for the oracle's copy of the corpus")
    free, _ = torch.cuda.mem_get_info()
    if free < 120e9:
        pytest.skip("needs ~100 GB of device memory")
    cfg = CONFIGS["large"]
    dev = torch.device("cuda:0")
    corp = make_corpus(cfg, device=dev)
    assert abs(corp.doclens.float().mean().item() - 68.0) < 0.3 and 5.9e8 < corp.n_tokens < 6.1e8
    q = make_queries(cfg, 256, device=dev)
    gix = pkg.Index(corp.centroids, corp.cids, corp.codes, corp.doclens, cfg.nbits, cfg.res_lo, cfg.res_hi)
    oix = oracle.make_index(corp.centroids, corp.cids, corp.codes, corp.doclens, cfg.nbits, cfg.res_lo, cfg.res_hi)
    yield cfg, corp, gix, oix, q
    gix.close()


def _rows(taps, rows, table=None):
    """Host copies of the sampled rows of the taps (the full [256, max_candidates] arrays are gigabytes)."""
    out = {}
    for name in ("probes", "cand", "n_cand", "ci", "pruned", "n_pruned", "score4"):
        t = getattr(taps, name)
        if t is not None:
            out[name] = t[list(rows)].cpu().numpy()
    return out


def _properties(taps, ids, sc, n_prune, k, N):
    """What holds at any size, for every query of the batch, on the device (no bulk copies)."""
    n_cand = taps.n_cand.to(torch.int64)
    maxc = taps.cand.shape[1]
    inside = torch.arange(maxc, device=ids.device)[None, :] < n_cand[:, None]
    cand = taps.cand.to(torch.int64)
    assert bool(((cand[:, 1:] > cand[:, :-1]) | ~inside[:, 1:]).all())              # ascending, no duplicates
    assert bool(((cand >= 0) & (cand < N) | ~inside).all())
    m = taps.n_pruned.to(torch.int64)
    assert torch.equal(m, torch.clamp(n_cand, max=n_prune))
    pruned = taps.pruned.to(torch.int64)
    valid = torch.arange(n_prune, device=ids.device)[None, :] < m[:, None]
    assert bool(((pruned[:, 1:] > pruned[:, :-1]) | ~valid[:, 1:]).all())
    assert bool((pruned[~valid] == -1).all())
    for b in range(ids.shape[0]):                                                    # survivors are candidates
        pb = pruned[b, :int(m[b])]
        cb = cand[b, :int(n_cand[b])]
        pos = torch.searchsorted(cb, pb).clamp_(max=cb.numel() - 1)
        assert torch.equal(cb[pos], pb)
        # the result is the best k of the survivors by (score descending, id ascending)
        s4 = taps.score4[b, :int(m[b])].double()
        order = np.lexsort((pb.cpu().numpy(), -s4.cpu().numpy()))[:k]
        got = ids[b][ids[b] >= 0].to(torch.int64).cpu().numpy()
        assert np.array_equal(pb.cpu().numpy()[order], got)
    assert bool((sc[:, 1:] <= sc[:, :-1]).all())


def test_large_corpus_full_size_sampled_queries(large):
    cfg, corp, gix, oix, q = large
    B, maxc = 256, 512 * 1024
    taps = gix.alloc_taps(B, cfg.q_len, cfg.nprobe, cfg.n_prune, max_candidates=maxc, table=False)
    ids, sc = gix.search(q, cfg.nprobe, cfg.n_prune, cfg.k, max_candidates=maxc, taps=taps)
    assert gix.status() == 0
    _properties(taps, ids, sc, cfg.n_prune, cfg.k, cfg.n_docs)
    sample = (77, 255)
    tn = _rows(taps, sample)
    ids_np, sc_np, q_np = ids.cpu().numpy(), sc.cpu().numpy(), q.cpu().numpy()
    # stage 1 for the two sampled queries, on its own: 64 query tokens x all 262,144 centroids
    t1 = gix.alloc_taps(2, cfg.q_len, cfg.nprobe, cfg.n_prune, max_candidates=1024, table=True)
    q2 = torch.stack([q[77], q[255]]).contiguous()
    gix.run_stages(1, 1, q2, 2, cfg.q_len, cfg.nprobe, cfg.n_prune, cfg.k, t1, max_candidates=1024)
    tables = t1.score_table.cpu().numpy()
    for j, b in enumerate(sample):
        res = oracle.pipeline(q_np[b], oix, cfg.nprobe, cfg.n_prune, cfg.k)
        assert np.array_equal(tables[j], res.S)
        # check_query enforces the tolerance rule; with k = 100 a swap between two fp32 near-ties can move positions
        assert check_query(tn, j, res, ids_np[b], sc_np[b], cfg.k, cfg.n_prune, table=False) <= 4


def test_sweep_ground_truth_scorer_on_a_10k_document_sample_matches_oracle(large):
    """bench.brute_force_maxsim (the recall sweeps' ground truth, independent of the library) on 10,000 documents drawn
    from the whole Large corpus against the oracle's exhaustive scores of the same documents, two queries."""
    import bench
    cfg, corp, gix, oix, q = large
    dev = q.device
    g = torch.Generator(device="cpu")
    g.manual_seed(5)
    docs = torch.sort(torch.randperm(cfg.n_docs, generator=g)[:10_000]).values
    off = torch.from_numpy(oix.doc_off)
    tok = torch.cat([torch.arange(int(off[d]), int(off[d + 1])) for d in docs.tolist()]).to(dev)
    sc = bench.brute_force_maxsim(corp.centroids, corp.cids[tok], corp.codes[tok], corp.doclens[docs.to(dev)],
                                  cfg.nbits, cfg.res_lo, cfg.res_hi, q[:2].contiguous()).cpu().numpy()
    q_np = q[:2].cpu().numpy()
    for b in range(2):
        ref = oracle.score_docs(q_np[b], docs.numpy().astype(np.int32), oix)
        assert np.abs(sc[b] - ref).max() <= 1e-5 * max(1.0, float(np.abs(ref).max()))


def test_large_sweep_extreme_point_nprobe32_nprune16384_k1000(large):
    """The recall sweep's largest point in its launch shape: 256 queries per call, nprobe 32 (about two million
    candidates per query, capacity as the benchmark sizes it), n_prune 16384 (a real selection at the API's maximum),
    k 1000 (the 16,384-key sorting network of stage 5)."""
    import bench
    cfg, corp, gix, oix, q = large
    B, P, n_prune, k = 256, 32, 16384, 1000
    maxc = bench.candidate_capacity(gix, q, cfg.q_len, P, n_prune, k)
    assert 16384 < maxc < cfg.n_docs
    taps = gix.alloc_taps(B, cfg.q_len, P, n_prune, max_candidates=maxc, table=False)
    ids, sc = gix.search(q, P, n_prune, k, max_candidates=maxc, taps=taps)
    assert gix.status() == 0
    assert int(taps.n_cand.min()) > n_prune
    _properties(taps, ids, sc, n_prune, k, cfg.n_docs)
    b = 201
    tn = _rows(taps, (b,))
    del taps
    torch.cuda.empty_cache()
    res = oracle.pipeline(q[b].cpu().numpy(), oix, P, n_prune, k)
    # k = 1000 of 16,384 survivors: a few fp32 near-ties may swap positions (the rule inside check_query bounds them)
    assert check_query(tn, 0, res, ids[b].cpu().numpy(), sc[b].cpu().numpy(), k, n_prune, table=False) <= 16


def test_large_partial_score_refinement_sampled_query(large):
    cfg, corp, gix, oix, q = large
    gix.enable_partial()
    B, maxc = 256, 512 * 1024
    taps = gix.alloc_taps(B, cfg.q_len, cfg.nprobe, cfg.n_prune, max_candidates=maxc, table=False)
    ids, sc = gix.search(q, cfg.nprobe, cfg.n_prune, cfg.k, max_candidates=maxc, taps=taps, partial=True)
    assert gix.status() == 0
    _properties(taps, ids, sc, cfg.n_prune, cfg.k, cfg.n_docs)
    b = 123
    tn = _rows(taps, (b,))
    del taps
    torch.cuda.empty_cache()
    res = oracle.pipeline(q[b].cpu().numpy(), oix, cfg.nprobe, cfg.n_prune, cfg.k, partial=True)
    assert check_query(tn, 0, res, ids[b].cpu().numpy(), sc[b].cpu().numpy(), cfg.k, cfg.n_prune, table=False) <= 4


def test_large_rabitq_pipeline_sampled_query(large):
    """The paper's pipeline on RaBitQ 1-bit codes at full size, batch 256: one sampled query bit for bit (partial 1-bit
    scores of every candidate, pruned ids, complete 1-bit scores, final ids and scores)."""
    import psutil
    from synth import make_corpus
    cfg, corp, gix, oix, q = large
    if psutil.virtual_memory().available < 24e9:
        pytest.skip("needs ~12 GB more host memory for the oracle's copy of the 1-bit codes")
    dev = q.device
    again = make_corpus(cfg, device=dev, rabitq=True)           # same seeds: the same tokens, now with their 1-bit codes
    assert torch.equal(again.cids[:1 << 20], corp.cids[:1 << 20])
    rot, bits, inv = again.rotation, again.rq_bits, again.rq_inv_dot
    del again
    torch.cuda.empty_cache()
    gix.attach_rabitq(rot, bits, inv)
    rq = oracle.make_rabitq(rot, bits, inv)
    B, maxc = 256, 512 * 1024
    taps = gix.alloc_taps(B, cfg.q_len, cfg.nprobe, cfg.n_prune, max_candidates=maxc, table=False)
    ids, sc = gix.search(q, cfg.nprobe, cfg.n_prune, cfg.k, max_candidates=maxc, taps=taps, rabitq=True)
    assert gix.status() == 0
    b = 64
    res = oracle.pipeline_rabitq(q[b].cpu().numpy(), oix, rq, cfg.nprobe, cfg.n_prune, cfg.k)
    n = int(taps.n_cand[b])
    assert n == len(res.cand) and np.array_equal(taps.cand[b, :n].cpu().numpy(), res.cand)
    assert np.array_equal(taps.ci[b, :n].cpu().numpy(), res.ci.view(np.int32)), "partial 1-bit scores differ"
    m = int(taps.n_pruned[b])
    assert np.array_equal(taps.pruned[b, :m].cpu().numpy(), res.pruned)
    assert np.array_equal(taps.score4[b, :m].cpu().numpy(), res.score4), "complete 1-bit scores differ"
    assert np.array_equal(ids[b].cpu().numpy(), res.ids) and np.array_equal(sc[b].cpu().numpy(), res.scores)
