"""Parity at the benchmark's full size and launch configuration: the Mid corpus (500k documents, ~60M tokens,
65,536 centroids), batch 256, nprobe 4, n_prune 1024, k 10 -- sampled queries checked stage by stage against the
oracle, every query checked for the properties that hold at any size."""
import numpy as np
import pytest
import torch

import oracle
from parity import check_query, taps_to_numpy

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mid():
    import paper_2608_23553_b200 as pkg
    from synth import CONFIGS, make_corpus, make_queries
    cfg = CONFIGS["mid"]
    dev = torch.device("cuda:0")
    corp = make_corpus(cfg, device=dev)
    q = make_queries(cfg, device=dev)
    gix = pkg.Index(corp.centroids, corp.cids, corp.codes, corp.doclens, cfg.nbits, cfg.res_lo, cfg.res_hi)
    oix = oracle.make_index(corp.centroids, corp.cids, corp.codes, corp.doclens, cfg.nbits, cfg.res_lo, cfg.res_hi)
    return cfg, corp, gix, oix, q


def test_mid_batch256_sampled_queries_match_oracle_and_all_queries_are_valid(mid):
    cfg, corp, gix, oix, q = mid
    B = 256
    qb = q[:B].contiguous()
    taps = gix.alloc_taps(B, cfg.q_len, cfg.nprobe, cfg.n_prune, table=False)
    ids, sc = gix.search(qb, cfg.nprobe, cfg.n_prune, cfg.k, taps=taps)
    assert gix.status() == 0
    tn = taps_to_numpy(taps)
    ids_np, sc_np = ids.cpu().numpy(), sc.cpu().numpy()
    q_np = qb.cpu().numpy()
    # sampled queries: every stage against the oracle (first, last and one in the middle of the batch)
    for b in (0, 131, 255):
        res = oracle.pipeline(q_np[b], oix, cfg.nprobe, cfg.n_prune, cfg.k)
        assert check_query(tn, b, res, ids_np[b], sc_np[b], cfg.k, cfg.n_prune, table=False) == 0
    # every query: properties that hold at any size
    assert np.all(tn["n_pruned"] == cfg.n_prune)
    for b in range(B):
        n = int(tn["n_cand"][b])
        cand = tn["cand"][b, :n]
        assert n > cfg.n_prune and np.all(np.diff(cand) > 0) and cand[0] >= 0 and cand[-1] < oix.N
        pruned = tn["pruned"][b]
        assert np.all(np.diff(pruned) > 0) and np.all(np.isin(pruned, cand))
        # the kept documents are exactly those with the largest (CI, -id)
        ci = tn["ci"][b, :n]
        order = np.lexsort((cand, -ci.astype(np.int64)))[:cfg.n_prune]
        assert np.array_equal(np.sort(cand[order]), pruned)
        assert np.all(np.isin(ids_np[b], pruned)) and np.all(np.diff(sc_np[b]) <= 0)
        pos = np.searchsorted(pruned, ids_np[b])
        assert np.array_equal(tn["score4"][b][pos], sc_np[b])
        best = np.lexsort((pruned, -tn["score4"][b].astype(np.float64)))[:cfg.k]
        assert np.array_equal(pruned[best], ids_np[b])
    # a batch equals the same queries one by one
    for b in (3, 200):
        i1, s1 = gix.search(qb[b:b + 1].contiguous(), cfg.nprobe, cfg.n_prune, cfg.k)
        assert torch.equal(i1[0], ids[b]) and torch.equal(s1[0], sc[b])


def test_mid_score_table_sampled_rows_match_oracle(mid):
    cfg, corp, gix, oix, q = mid
    B = 2
    taps = gix.alloc_taps(B, cfg.q_len, cfg.nprobe, cfg.n_prune, table=True)
    gix.run_stages(1, 1, q[5:7].contiguous(), B, cfg.q_len, cfg.nprobe, cfg.n_prune, cfg.k, taps)
    S = oracle.score_table(q[5].cpu().numpy(), oix.centroids)
    assert np.array_equal(taps.score_table[0].cpu().numpy(), S)


def test_mid_score_table_in_the_batch256_launch_matches_oracle(mid):
    """Stage 1 in the configuration the benchmark times (256 queries per call: the 48-row query tiles straddle query
    boundaries and the grid is split over query tiles): every entry of the tables of eight queries spread over the
    batch, 8 x 32 query tokens x 65,536 centroids."""
    cfg, corp, gix, oix, q = mid
    B = 256
    taps = gix.alloc_taps(B, cfg.q_len, cfg.nprobe, cfg.n_prune, max_candidates=1024, table=True, ci=False)
    gix.run_stages(1, 1, q[:B].contiguous(), B, cfg.q_len, cfg.nprobe, cfg.n_prune, cfg.k, taps, max_candidates=1024)
    q_np = q[:B].cpu().numpy()
    for b in (0, 1, 2, 37, 100, 191, 254, 255):
        S = oracle.score_table(q_np[b], oix.centroids)
        assert np.array_equal(taps.score_table[b].cpu().numpy(), S), "query %d" % b
    del taps
    torch.cuda.empty_cache()


def test_mid_batch256_four_document_shards_equal_the_single_index(mid):
    """The document-sharded search at the benchmark's size: four shards of 125k documents, their phases run one after
    the other on this GPU, merged ids and scores equal the single index's for every query."""
    import paper_2608_23553_b200 as pkg
    from paper_2608_23553_b200.sharded import ShardEngine, shard_ranges
    cfg, corp, gix, oix, q = mid
    qb = q[:256].contiguous()
    ref_ids, ref_sc = gix.search(qb, cfg.nprobe, cfg.n_prune, cfg.k)
    off = torch.cat([torch.zeros(1, dtype=torch.int64, device=qb.device), torch.cumsum(corp.doclens.to(torch.int64), 0)])
    engines = []
    for lo, hi in shard_ranges(cfg.n_docs, 4):
        t0, t1 = int(off[lo]), int(off[hi])
        ix = pkg.Index(corp.centroids, corp.cids[t0:t1].contiguous(), corp.codes[t0:t1].contiguous(),
                       corp.doclens[lo:hi].contiguous(), cfg.nbits, cfg.res_lo, cfg.res_hi)
        engines.append(ShardEngine(ix, lo, "ci"))
    local = [e.local_phase(qb, cfg.nprobe, cfg.n_prune, cfg.k) for e in engines]
    for e in engines:
        e.check()
    all_ids = torch.stack([l[0] for l in local]).contiguous()
    all_sc3 = torch.stack([l[1] for l in local]).contiguous()
    tops = [e.finish_phase(qb, cfg.nprobe, cfg.n_prune, cfg.k, all_ids, all_sc3) for e in engines]
    ids, sc = engines[0].merge_phase(torch.stack([t[0] for t in tops]).contiguous(),
                                     torch.stack([t[1] for t in tops]).contiguous())
    assert torch.equal(ids, ref_ids) and torch.equal(sc, ref_sc)


def test_sweep_ground_truth_scorer_on_a_20k_document_slice_matches_oracle(mid):
    """bench.brute_force_maxsim (the recall sweeps' ground truth, independent of the library) on the first 20,000
    documents of the Mid corpus against the oracle's exhaustive scores, two queries."""
    import bench
    cfg, corp, gix, oix, q = mid
    n = 20_000
    T = int(corp.doclens[:n].to(torch.int64).sum())
    sc = bench.brute_force_maxsim(corp.centroids, corp.cids[:T], corp.codes[:T], corp.doclens[:n], cfg.nbits,
                                  cfg.res_lo, cfg.res_hi, q[:3].contiguous()).cpu().numpy()
    q_np = q[:3].cpu().numpy()
    docs = np.arange(n, dtype=np.int32)
    for b in (0, 2):
        ref = oracle.score_docs(q_np[b], docs, oix)
        assert np.abs(sc[b] - ref).max() <= 1e-5 * max(1.0, float(np.abs(ref).max()))
