"""GPU parity of the paper's candidate refinement (partial scores F', Algorithm 2) against the oracle: F' of every
candidate and the pruned ids bit-exact, later stages by the usual rules."""
import numpy as np
import pytest
import torch

import oracle
from helpers import random_corpus, unit_rows
from parity import check_query, taps_to_numpy

pytestmark = pytest.mark.gpu


def _check(gix, oix, q, nprobe, n_prune, k, sample=None, max_diffs=0):
    B, nq, _ = q.shape
    taps = gix.alloc_taps(B, nq, nprobe, n_prune, table=False)
    ids, sc = gix.search(torch.from_numpy(q).cuda(), nprobe, n_prune, k, taps=taps, partial=True)
    assert gix.status() == 0
    tn = taps_to_numpy(taps)
    ids, sc = ids.cpu().numpy(), sc.cpu().numpy()
    for b in (range(B) if sample is None else sample):
        res = oracle.pipeline(q[b], oix, nprobe, n_prune, k, partial=True)
        assert check_query(tn, b, res, ids[b], sc[b], k, n_prune, table=False) <= max_diffs


@pytest.mark.parametrize("D,nbits,nq,K,N,nprobe,n_prune,k", [
    (32, 2, 5, 16, 80, 2, 9, 3),
    (128, 2, 32, 64, 500, 4, 60, 10),
    (128, 1, 32, 64, 500, 4, 60, 10),
    (96, 2, 64, 48, 300, 8, 40, 12),
    (96, 1, 40, 48, 300, 3, 33, 5),
    (64, 2, 100, 32, 200, 32, 64, 20),       # every list probed: F' is the full low-bit score
    (32, 2, 6, 4, 1500, 2, 50, 10),          # four long lists of ~2,500 tokens each
])
def test_partial_refinement_small_corpora(D, nbits, nq, K, N, nprobe, n_prune, k):
    import paper_2608_23553_b200 as pkg
    cent, cids, codes, doclens = random_corpus(300 + D + nq, N, K, D, nbits, len_lo=1, len_hi=60)
    oix = oracle.make_index(cent, cids, codes, doclens, nbits)
    dev = torch.device("cuda:0")
    gix = pkg.Index(torch.from_numpy(cent).to(dev), torch.from_numpy(cids).to(dev), torch.from_numpy(codes).to(dev),
                    torch.from_numpy(doclens).to(dev), nbits)
    q = np.stack([unit_rows(np.random.default_rng(b), nq, D) for b in range(3)])
    with pytest.raises(pkg.ChimeraError):                    # not enabled yet
        gix.search(torch.from_numpy(q).cuda(), nprobe, n_prune, k, partial=True)
    gix.enable_partial()
    _check(gix, oix, q, nprobe, n_prune, k)
    # the default search is unaffected by the extra lists
    ids_a, _ = gix.search(torch.from_numpy(q).cuda(), nprobe, n_prune, k)
    res = oracle.pipeline(q[0], oix, nprobe, n_prune, k)
    assert np.array_equal(np.sort(ids_a[0].cpu().numpy()), np.sort(res.ids))


@pytest.mark.parametrize("nbits", [2, 1])
def test_partial_refinement_hashed_table_equals_dense_and_oracle(nbits):
    """With enough queries per call and a corpus large enough, the (candidate, query token) maxima live in an
    open-addressing table instead of dense rows.  40 queries (on a B200) on 30,000 documents take that path; the same queries one
    at a time take the dense path; both must agree bit for bit in F' of every candidate, pruned ids and final results,
    and sampled queries must match the oracle."""
    import paper_2608_23553_b200 as pkg
    D, nq, K, N, nprobe, n_prune, k = 64, 32, 4096, 30000, 2, 300, 20
    cent, cids, codes, doclens = random_corpus(4242 + nbits, N, K, D, nbits, len_lo=1, len_hi=40)
    oix = oracle.make_index(cent, cids, codes, doclens, nbits)
    dev = torch.device("cuda:0")
    gix = pkg.Index(torch.from_numpy(cent).to(dev), torch.from_numpy(cids).to(dev), torch.from_numpy(codes).to(dev),
                    torch.from_numpy(doclens).to(dev), nbits)
    gix.enable_partial()
    # calls of up to (SM count / 4) queries keep dense rows; three more queries and the table is hashed, which shows in
    # the workspace: more queries, yet fewer bytes
    small = torch.cuda.get_device_properties(0).multi_processor_count // 4
    B = small + 3
    assert gix.workspace_bytes(B, nq, nprobe, n_prune, k) < gix.workspace_bytes(small, nq, nprobe, n_prune, k)
    q = np.stack([unit_rows(np.random.default_rng(900 + b), nq, D) for b in range(B)])
    qd = torch.from_numpy(q).cuda()
    taps = gix.alloc_taps(B, nq, nprobe, n_prune, table=False)
    ids, sc = gix.search(qd, nprobe, n_prune, k, taps=taps, partial=True)
    assert gix.status() == 0
    tn = taps_to_numpy(taps)
    ids_np, sc_np = ids.cpu().numpy(), sc.cpu().numpy()
    for b in (0, 17, B - 1):
        res = oracle.pipeline(q[b], oix, nprobe, n_prune, k, partial=True)
        assert check_query(tn, b, res, ids_np[b], sc_np[b], k, n_prune, table=False) == 0
    for b in range(B):
        t1 = gix.alloc_taps(1, nq, nprobe, n_prune, table=False)
        i1, s1 = gix.search(qd[b:b + 1].contiguous(), nprobe, n_prune, k, taps=t1, partial=True)
        n = int(t1.n_cand[0])
        assert n == int(taps.n_cand[b])
        assert torch.equal(t1.ci[0, :n], taps.ci[b, :n]) and torch.equal(t1.pruned[0], taps.pruned[b])
        assert torch.equal(i1[0], ids[b]) and torch.equal(s1[0], sc[b])


def test_partial_refinement_tiny_config_and_batch_invariance():
    import paper_2608_23553_b200 as pkg
    from synth import CONFIGS, make_corpus, make_queries
    cfg = CONFIGS["tiny"]
    corp = make_corpus(cfg)
    oix = oracle.make_index(corp.centroids, corp.cids, corp.codes, corp.doclens, cfg.nbits, cfg.res_lo, cfg.res_hi)
    gix = pkg.Index(corp.centroids.cuda(), corp.cids.cuda(), corp.codes.cuda(), corp.doclens.cuda(), cfg.nbits,
                    cfg.res_lo, cfg.res_hi)
    gix.enable_partial()
    q = make_queries(cfg).numpy()
    _check(gix, oix, q, cfg.nprobe, cfg.n_prune, cfg.k)
    qd = torch.from_numpy(q).cuda()
    ids16, sc16 = gix.search(qd, cfg.nprobe, cfg.n_prune, cfg.k, partial=True)
    ids16, sc16 = ids16.clone(), sc16.clone()
    for b in (0, 7, 15):
        i1, s1 = gix.search(qd[b:b + 1].contiguous(), cfg.nprobe, cfg.n_prune, cfg.k, partial=True)
        assert torch.equal(i1[0], ids16[b]) and torch.equal(s1[0], sc16[b])


def test_partial_refinement_mid_batch256_sampled():
    import paper_2608_23553_b200 as pkg
    from synth import CONFIGS, make_corpus, make_queries
    cfg = CONFIGS["mid"]
    dev = torch.device("cuda:0")
    corp = make_corpus(cfg, device=dev)
    q = make_queries(cfg, 256, device=dev).cpu().numpy()
    gix = pkg.Index(corp.centroids, corp.cids, corp.codes, corp.doclens, cfg.nbits, cfg.res_lo, cfg.res_hi)
    gix.enable_partial()
    oix = oracle.make_index(corp.centroids, corp.cids, corp.codes, corp.doclens, cfg.nbits, cfg.res_lo, cfg.res_hi)
    _check(gix, oix, q, cfg.nprobe, cfg.n_prune, cfg.k, sample=(0, 255), max_diffs=2)
    # few queries per call: the selection runs over several blocks per query (another code path); against the oracle,
    # and bit-identical to the same queries inside the batch of 256
    _check(gix, oix, q[254:256], cfg.nprobe, cfg.n_prune, cfg.k, max_diffs=2)
    qd = torch.from_numpy(q).cuda()
    big = gix.search(qd, cfg.nprobe, cfg.n_prune, cfg.k, partial=True)
    for lo, hi in ((0, 1), (100, 103)):
        small = gix.search(qd[lo:hi].contiguous(), cfg.nprobe, cfg.n_prune, cfg.k, partial=True)
        assert torch.equal(small[0], big[0][lo:hi]) and torch.equal(small[1], big[1][lo:hi])
    # and the same single-query search replayed from a CUDA graph (the multi-block selection clears its histograms
    # with a memset node)
    g = pkg.GraphedSearch(gix, 1, cfg.q_len, cfg.nprobe, cfg.n_prune, cfg.k, partial=True)
    for b in (0, 17):
        ids_g, sc_g = g(qd[b:b + 1])
        torch.cuda.synchronize()
        assert torch.equal(ids_g, big[0][b:b + 1]) and torch.equal(sc_g, big[1][b:b + 1])


def test_partial_and_rabitq_edge_cases():
    """Few candidates (k_refine and k larger than the candidate set), and a candidate capacity that overflows."""
    import paper_2608_23553_b200 as pkg
    from synth import CONFIGS, encode_rabitq_1bit, random_rotation
    D, K, N = 32, 16, 40
    cent, cids, codes, doclens = random_corpus(77, N, K, D, 2, len_lo=1, len_hi=4)
    rng = np.random.default_rng(78)
    raw = unit_rows(rng, len(cids), D)
    P = random_rotation(CONFIGS["tiny"].replace(dim=D, seed=9))
    bits, inv = encode_rabitq_1bit(torch.from_numpy(raw), P)
    oix = oracle.make_index(cent, cids, codes, doclens, 2)
    rq = oracle.make_rabitq(P, bits, inv)
    dev = torch.device("cuda:0")
    gix = pkg.Index(torch.from_numpy(cent).to(dev), torch.from_numpy(cids).to(dev), torch.from_numpy(codes).to(dev),
                    torch.from_numpy(doclens).to(dev), 2)
    gix.attach_rabitq(P.to(dev), bits.to(dev), inv.to(dev))          # also builds the token lists
    q = unit_rows(rng, 4, D)[None]
    qd = torch.from_numpy(q).cuda()
    for kw, ref in (({"partial": True}, lambda: oracle.pipeline(q[0], oix, 1, 100, 200, partial=True)),
                    ({"rabitq": True}, lambda: oracle.pipeline_rabitq(q[0], oix, rq, 1, 100, 200))):
        ids, sc = gix.search(qd, 1, 100, 200, **kw)
        assert gix.status() == 0
        res = ref()
        n = int((res.ids >= 0).sum())
        assert n < 100 and np.array_equal(ids[0].cpu().numpy(), res.ids)
        assert np.all(np.isneginf(sc[0, n:].cpu().numpy()))
        gix.search(qd, 8, 10, 5, max_candidates=4, **kw)             # more candidates than the capacity
        assert gix.status() == 4
        gix.search(qd, 8, 10, 5, **kw)
        assert gix.status() == 0
