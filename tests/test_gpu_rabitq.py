"""GPU parity of the paper's pipeline on RaBitQ 1-bit codes (rotation, partial 1-bit refinement, complete 1-bit
document scores) against the oracle: every value, float scores included, bit for bit (the arithmetic is fixed: integer
contractions, two fp32 multiplications, sums over query tokens in increasing order)."""
import numpy as np
import pytest
import torch

import oracle
from helpers import random_corpus, unit_rows

pytestmark = pytest.mark.gpu


def _run(gix, oix, rq, q, nprobe, k_refine, k, sample=None):
    B, nq, _ = q.shape
    taps = gix.alloc_taps(B, nq, nprobe, k_refine, table=False)
    ids, sc = gix.search(torch.from_numpy(q).cuda(), nprobe, k_refine, k, taps=taps, rabitq=True)
    assert gix.status() == 0
    ids, sc = ids.cpu().numpy(), sc.cpu().numpy()
    for b in (range(B) if sample is None else sample):
        res = oracle.pipeline_rabitq(q[b], oix, rq, nprobe, k_refine, k)
        n = int(taps.n_cand[b])
        assert n == len(res.cand) and np.array_equal(taps.cand[b, :n].cpu().numpy(), res.cand)
        assert np.array_equal(taps.ci[b, :n].cpu().numpy(), res.ci.view(np.int32)), "partial 1-bit scores differ"
        m = int(taps.n_pruned[b])
        assert np.array_equal(taps.pruned[b, :m].cpu().numpy(), res.pruned)
        assert np.array_equal(taps.score4[b, :m].cpu().numpy(), res.score4), "complete 1-bit scores differ"
        assert np.array_equal(ids[b], res.ids) and np.array_equal(sc[b], res.scores)


@pytest.mark.parametrize("D,nq,K,N,nprobe,k_refine,k", [
    (32, 5, 16, 80, 2, 9, 3),
    (128, 32, 64, 500, 4, 60, 10),
    (96, 64, 48, 300, 8, 40, 12),
    (64, 40, 32, 200, 32, 200, 20),          # every list probed, nothing pruned: complete scores of every document
])
def test_rabitq_pipeline_small_corpora(D, nq, K, N, nprobe, k_refine, k):
    import paper_2608_23553_b200 as pkg
    from synth import CONFIGS, encode_rabitq_1bit, random_rotation
    cent, cids, codes, doclens = random_corpus(500 + D + nq, N, K, D, 2, len_lo=1, len_hi=60)
    rng = np.random.default_rng(D + nq)
    raw = unit_rows(rng, len(cids), D)
    P = random_rotation(CONFIGS["tiny"].replace(dim=D, seed=3))
    bits, inv = encode_rabitq_1bit(torch.from_numpy(raw), P)
    oix = oracle.make_index(cent, cids, codes, doclens, 2)
    rq = oracle.make_rabitq(P, bits, inv)
    dev = torch.device("cuda:0")
    gix = pkg.Index(torch.from_numpy(cent).to(dev), torch.from_numpy(cids).to(dev), torch.from_numpy(codes).to(dev),
                    torch.from_numpy(doclens).to(dev), 2)
    q = np.stack([unit_rows(np.random.default_rng(b), nq, D) for b in range(3)])
    with pytest.raises(pkg.ChimeraError):
        gix.search(torch.from_numpy(q).cuda(), nprobe, k_refine, k, rabitq=True)
    gix.attach_rabitq(P.to(dev), bits.to(dev), inv.to(dev))
    _run(gix, oix, rq, q, nprobe, k_refine, k)


def test_rabitq_pipeline_tiny_config():
    import paper_2608_23553_b200 as pkg
    from synth import CONFIGS, make_corpus, make_queries
    cfg = CONFIGS["tiny"]
    corp = make_corpus(cfg, rabitq=True)
    oix = oracle.make_index(corp.centroids, corp.cids, corp.codes, corp.doclens, cfg.nbits, cfg.res_lo, cfg.res_hi)
    rq = oracle.make_rabitq(corp.rotation, corp.rq_bits, corp.rq_inv_dot)
    gix = pkg.Index(corp.centroids.cuda(), corp.cids.cuda(), corp.codes.cuda(), corp.doclens.cuda(), cfg.nbits,
                    cfg.res_lo, cfg.res_hi)
    gix.attach_rabitq(corp.rotation.cuda(), corp.rq_bits.cuda(), corp.rq_inv_dot.cuda())
    q = make_queries(cfg).numpy()
    _run(gix, oix, rq, q, cfg.nprobe, cfg.n_prune, cfg.k)


def test_rabitq_pipeline_mid_batch256_sampled():
    import paper_2608_23553_b200 as pkg
    from synth import CONFIGS, make_corpus, make_queries
    cfg = CONFIGS["mid"]
    dev = torch.device("cuda:0")
    corp = make_corpus(cfg, device=dev, rabitq=True)
    q = make_queries(cfg, 256, device=dev).cpu().numpy()
    gix = pkg.Index(corp.centroids, corp.cids, corp.codes, corp.doclens, cfg.nbits, cfg.res_lo, cfg.res_hi)
    gix.attach_rabitq(corp.rotation, corp.rq_bits, corp.rq_inv_dot)
    oix = oracle.make_index(corp.centroids, corp.cids, corp.codes, corp.doclens, cfg.nbits, cfg.res_lo, cfg.res_hi)
    rq = oracle.make_rabitq(corp.rotation, corp.rq_bits, corp.rq_inv_dot)
    _run(gix, oix, rq, q, cfg.nprobe, cfg.n_prune, cfg.k, sample=(0, 255))
    # few queries per call: the selection runs over several blocks per query (another code path)
    _run(gix, oix, rq, q[254:256], cfg.nprobe, cfg.n_prune, cfg.k)
    qd = torch.from_numpy(q).cuda()
    big = gix.search(qd, cfg.nprobe, cfg.n_prune, cfg.k, rabitq=True)
    small = gix.search(qd[7:10].contiguous(), cfg.nprobe, cfg.n_prune, cfg.k, rabitq=True)
    assert torch.equal(small[0], big[0][7:10]) and torch.equal(small[1], big[1][7:10])
