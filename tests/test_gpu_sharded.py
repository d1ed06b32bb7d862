"""Document-sharded search (Sec. 3.3 scaling sketch) on one GPU: the shards' phases run one after the other in one
process and the all-gathers are stacks, so no kernel waits on another.  The merged result must equal the unsharded
search of the same library bit for bit (ids and float scores), and the oracle's by the usual rules."""
import numpy as np
import pytest
import torch

import oracle
from helpers import random_corpus, unit_rows
from parity import check_topk

pytestmark = pytest.mark.gpu


def _slice_corpus(cids, codes, doclens, lo, hi, extra=()):
    off = np.concatenate([[0], np.cumsum(doclens, dtype=np.int64)])
    t0, t1 = int(off[lo]), int(off[hi])
    return (cids[t0:t1], codes[t0:t1], doclens[lo:hi]) + tuple(e[t0:t1] for e in extra)


def _emulate(engines, q, nprobe, n_prune, k):
    """All ranks in lockstep; torch.stack stands in for the rank-ordered all-gather."""
    from paper_2608_23553_b200.sharded import ShardedSearcher
    local = [e.local_phase(q, nprobe, n_prune, k) for e in engines]
    for e in engines:
        e.check()
    all_ids = torch.stack([l[0] for l in local]).contiguous()
    all_sc3 = torch.stack([l[1] for l in local]).contiguous()
    tops = [e.finish_phase(q, nprobe, n_prune, k, all_ids, all_sc3) for e in engines]
    top_ids = torch.stack([t[0] for t in tops]).contiguous()
    top_sc = torch.stack([t[1] for t in tops]).contiguous()
    merged = [e.merge_phase(top_ids, top_sc) for e in engines]
    for m in merged[1:]:                                  # every rank ends with the same answer
        assert torch.equal(m[0], merged[0][0]) and torch.equal(m[1], merged[0][1])
    # the searcher's own sequencing on rank 0, fed by the other ranks' tensors
    # (the fifth exchange carries every rank's device status word, so that a failure is raised on all ranks together)
    feeds = iter([all_ids, all_sc3, top_ids, top_sc, torch.stack([e.status_word() for e in engines])])
    s = ShardedSearcher(engines[0], gather=lambda t: next(feeds))
    ids0, sc0 = s.search(q, nprobe, n_prune, k)
    assert torch.equal(ids0, merged[0][0]) and torch.equal(sc0, merged[0][1])
    return merged[0]


@pytest.mark.parametrize("mode", ["ci", "partial", "rabitq"])
@pytest.mark.parametrize("world,D,nbits,nq,K,N,nprobe,n_prune,k", [
    (2, 128, 2, 32, 64, 600, 4, 50, 10),
    (3, 128, 2, 32, 64, 601, 2, 300, 20),        # a shard holds fewer candidates than n_prune
    (3, 96, 1, 64, 48, 400, 8, 40, 12),
    (4, 64, 2, 20, 32, 200, 32, 64, 100),        # k > n_prune: padded lists are merged
    (1, 128, 2, 32, 64, 300, 4, 50, 10),         # a single shard is the plain search
])
def test_sharded_equals_unsharded(mode, world, D, nbits, nq, K, N, nprobe, n_prune, k):
    import paper_2608_23553_b200 as pkg
    from paper_2608_23553_b200.sharded import ShardEngine, shard_ranges
    from synth import CONFIGS, encode_rabitq_1bit, random_rotation
    if mode == "rabitq" and nbits != 2:
        pytest.skip("the RaBitQ tests index 2-bit residual codes beside the 1-bit codes")
    cent, cids, codes, doclens = random_corpus(900 + D + nq + world, N, K, D, nbits, len_lo=1, len_hi=40)
    dev = torch.device("cuda:0")
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)          # noqa: E731
    extra, P = (), None
    if mode == "rabitq":
        raw = unit_rows(np.random.default_rng(D + nq), len(cids), D)
        P = random_rotation(CONFIGS["tiny"].replace(dim=D, seed=3))
        bits, inv = encode_rabitq_1bit(torch.from_numpy(raw), P)
        extra = (bits.numpy(), inv.numpy())

    def build(c, co, dl, ex):
        ix = pkg.Index(t(cent), t(c), t(co), t(dl), nbits)
        if mode == "partial":
            ix.enable_partial()
        if mode == "rabitq":
            ix.attach_rabitq(P.to(dev) if torch.is_tensor(P) else t(P), t(ex[0]), t(ex[1]))
        return ix

    full = build(cids, codes, doclens, extra)
    engines = []
    for lo, hi in shard_ranges(N, world):
        sl = _slice_corpus(cids, codes, doclens, lo, hi, extra)
        engines.append(ShardEngine(build(sl[0], sl[1], sl[2], sl[3:]), lo, mode))
    q = torch.from_numpy(np.stack([unit_rows(np.random.default_rng(b), nq, D) for b in range(5)])).to(dev)
    kw = {"partial": mode == "partial", "rabitq": mode == "rabitq"}
    ref_ids, ref_sc = full.search(q, nprobe, n_prune, k, **kw)
    assert full.status() == 0
    ids, sc = _emulate(engines, q, nprobe, n_prune, k)
    assert torch.equal(ids, ref_ids), "sharded ids differ from the single index"
    assert torch.equal(sc, ref_sc), "sharded scores differ from the single index"
    if mode == "ci":                                       # and against the oracle on the whole corpus
        oix = oracle.make_index(cent, cids, codes, doclens, nbits)
        for b in range(q.shape[0]):
            res = oracle.pipeline(q[b].cpu().numpy(), oix, nprobe, n_prune, k)
            check_topk(ids[b].cpu().numpy(), sc[b].cpu().numpy(), res, k, nq)


def test_sharded_tiny_config_three_shards():
    import paper_2608_23553_b200 as pkg
    from paper_2608_23553_b200.sharded import ShardEngine, shard_ranges
    from synth import CONFIGS, make_corpus, make_queries
    cfg = CONFIGS["tiny"]
    corp = make_corpus(cfg)
    cids, codes, doclens = corp.cids.numpy(), corp.codes.numpy(), corp.doclens.numpy()
    dev = torch.device("cuda:0")
    full = pkg.Index(corp.centroids.to(dev), corp.cids.to(dev), corp.codes.to(dev), corp.doclens.to(dev), cfg.nbits,
                     cfg.res_lo, cfg.res_hi)
    engines = []
    for lo, hi in shard_ranges(cfg.n_docs, 3):
        c, co, dl = _slice_corpus(cids, codes, doclens, lo, hi)
        ix = pkg.Index(corp.centroids.to(dev), torch.from_numpy(c).to(dev), torch.from_numpy(co).to(dev),
                       torch.from_numpy(dl).to(dev), cfg.nbits, cfg.res_lo, cfg.res_hi)
        engines.append(ShardEngine(ix, lo, "ci"))
    q = make_queries(cfg).to(dev)
    ref_ids, ref_sc = full.search(q, cfg.nprobe, cfg.n_prune, cfg.k)
    ids, sc = _emulate(engines, q, cfg.nprobe, cfg.n_prune, cfg.k)
    assert torch.equal(ids, ref_ids) and torch.equal(sc, ref_sc)


def test_merge_rejects_oversized_lists():
    import paper_2608_23553_b200 as pkg
    from paper_2608_23553_b200.sharded import ShardEngine
    dev = torch.device("cuda:0")
    ids = torch.zeros(4, 1, 8192, dtype=torch.int32, device=dev)
    sc = torch.zeros(4, 1, 8192, dtype=torch.float32, device=dev)
    with pytest.raises(pkg.ChimeraError):
        ShardEngine.merge_phase(None, ids, sc)
