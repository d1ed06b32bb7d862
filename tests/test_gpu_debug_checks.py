"""Checks that only the debug build of the library (libchimera_debug.so, loaded with CHIMERA_DEBUG_LIB=1) can make:
guard regions between workspace regions stay intact through every pipeline, a damaged guard is found, and an index out
of range is reported and not dereferenced.  tests/test_gpu_debug_build.py runs this file (and the parity and fuzz
tests) in a process that loads the debug build; in an ordinary run these tests skip."""
import numpy as np
import pytest
import torch

import oracle
from parity import check_query, taps_to_numpy

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dbg():
    import paper_2608_23553_b200 as pkg
    if pkg.lib().chimera_is_debug_build() != 1:
        pytest.skip("needs the debug build (CHIMERA_DEBUG_LIB=1)")
    from synth import CONFIGS, make_corpus, make_queries
    cfg = CONFIGS["tiny"].replace(n_docs=1500, n_centroids=256, n_queries=4)       # 1500 is not a multiple of 32
    corp = make_corpus(cfg, rabitq=True)
    q = make_queries(cfg)
    dev = torch.device("cuda:0")
    gix = pkg.Index(corp.centroids.to(dev), corp.cids.to(dev), corp.codes.to(dev), corp.doclens.to(dev), cfg.nbits,
                    cfg.res_lo, cfg.res_hi)
    gix.attach_rabitq(corp.rotation.to(dev), corp.rq_bits.to(dev), corp.rq_inv_dot.to(dev))
    oix = oracle.make_index(corp.centroids, corp.cids, corp.codes, corp.doclens, cfg.nbits, cfg.res_lo, cfg.res_hi)
    return pkg, cfg, gix, oix, q


def test_guard_regions_stay_intact_through_every_pipeline_and_damage_is_found(dbg):
    pkg, cfg, gix, oix, q = dbg
    qd = q.cuda()
    B, nq, P, n_prune, k = q.shape[0], cfg.q_len, cfg.nprobe, 64, cfg.k
    for kw in ({}, {"partial": True}, {"rabitq": True}):
        taps = gix.alloc_taps(B, nq, P, n_prune)
        gix.search(qd, P, n_prune, k, taps=taps, **kw)
        assert gix.status() == 0
        assert gix.workspace_check(B, nq, P, n_prune, k) == -1
    # damage the last guard region (the last 256 bytes of the workspace) from the host side: it must be found
    nbytes = gix.workspace_bytes(B, nq, P, n_prune, k)
    gix._ws[nbytes - 7] = 0
    torch.cuda.synchronize()
    bad = gix.workspace_check(B, nq, P, n_prune, k)
    assert bad >= 0
    gix.search(qd, P, n_prune, k)                      # the next search rewrites the patterns
    assert gix.workspace_check(B, nq, P, n_prune, k) == -1


def test_an_out_of_range_document_id_is_reported_and_not_dereferenced(dbg):
    pkg, cfg, gix, oix, q = dbg
    qd = q.cuda()
    B, nq, P, n_prune, k = q.shape[0], cfg.q_len, cfg.nprobe, 64, cfg.k
    taps = gix.alloc_taps(B, nq, P, n_prune)
    gix.search(qd, P, n_prune, k, taps=taps)
    assert gix.status() == 0
    # stage 3 onwards from a candidate list whose last entry is the first id past the corpus (N itself: even an
    # unchecked access would stay inside the arrays' allocations; the debug build must not make it at all)
    n0 = int(taps.n_cand[0])
    taps.cand[0, n0 - 1] = oix.N
    gix.run_stages(3, 5, qd, B, nq, P, n_prune, k, taps)
    assert gix.status() == 7                           # CHIMERA_DEBUG_CHECK_FAILED
    # and the library is fine afterwards: an ordinary search equals the oracle
    taps = gix.alloc_taps(B, nq, P, n_prune)
    ids, sc = gix.search(qd, P, n_prune, k, taps=taps)
    assert gix.status() == 0
    tn = taps_to_numpy(taps)
    res = oracle.pipeline(q[1].numpy(), oix, P, n_prune, k)
    check_query(tn, 1, res, ids[1].cpu().numpy(), sc[1].cpu().numpy(), k, n_prune)
