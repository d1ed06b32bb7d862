"""The give-up path of the bounded device-side waits, exercised without faulting or hanging the GPU: a test hook makes
the two tensor-core kernels issue no TMA load, so their mbarrier waits run into a (shortened) limit with nothing in
flight; every block sets the TIMEOUT status bit, frees its tensor memory and returns.  The context stays usable and the
next ordinary search is correct."""
import ctypes
import time

import numpy as np
import pytest
import torch

import oracle
from parity import check_query, taps_to_numpy

pytestmark = pytest.mark.gpu

TIMEOUT = 5


def test_waits_that_run_out_report_timeout_and_leave_the_context_usable():
    import paper_2608_23553_b200 as pkg
    from synth import CONFIGS, make_corpus, make_queries
    L = pkg.lib()
    cfg = CONFIGS["tiny"].replace(n_docs=1500, n_centroids=256, n_queries=3)
    corp = make_corpus(cfg)
    q = make_queries(cfg)
    oix = oracle.make_index(corp.centroids, corp.cids, corp.codes, corp.doclens, cfg.nbits, cfg.res_lo, cfg.res_hi)
    dev = torch.device("cuda:0")
    gix = pkg.Index(corp.centroids.to(dev), corp.cids.to(dev), corp.codes.to(dev), corp.doclens.to(dev), cfg.nbits,
                    cfg.res_lo, cfg.res_hi)
    qd = q.to(dev)
    nprobe, n_prune, k = cfg.nprobe, 64, cfg.k
    gix.search(qd, nprobe, n_prune, k)
    assert gix.status() == 0
    try:
        # ~1 ms limit (2,000,000 cycles), no TMA loads: stage 1's waits give up first
        assert L.chimera_test_wait_fault(ctypes.c_int32(1), ctypes.c_int64(2_000_000)) == 0
        t0 = time.perf_counter()
        gix.search(qd, nprobe, n_prune, k)
        assert gix.status() == TIMEOUT                      # synchronises: the kernels returned by themselves
        assert time.perf_counter() - t0 < 5.0
        # stage 4 alone (its predecessors' results supplied): the same for the second tensor-core kernel
        L.chimera_test_wait_fault(ctypes.c_int32(0), ctypes.c_int64(0))
        taps = gix.alloc_taps(q.shape[0], cfg.q_len, nprobe, n_prune)
        gix.search(qd, nprobe, n_prune, k, taps=taps)
        assert gix.status() == 0
        L.chimera_test_wait_fault(ctypes.c_int32(1), ctypes.c_int64(2_000_000))
        gix.run_stages(4, 5, qd, q.shape[0], cfg.q_len, nprobe, n_prune, k, taps)
        assert gix.status() == TIMEOUT
    finally:
        L.chimera_test_wait_fault(ctypes.c_int32(0), ctypes.c_int64(0))
    # normal operation again, same index, same workspace: every stage equals the oracle
    taps = gix.alloc_taps(q.shape[0], cfg.q_len, nprobe, n_prune)
    ids, sc = gix.search(qd, nprobe, n_prune, k, taps=taps)
    assert gix.status() == 0
    tn = taps_to_numpy(taps)
    ids, sc = ids.cpu().numpy(), sc.cpu().numpy()
    for b in range(q.shape[0]):
        res = oracle.pipeline(q[b].numpy(), oix, nprobe, n_prune, k)
        check_query(tn, b, res, ids[b], sc[b], k, n_prune)
