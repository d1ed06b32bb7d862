"""Stages 1 and 2a run together (chimera_search / chimera_run_stages over both): the probes come out of the score
table's epilogue through per-row key queues (Sec. 3.2 step 1: the top-n_probe centroids of a query token).  These
cases have enough centroids for that path (at least 8 sample tiles of 128 centroids at the sampling stride of the
nprobe in question) and compare the score table and the probes, bit for bit, with the oracle's table and its top
nprobe by (score descending, centroid id ascending); the same probes must come out of the separate probe stage."""
import numpy as np
import pytest
import torch

import oracle
from helpers import random_corpus, unit_rows

pytestmark = pytest.mark.gpu


def _run(cent, nq, B, nprobe, seed, q=None):
    import paper_2608_23553_b200 as pkg
    K, D = cent.shape
    rng = np.random.default_rng(seed)
    n_docs = 64
    doclens = rng.integers(1, 8, size=n_docs).astype(np.int32)
    T = int(doclens.sum())
    cids = rng.integers(0, K, size=T).astype(np.int32)
    codes = rng.integers(0, 256, size=(T, D // 4)).astype(np.uint8)
    dev = torch.device("cuda:0")
    gix = pkg.Index(torch.from_numpy(cent).to(dev), torch.from_numpy(cids).to(dev), torch.from_numpy(codes).to(dev),
                    torch.from_numpy(doclens).to(dev), 2)
    if q is None:
        q = np.stack([unit_rows(rng, nq, D) for _ in range(B)])
    qd = torch.from_numpy(q).to(dev)
    assert gix.probe_plan(B, nq, nprobe) > 1                       # enough centroids for the joint form
    taps = gix.alloc_taps(B, nq, nprobe, 8)
    pkg.profile_read()
    gix.run_stages(1, 2, qd, B, nq, nprobe, 8, 4, taps)            # both stages in one call: the queue path
    assert gix.status() == 0
    launches = pkg.profile_read()[1]
    # digits + the sample's tiles + the other tiles; sample lists (2 kernels) + bounds + merge + the flagged table scan (2)
    assert launches["score_table"] == 3 and launches["probes"] == 6, launches
    together = taps.probes.cpu().numpy().copy()
    table = taps.score_table.cpu().numpy().copy()
    gix.run_stages(2, 2, qd, B, nq, nprobe, 8, 4, taps)            # stage 2 alone: the table scan
    assert gix.status() == 0
    assert pkg.profile_read()[1]["probes"] == 2
    alone = taps.probes.cpu().numpy()
    gix.close()
    return q, table, together, alone


@pytest.mark.parametrize("K,nq,B,nprobe", [
    (4096 + 77, 32, 3, 32),        # stride 4: 33 tiles, ragged last tile, 9 sample tiles
    (8192 + 130, 40, 2, 16),       # stride 8, q_len not a multiple of the tile (rows straddle queries)
    (4096 + 77, 36, 2, 32),        # q_len a multiple of 4 only
    (32768, 64, 2, 7),             # stride 18 (not a power of two), two column groups
    (32768 + 1, 32, 5, 4),         # stride 32: the configurations' nprobe
    (32768 + 129, 32, 1, 1),       # nprobe 1 (the longest-tailed queue length), one query
])
def test_probes_from_the_epilogue_match_oracle(K, nq, B, nprobe):
    rng = np.random.default_rng(K + nprobe)
    cent = unit_rows(rng, K, 64)
    q, table, together, alone = _run(cent, nq, B, nprobe, seed=K)
    for b in range(B):
        S = oracle.score_table(q[b], cent)
        assert np.array_equal(table[b], S), "score table differs"
        want = oracle.probes(S, nprobe)
        assert np.array_equal(together[b], want), "probes of the joint stages differ"
        assert np.array_equal(alone[b], want), "probes of the separate stage differ"


def test_overflowing_queues_fall_back_to_the_table_scan():
    """30,000 copies of one centroid: for a query token close to it every copy reaches the bound, the queue overflows
    (capacity 1024) and the query is redone by the table scan; ties go to the lowest centroid ids.  The other query's
    tokens are far from the copies and stay on the queue path."""
    K, D, nq, nprobe = 33000, 64, 32, 4
    rng = np.random.default_rng(99)
    cent = unit_rows(rng, K, D)
    hot = unit_rows(rng, 1, D)[0]
    where = rng.permutation(K)[:30000]
    cent[where] = hot
    q = np.stack([unit_rows(rng, nq, D) for _ in range(2)])
    q[0, :8] = hot                                                # eight tokens of query 0 equal the copied centroid
    q, table, together, alone = _run(cent, nq, 2, nprobe, seed=5, q=q.astype(np.float32))
    for b in range(2):
        S = oracle.score_table(q[b], cent)
        want = oracle.probes(S, nprobe)
        assert np.array_equal(together[b], want)
        assert np.array_equal(alone[b], want)
    assert np.array_equal(together[0, 0], np.sort(where)[:nprobe])     # the tie goes to the lowest ids


def test_full_search_uses_the_joint_stages_and_matches_oracle():
    """End to end on a corpus with 33,000 centroids: chimera_search (joint stages) against the oracle's pipeline."""
    import paper_2608_23553_b200 as pkg
    from parity import check_query, taps_to_numpy
    K, D, N, nq, B = 33000, 64, 3000, 32, 4
    cent, cids, codes, doclens = random_corpus(17, N, K, D, 2, len_lo=4, len_hi=40)
    # random ids over 33,000 centroids would leave every probed list nearly empty: fold the ids onto 600 centroids
    cids = (cids % 600).astype(np.int32) * 55
    dev = torch.device("cuda:0")
    gix = pkg.Index(torch.from_numpy(cent).to(dev), torch.from_numpy(cids).to(dev), torch.from_numpy(codes).to(dev),
                    torch.from_numpy(doclens).to(dev), 2)
    oix = oracle.make_index(cent, cids, codes, doclens, 2)
    rng = np.random.default_rng(3)
    # query tokens near used centroids, so that the probes retrieve documents
    q = np.stack([cent[(rng.integers(0, 600, size=nq)) * 55] + 0.3 * unit_rows(rng, nq, D) for _ in range(B)])
    q = (q / np.linalg.norm(q, axis=-1, keepdims=True)).astype(np.float32)
    taps = gix.alloc_taps(B, nq, 4, 64)
    ids, sc = gix.search(torch.from_numpy(q).to(dev), 4, 64, 10, taps=taps)
    assert gix.status() == 0
    tn = taps_to_numpy(taps)
    assert int(tn["n_cand"].min()) > 64
    for b in range(B):
        res = oracle.pipeline(q[b], oix, 4, 64, 10)
        check_query(tn, b, res, ids[b].cpu().numpy(), sc[b].cpu().numpy(), 10, 64)
    gix.close()


def test_random_shapes_of_both_forms_match_oracle():
    """Random (dimension, centroid count, nprobe, q_len, batch) draws, a third of them with masses of duplicated
    centroids (ties; sometimes overflowing queues): whichever form of stage 2a the library chooses, the table and the
    probes are the oracle's."""
    import paper_2608_23553_b200 as pkg
    rng = np.random.default_rng(2024)
    dev = torch.device("cuda:0")
    forms = set()
    for case in range(14):
        D = int(rng.choice([32, 64, 96, 128]))
        K = int(rng.integers(1100, 50000))
        P = int(rng.integers(1, 40))
        nq = int(rng.choice([4, 8, 12, 16, 20, 32, 36, 48, 64, 100]))
        B = int(rng.integers(1, 5))
        dup = case % 3 == 2
        cent = unit_rows(rng, K, D)
        if dup:
            dst = rng.permutation(K)[:K // 2]
            cent[dst] = cent[int(rng.integers(0, K))] if case % 2 == 0 else cent[rng.integers(0, K, size=K // 2)]
        doclens = rng.integers(1, 6, size=32).astype(np.int32)
        T = int(doclens.sum())
        cids = rng.integers(0, K, size=T).astype(np.int32)
        codes = rng.integers(0, 256, size=(T, D // 4)).astype(np.uint8)
        gix = pkg.Index(torch.from_numpy(cent).to(dev), torch.from_numpy(cids).to(dev),
                        torch.from_numpy(codes).to(dev), torch.from_numpy(doclens).to(dev), 2)
        q = np.stack([unit_rows(rng, nq, D) for _ in range(B)])
        if dup:
            q[0, 0] = cent[dst[0]]                      # a query token equal to a duplicated centroid
        forms.add(gix.probe_plan(B, nq, P) > 1)
        taps = gix.alloc_taps(B, nq, P, 4)
        gix.run_stages(1, 2, torch.from_numpy(q).to(dev), B, nq, P, 4, 2, taps)
        assert gix.status() == 0
        got, tab = taps.probes.cpu().numpy(), taps.score_table.cpu().numpy()
        for b in range(B):
            S = oracle.score_table(q[b], cent)
            assert np.array_equal(tab[b], S), (case, D, K, P, nq, B)
            assert np.array_equal(got[b], oracle.probes(S, P)), (case, D, K, P, nq, B)
        gix.close()
    assert forms == {True, False}                       # the draw covers both forms
