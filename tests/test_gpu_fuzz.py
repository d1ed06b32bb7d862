"""Seeded random small configurations through all three pipelines against the oracle (ragged sizes, every supported
dim / bit width, q_len on both sides of the kernel variants' boundaries)."""
import numpy as np
import pytest
import torch

import oracle
from helpers import random_corpus, unit_rows
from parity import check_query, taps_to_numpy

pytestmark = pytest.mark.gpu


def _cases(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(n):
        D = int(rng.choice([32, 64, 96, 128]))
        nbits = int(rng.choice([1, 2]))
        nq = int(rng.choice([1, 3, 16, 31, 32, 33, 48, 64, 65, 90, 127]))
        K = int(rng.integers(2, 200))
        N = int(rng.integers(1, 700))
        nprobe = int(rng.integers(1, min(K, 64) + 1))
        n_prune = int(rng.integers(1, 300))
        k = int(rng.integers(1, 120))
        len_hi = int(rng.choice([1, 5, 40, 150]))
        out.append((D, nbits, nq, K, N, nprobe, n_prune, k, len_hi, int(rng.integers(1 << 30))))
    return out


def _larger_cases(n, seed):
    """Corpora of thousands to tens of thousands of documents: long candidate lists, the multi-block selections that
    serve small batches, n_prune and k in the thousands."""
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(n):
        D = int(rng.choice([32, 64, 96, 128]))
        nbits = int(rng.choice([1, 2]))
        nq = int(rng.choice([8, 32, 32, 64, 33, 100]))
        K = int(rng.choice([64, 300, 1024, 4096]))
        N = int(rng.choice([3000, 9000, 20000, 40000, 70000]))
        nprobe = min(int(rng.choice([1, 2, 4, 8, 32])), K)
        n_prune = int(rng.choice([10, 256, 1024, 5000]))
        k = int(rng.choice([1, 10, 100, 1000]))
        len_hi = int(rng.choice([3, 20, 60]))
        out.append((D, nbits, nq, K, N, nprobe, n_prune, k, len_hi, int(rng.integers(1 << 30))))
    return out


@pytest.mark.parametrize("case", _cases(24, 2024) + _larger_cases(10, 77))
def test_random_configuration_all_pipelines(case):
    import paper_2608_23553_b200 as pkg
    from synth import CONFIGS, encode_rabitq_1bit, random_rotation
    D, nbits, nq, K, N, nprobe, n_prune, k, len_hi, seed = case
    cent, cids, codes, doclens = random_corpus(seed, N, K, D, nbits, len_lo=1, len_hi=len_hi)
    rng = np.random.default_rng(seed + 1)
    oix = oracle.make_index(cent, cids, codes, doclens, nbits)
    dev = torch.device("cuda:0")
    gix = pkg.Index(torch.from_numpy(cent).to(dev), torch.from_numpy(cids).to(dev), torch.from_numpy(codes).to(dev),
                    torch.from_numpy(doclens).to(dev), nbits)
    B = int(rng.integers(1, 4))
    q = np.stack([unit_rows(rng, nq, D) for _ in range(B)])
    qd = torch.from_numpy(q).cuda()
    # 1. the specified pipeline
    taps = gix.alloc_taps(B, nq, nprobe, n_prune)
    ids, sc = gix.search(qd, nprobe, n_prune, k, taps=taps)
    assert gix.status() == 0
    tn = taps_to_numpy(taps)
    for b in range(B):
        res = oracle.pipeline(q[b], oix, nprobe, n_prune, k)
        check_query(tn, b, res, ids[b].cpu().numpy(), sc[b].cpu().numpy(), k, n_prune)
    # 2. partial-score refinement
    gix.enable_partial()
    taps = gix.alloc_taps(B, nq, nprobe, n_prune, table=False)
    ids, sc = gix.search(qd, nprobe, n_prune, k, taps=taps, partial=True)
    assert gix.status() == 0
    tn = taps_to_numpy(taps)
    for b in range(B):
        res = oracle.pipeline(q[b], oix, nprobe, n_prune, k, partial=True)
        check_query(tn, b, res, ids[b].cpu().numpy(), sc[b].cpu().numpy(), k, n_prune, table=False)
    # 3. RaBitQ 1-bit pipeline (q_len <= 64)
    if nq <= 64:
        raw = unit_rows(rng, len(cids), D)
        P = random_rotation(CONFIGS["tiny"].replace(dim=D, seed=seed % 1000))
        bits, inv = encode_rabitq_1bit(torch.from_numpy(raw), P)
        rq = oracle.make_rabitq(P, bits, inv)
        gix.attach_rabitq(P.to(dev), bits.to(dev), inv.to(dev))
        taps = gix.alloc_taps(B, nq, nprobe, n_prune, table=False)
        ids, sc = gix.search(qd, nprobe, n_prune, k, taps=taps, rabitq=True)
        assert gix.status() == 0
        for b in range(B):
            res = oracle.pipeline_rabitq(q[b], oix, rq, nprobe, n_prune, k)
            n = int(taps.n_cand[b])
            assert np.array_equal(taps.ci[b, :n].cpu().numpy(), res.ci.view(np.int32))
            assert np.array_equal(taps.pruned[b, :len(res.pruned)].cpu().numpy(), res.pruned)
            assert np.array_equal(ids[b].cpu().numpy(), res.ids) and np.array_equal(sc[b].cpu().numpy(), res.scores)
