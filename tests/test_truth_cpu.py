"""The recall sweeps' ground-truth scorer (bench.brute_force_maxsim: exhaustive MaxSim from the definition in plain
torch, independent of the CUDA library) against the CPU oracle's exhaustive scores, on the CPU.  The GPU tests repeat
this at the sizes the sweep uses."""
import os
import sys

import numpy as np
import pytest
import torch

import oracle
from helpers import random_corpus, unit_rows

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))


@pytest.mark.parametrize("D,nbits,nq,N,chunk", [(32, 2, 5, 70, 40), (96, 1, 8, 40, 1 << 18), (128, 2, 32, 30, 17)])
def test_brute_force_scorer_equals_oracle_exhaustive_scores(D, nbits, nq, N, chunk):
    import bench
    cent, cids, codes, doclens = random_corpus(D + nq, N, 8, D, nbits, len_lo=1, len_hi=9)
    q = np.stack([unit_rows(np.random.default_rng(b), nq, D) for b in range(3)])
    oix = oracle.make_index(cent, cids, codes, doclens, nbits)
    sc = bench.brute_force_maxsim(torch.from_numpy(cent), torch.from_numpy(cids), torch.from_numpy(codes),
                                  torch.from_numpy(doclens), nbits, -0.25, 0.25, torch.from_numpy(q), q_group=2,
                                  chunk_tokens=chunk).numpy()
    for b in range(3):
        ref = oracle.score_docs(q[b], np.arange(N, dtype=np.int32), oix)
        assert np.abs(sc[b] - ref).max() <= 1e-5
