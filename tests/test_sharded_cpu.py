"""Document-sharded search (Sec. 3.3 scaling sketch), host side, on two and three gloo ranks on the CPU: the phase
sequencing and the all-gathers of paper_2608_23553_b200.sharded with an engine that computes the phases with the CPU
oracle (the CUDA engine has the same three methods and is checked on the GPU against the single-index search).  What
must hold, and what a wrong protocol breaks: the merged top-k equals the oracle's pipeline on the whole corpus, ids
and float scores exactly."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
INT_MIN = -2 ** 31


class OracleEngine:
    """The three phases, each written out from its definition with the oracle's stage functions."""

    def __init__(self, oracle, oix, doc_base, partial=False):
        self.o, self.oix, self.base, self.partial = oracle, oix, doc_base, partial

    def local_phase(self, q, nprobe, n_prune, k, max_candidates=0):
        B = q.shape[0]
        ids = np.full((B, n_prune), -1, np.int32)
        sc3 = np.full((B, n_prune), INT_MIN, np.int32)
        for b in range(B):
            res = self.o.pipeline(q[b].numpy(), self.oix, nprobe, n_prune, k, partial=self.partial)
            m = len(res.pruned)
            ids[b, :m] = res.pruned + self.base
            sc3[b, :m] = res.ci[np.searchsorted(res.cand, res.pruned)]
        return torch.from_numpy(ids), torch.from_numpy(sc3)

    def finish_phase(self, q, nprobe, n_prune, k, all_ids, all_sc3, max_candidates=0):
        B = q.shape[0]
        out_ids = np.full((B, k), -1, np.int32)
        out_sc = np.full((B, k), -np.inf, np.float32)
        for b in range(B):
            gid = all_ids[:, b].reshape(-1).numpy()
            s3 = all_sc3[:, b].reshape(-1).numpy().astype(np.int64)
            keep = gid >= 0
            gid, s3 = gid[keep], s3[keep]
            order = np.lexsort((gid, -s3))[:n_prune]                 # score descending, id ascending
            mine = np.sort(gid[order])
            mine = mine[(mine >= self.base) & (mine < self.base + self.oix.N)] - self.base
            s4 = self.o.score_docs(q[b].numpy(), mine.astype(np.int32), self.oix)
            ids, sc = self.o.topk(mine.astype(np.int32), s4, k)
            out_ids[b] = np.where(ids >= 0, ids + self.base, -1)
            out_sc[b] = sc
        return torch.from_numpy(out_ids), torch.from_numpy(out_sc)

    def merge_phase(self, all_ids, all_scores):
        world, B, k = all_ids.shape
        out_ids = np.full((B, k), -1, np.int32)
        out_sc = np.full((B, k), -np.inf, np.float32)
        for b in range(B):
            gid = all_ids[:, b].reshape(-1).numpy()
            sc = all_scores[:, b].reshape(-1).numpy()
            keep = gid >= 0
            gid, sc = gid[keep], sc[keep]
            order = np.lexsort((gid, -sc.astype(np.float64)))[:k]
            out_ids[b, :len(order)] = gid[order]
            out_sc[b, :len(order)] = sc[order]
        return torch.from_numpy(out_ids), torch.from_numpy(out_sc)


def _corpus(seed, N, K, D, nbits):
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from helpers import random_corpus, unit_rows
    cent, cids, codes, doclens = random_corpus(seed, N, K, D, nbits, len_lo=1, len_hi=20)
    q = np.stack([unit_rows(np.random.default_rng(100 + b), 8, D) for b in range(3)])
    return cent, cids, codes, doclens, q


def _rank(rank, world, port, partial, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    from paper_2608_23553_b200.sharded import ShardedSearcher, shard_ranges
    N, K, D, nbits, nprobe, n_prune, k = 151, 24, 32, 2, 3, 20, 7
    cent, cids, codes, doclens, q = _corpus(7, N, K, D, nbits)
    lo, hi = shard_ranges(N, world)[rank]
    off = np.concatenate([[0], np.cumsum(doclens, dtype=np.int64)])
    t0, t1 = int(off[lo]), int(off[hi])
    oix = oracle.make_index(cent, cids[t0:t1], codes[t0:t1], doclens[lo:hi], nbits)
    searcher = ShardedSearcher(OracleEngine(oracle, oix, lo, partial))
    ids, sc = searcher.search(torch.from_numpy(q), nprobe, n_prune, k)
    full = oracle.make_index(cent, cids, codes, doclens, nbits)
    ok = True
    for b in range(q.shape[0]):
        res = oracle.pipeline(q[b], full, nprobe, n_prune, k, partial=partial)
        ok = ok and np.array_equal(ids[b].numpy(), res.ids) and np.array_equal(sc[b].numpy(), res.scores)
    out[rank] = ok
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("world,partial", [(2, False), (3, False), (2, True)])
def test_sharded_protocol_reproduces_the_single_index_result(world, partial):
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_rank, args=(world, 29741 + os.getpid() % 200 + 7 * world + int(partial), partial, out), nprocs=world,
                 join=True)
        assert all(out[r] for r in range(world)) and len(out) == world


class _FlaggingEngine(OracleEngine):
    """An engine whose device status is non-zero on one rank (as after a candidate overflow there)."""

    def __init__(self, *a, flag=0):
        super().__init__(*a)
        self.flag = flag

    def status_word(self):
        return torch.tensor([self.flag], dtype=torch.int32)


def _rank_flagged(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    import datetime
    dist.init_process_group("gloo", rank=rank, world_size=world, timeout=datetime.timedelta(seconds=60))
    import oracle
    from paper_2608_23553_b200.sharded import ShardedSearcher, ShardError, shard_ranges
    N, K, D, nbits = 90, 16, 32, 2
    cent, cids, codes, doclens, q = _corpus(11, N, K, D, nbits)
    lo, hi = shard_ranges(N, world)[rank]
    off = np.concatenate([[0], np.cumsum(doclens, dtype=np.int64)])
    oix = oracle.make_index(cent, cids[int(off[lo]):int(off[hi])], codes[int(off[lo]):int(off[hi])], doclens[lo:hi], nbits)
    searcher = ShardedSearcher(_FlaggingEngine(oracle, oix, lo, False, flag=1 if rank == 1 else 0))
    try:
        searcher.search(torch.from_numpy(q), 2, 10, 5)
        out[rank] = "no error"
    except ShardError as e:
        out[rank] = list(e.status)
    # every rank is still in step: a further collective completes
    dist.barrier()
    quiet = ShardedSearcher(_FlaggingEngine(oracle, oix, lo, False, flag=1 if rank == 1 else 0), check=False)
    quiet.search(torch.from_numpy(q), 2, 10, 5)
    out["quiet%d" % rank] = quiet.last_status.tolist()
    dist.barrier()
    dist.destroy_process_group()


def test_one_ranks_bad_status_raises_on_every_rank_after_the_collectives():
    world = 3
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_rank_flagged, args=(world, 29951 + os.getpid() % 200, out), nprocs=world, join=True)
        for r in range(world):
            assert out[r] == [0, 1, 0]
            assert out["quiet%d" % r] == [0, 1, 0]


def test_shard_ranges_partition_the_documents():
    sys.path.insert(0, ROOT)
    from paper_2608_23553_b200.sharded import shard_ranges
    for n, w in [(10, 1), (10, 3), (7, 7), (1000003, 8)]:
        r = shard_ranges(n, w)
        assert r[0][0] == 0 and r[-1][1] == n and len(r) == w
        assert all(a[1] == b[0] for a, b in zip(r, r[1:]))
        sizes = [hi - lo for lo, hi in r]
        assert max(sizes) - min(sizes) <= 1 and min(sizes) >= 1
    with pytest.raises(ValueError):
        shard_ranges(3, 4)


def test_shard_entry_points_reject_bad_arguments_without_a_device():
    import ctypes
    sys.path.insert(0, ROOT)
    from paper_2608_23553_b200 import binding, build
    build.build()
    L = binding.lib()
    i64 = ctypes.c_int64
    assert L.chimera_shard_local(None, None, 1, 32, 4, 16, 10, i64(0), 0, i64(0), None, ctypes.c_size_t(0), None, None,
                                 None) == 1
    assert L.chimera_shard_finish(None, None, 1, 32, 4, 16, 10, i64(0), 0, i64(0), 2, None, None, None,
                                  ctypes.c_size_t(0), None, None, None) == 1
    assert L.chimera_shard_merge_topk(None, None, 2, 1, 10, None, None, None) == 1
    fake = ctypes.c_void_p(256)
    assert L.chimera_shard_merge_topk(fake, fake, 4, 1, 8192, None, fake, fake) == 6      # world * k > 16384
    assert L.chimera_shard_merge_topk(fake, fake, 0, 1, 10, None, fake, fake) == 1
