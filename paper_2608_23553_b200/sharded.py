"""Document-sharded search over several GPUs, one process per GPU (the scaling sketch of Sec. 3.3).

The documents are split into `world` contiguous id ranges in rank order; every rank indexes its own range and all
centroids.  Queries are the same on every rank.  A search is three library calls with two all-gathers of ids and
scores between them (never codes):

    local top n_prune + stage-3 scores --all-gather--> global top n_prune, own survivors scored, local top-k
                                       --all-gather--> merged top-k

Stage-3 scores are integers that do not depend on the shard and a document's stage-4 score does not depend on the
shard it is scored in, so the result equals the single-index result bit for bit.

The exchange is a plain collective of a few KB per query (torch.distributed: NCCL between GPUs); there is no compute to
overlap it with, so it is not fused into a kernel.  `ShardedSearcher` only sequences the phases; the phases themselves
are an engine's: `ShardEngine` runs them in the CUDA library.
"""
from __future__ import annotations

import ctypes
from typing import Callable, List, Optional, Tuple

import torch

from .binding import Index, _check, _ptr, _stream, lib

MODES = {"ci": 0, "partial": 1, "rabitq": 2}


def shard_ranges(n_docs: int, world: int) -> List[Tuple[int, int]]:
    """Contiguous, near-equal document ranges [lo, hi) in rank order; the first n_docs % world ranks get one more."""
    if world < 1 or n_docs < world:
        raise ValueError("need 1 <= world <= n_docs")
    base, extra = divmod(n_docs, world)
    out, lo = [], 0
    for r in range(world):
        hi = lo + base + (1 if r < extra else 0)
        out.append((lo, hi))
        lo = hi
    return out


class ShardEngine:
    """The three phases of a sharded search on one rank's Index (all work in the CUDA library)."""

    def __init__(self, index: Index, doc_base: int, mode: str = "ci"):
        self.index, self.doc_base, self.mode = index, int(doc_base), MODES[mode]
        self.device = index.device

    def _common(self, queries, nprobe, n_prune, k, max_candidates):
        assert queries.is_cuda and queries.dtype == torch.float32 and queries.is_contiguous()
        B, q_len, dim = queries.shape
        assert dim == self.index.dim
        ws = self.index._workspace(self.index.workspace_bytes(B, q_len, nprobe, n_prune, k, max_candidates))
        head = (self.index._h, _ptr(queries), ctypes.c_int32(B), ctypes.c_int32(q_len), ctypes.c_int32(nprobe),
                ctypes.c_int32(n_prune), ctypes.c_int32(k), ctypes.c_int64(max_candidates), ctypes.c_int32(self.mode),
                ctypes.c_int64(self.doc_base))
        return B, ws, head

    def local_phase(self, queries, nprobe, n_prune, k, max_candidates=0):
        """-> (global ids [B, n_prune] int32 ascending, -1 padded; stage-3 scores [B, n_prune] int32)."""
        B, ws, head = self._common(queries, nprobe, n_prune, k, max_candidates)
        ids = torch.empty(B, n_prune, dtype=torch.int32, device=self.device)
        sc3 = torch.empty(B, n_prune, dtype=torch.int32, device=self.device)
        with torch.cuda.device(self.device):
            _check(lib().chimera_shard_local(*head, _ptr(ws), ctypes.c_size_t(ws.numel()), _stream(), _ptr(ids),
                                             _ptr(sc3)))
        return ids, sc3

    def finish_phase(self, queries, nprobe, n_prune, k, all_ids, all_sc3, max_candidates=0):
        """all_ids / all_sc3: [world, B, n_prune] gathered in rank order -> this rank's top-k (global ids, scores)."""
        B, ws, head = self._common(queries, nprobe, n_prune, k, max_candidates)
        world = all_ids.shape[0]
        assert all_ids.shape == (world, B, n_prune) and all_sc3.shape == all_ids.shape
        assert all_ids.is_contiguous() and all_sc3.is_contiguous()
        ids = torch.empty(B, k, dtype=torch.int32, device=self.device)
        scores = torch.empty(B, k, dtype=torch.float32, device=self.device)
        with torch.cuda.device(self.device):
            _check(lib().chimera_shard_finish(*head, ctypes.c_int32(world), _ptr(all_ids), _ptr(all_sc3), _ptr(ws),
                                              ctypes.c_size_t(ws.numel()), _stream(), _ptr(ids), _ptr(scores)))
        return ids, scores

    def merge_phase(self, all_ids, all_scores):
        """all_ids / all_scores: [world, B, k] -> the best k of the union per query."""
        world, B, k = all_ids.shape
        assert all_ids.is_contiguous() and all_scores.is_contiguous()
        ids = torch.empty(B, k, dtype=torch.int32, device=all_ids.device)
        scores = torch.empty(B, k, dtype=torch.float32, device=all_ids.device)
        with torch.cuda.device(all_ids.device):
            _check(lib().chimera_shard_merge_topk(_ptr(all_ids), _ptr(all_scores), ctypes.c_int32(world),
                                                  ctypes.c_int32(B), ctypes.c_int32(k), _stream(), _ptr(ids),
                                                  _ptr(scores)))
        return ids, scores

    def status_word(self) -> torch.Tensor:
        """The workspace's raw device-side status bits (candidate overflow, bad query element, bounded wait given up)
        as an int32 device tensor of one element, without synchronising the host.  The finish phase keeps the bits the
        local phase set, so reading it after the finish phase covers the whole search."""
        return self.index._ws[:4].view(torch.int32).clone()

    def check(self):
        """Raise if the phases so far overflowed the candidate capacity or a kernel gave up waiting (this rank only;
        synchronises).  ShardedSearcher does not use it: it exchanges the status words so that every rank raises."""
        st = self.index.status()
        if st:
            raise RuntimeError("shard workspace status %d" % st)


def all_gather_stack(t: torch.Tensor, group=None) -> torch.Tensor:
    """[...] on every rank -> [world, ...] in rank order (torch.distributed all-gather)."""
    import torch.distributed as dist
    world = dist.get_world_size(group)
    out = torch.empty((world,) + tuple(t.shape), dtype=t.dtype, device=t.device)
    dist.all_gather(list(out.unbind(0)), t.contiguous(), group=group)       # the views fill `out` in place
    return out


class ShardError(RuntimeError):
    """A rank's device-side status was non-zero (candidate overflow, bad query element, a bounded wait that gave up).
    Raised on EVERY rank, after all collectives of the search have completed; `status` lists each rank's bits."""

    def __init__(self, status: List[int]):
        bad = ", ".join("rank %d: 0x%x" % (r, s) for r, s in enumerate(status) if s)
        super().__init__("sharded search: device status non-zero on " + bad)
        self.status = status


class ShardedSearcher:
    """Sequences the phases of one rank.  `engine` provides local_phase / finish_phase / merge_phase and optionally
    status_word (ShardEngine); `gather` maps a tensor to the rank-ordered stack of every rank's tensor (default:
    all_gather_stack).

    Failure handling is collective: no rank raises between the collectives (a rank that left early would leave the
    others blocked in their next all-gather).  Each rank's status word travels with the second exchange, and after the
    merge every rank sees every rank's word and raises ShardError together.  check=False skips that host
    synchronisation (the caller reads `last_status`, a device tensor [world], when it chooses to)."""

    def __init__(self, engine, gather: Optional[Callable[[torch.Tensor], torch.Tensor]] = None, group=None,
                 check: bool = True):
        self.engine = engine
        self.gather = gather if gather is not None else (lambda t: all_gather_stack(t, group))
        self.check = check
        self.last_status = None

    def search(self, queries, nprobe: int, n_prune: int, k: int, max_candidates: int = 0):
        ids, sc3 = self.engine.local_phase(queries, nprobe, n_prune, k, max_candidates)
        all_ids, all_sc3 = self.gather(ids), self.gather(sc3)
        top_ids, top_scores = self.engine.finish_phase(queries, nprobe, n_prune, k, all_ids, all_sc3, max_candidates)
        all_top_ids, all_top_scores = self.gather(top_ids), self.gather(top_scores)
        if hasattr(self.engine, "status_word"):
            self.last_status = self.gather(self.engine.status_word()).view(-1)
        out = self.engine.merge_phase(all_top_ids, all_top_scores)
        if self.check and self.last_status is not None:
            words = [int(w) for w in self.last_status.cpu().tolist()]
            if any(words):
                raise ShardError(words)
        return out
