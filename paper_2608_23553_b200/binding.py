"""ctypes binding of libchimera's C ABI (declared in include/chimera.h).

Argument marshalling only: torch supplies device memory and the current CUDA stream, every computation runs inside
the library.  The library must have been built (`python -m paper_2608_23553_b200.build`); a missing library is an
error, never a fallback.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
# CHIMERA_DEBUG_LIB=1 loads the debug build (index checks before every gather, guard regions in the workspace)
_DEBUG = os.environ.get("CHIMERA_DEBUG_LIB", "0") == "1"
_LIB_PATH = os.path.join(_PKG, "libchimera_debug.so" if _DEBUG else "libchimera.so")
_lib = None

PROFILE_SLOTS = ("score_table", "probes", "gather", "centroid_interaction", "select", "residual_scores", "topk",
                 "misc", "ci_exact")

STATUS_NAMES = {0: "OK", 1: "INVALID_ARG", 2: "CUDA_ERROR", 3: "WORKSPACE_TOO_SMALL", 4: "CAPACITY_OVERFLOW",
                5: "TIMEOUT", 6: "UNSUPPORTED", 7: "DEBUG_CHECK_FAILED"}


class ChimeraError(RuntimeError):
    def __init__(self, code: int, text: str):
        super().__init__("chimera: %s (%d): %s" % (STATUS_NAMES.get(code, "?"), code, text))
        self.code = code


class _Desc(ctypes.Structure):
    _fields_ = [("dim", ctypes.c_int32), ("nbits", ctypes.c_int32), ("res_lo", ctypes.c_float),
                ("res_hi", ctypes.c_float), ("n_centroids", ctypes.c_int64), ("n_docs", ctypes.c_int64),
                ("n_tokens", ctypes.c_int64)]


class _Taps(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in
                ("score_table", "probes", "cand", "n_cand", "ci", "pruned", "n_pruned", "score4", "n_contenders")]


def library_path() -> str:
    return _LIB_PATH


def lib():
    """Load libchimera.so (built in-tree).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError("%s is not built: run `python -m paper_2608_23553_b200.build%s` "
                              "(there is no CPU fallback)" % (os.path.basename(_LIB_PATH), " --debug" if _DEBUG else ""))
        L = ctypes.CDLL(_LIB_PATH)
        L.chimera_last_error.restype = ctypes.c_char_p
        _lib = L
    return _lib


def _check(rc: int):
    if rc != 0:
        raise ChimeraError(rc, lib().chimera_last_error().decode())


def _ptr(t: Optional[torch.Tensor]):
    return ctypes.c_void_p(0 if t is None else t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


@dataclass
class Taps:
    """Intermediate results of a search (device tensors)."""
    score_table: Optional[torch.Tensor] = None   # [B, K, nq] int32
    probes: Optional[torch.Tensor] = None        # [B, nq, nprobe] int32
    cand: Optional[torch.Tensor] = None          # [B, maxc] int32
    n_cand: Optional[torch.Tensor] = None        # [B] int32
    ci: Optional[torch.Tensor] = None            # [B, maxc] int32
    pruned: Optional[torch.Tensor] = None        # [B, n_prune] int32
    n_pruned: Optional[torch.Tensor] = None      # [B] int32
    score4: Optional[torch.Tensor] = None        # [B, n_prune] float32
    n_contenders: Optional[torch.Tensor] = None  # [B] int32

    def _c(self) -> _Taps:
        c = _Taps()
        for name, _ in _Taps._fields_:
            t = getattr(self, name)
            setattr(c, name, 0 if t is None else t.data_ptr())
        return c


def profile_enable(on: bool):
    _check(lib().chimera_profile_enable(ctypes.c_int32(1 if on else 0)))


def profile_read():
    """({slot: ms}, {slot: kernel launches}) accumulated since the last read."""
    n = len(PROFILE_SLOTS)
    ms = (ctypes.c_float * n)()
    launches = (ctypes.c_int64 * n)()
    _check(lib().chimera_profile_read(ms, launches))
    return ({PROFILE_SLOTS[i]: float(ms[i]) for i in range(n)},
            {PROFILE_SLOTS[i]: int(launches[i]) for i in range(n)})


class Index:
    """Device-resident index.  Holds references to the tensors the library borrows (cids, codes)."""

    def __init__(self, centroids: torch.Tensor, cids: torch.Tensor, codes: torch.Tensor, doclens: torch.Tensor,
                 nbits: int, res_lo: float = -0.25, res_hi: float = 0.25):
        L = lib()
        for t in (centroids, cids, codes, doclens):
            if not t.is_cuda:
                raise ValueError("index arrays must be CUDA tensors")
        self.device = centroids.device
        self.centroids = centroids.contiguous().to(torch.float32)
        self.cids = cids.contiguous().to(torch.int32)
        self.codes = codes.contiguous().to(torch.uint8)
        self.doclens = doclens.contiguous().to(torch.int32)
        self.K, self.dim = self.centroids.shape
        self.N = self.doclens.numel()
        self.T = self.cids.numel()
        self.nbits = nbits
        desc = _Desc(self.dim, nbits, res_lo, res_hi, self.K, self.N, self.T)
        self._h = ctypes.c_void_p()
        with torch.cuda.device(self.device):
            _check(L.chimera_build_index(ctypes.byref(desc), _ptr(self.centroids), _ptr(self.cids), _ptr(self.codes),
                                         _ptr(self.doclens), _stream(), ctypes.byref(self._h)))
        self._ws = None

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            lib().chimera_destroy_index(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def info(self):
        desc = _Desc()
        entries = ctypes.c_int64()
        mx = ctypes.c_int32()
        _check(lib().chimera_index_info(self._h, ctypes.byref(desc), ctypes.byref(entries), ctypes.byref(mx)))
        return {"dim": desc.dim, "nbits": desc.nbits, "n_centroids": desc.n_centroids, "n_docs": desc.n_docs,
                "n_tokens": desc.n_tokens, "posting_entries": entries.value, "max_doclen": mx.value}

    def workspace_bytes(self, n_queries, q_len, nprobe, n_prune, k, max_candidates=0) -> int:
        out = ctypes.c_size_t()
        _check(lib().chimera_workspace_bytes(self._h, ctypes.c_int32(n_queries), ctypes.c_int32(q_len),
                                             ctypes.c_int32(nprobe), ctypes.c_int32(n_prune), ctypes.c_int32(k),
                                             ctypes.c_int64(max_candidates), ctypes.byref(out)))
        return out.value

    def _workspace(self, nbytes: int) -> torch.Tensor:
        if self._ws is None or self._ws.numel() < nbytes:
            self._ws = None
            self._ws = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        return self._ws

    def _maxc(self, max_candidates):
        return self.N if (max_candidates == 0 or max_candidates > self.N) else max_candidates

    def alloc_taps(self, B, q_len, nprobe, n_prune, max_candidates=0, table=True, ci=True) -> Taps:
        dev, i32 = self.device, torch.int32
        mc = self._maxc(max_candidates)
        return Taps(
            score_table=torch.empty(B, self.K, q_len, dtype=i32, device=dev) if table else None,
            probes=torch.empty(B, q_len, nprobe, dtype=i32, device=dev),
            cand=torch.empty(B, mc, dtype=i32, device=dev), n_cand=torch.empty(B, dtype=i32, device=dev),
            ci=torch.empty(B, mc, dtype=i32, device=dev) if ci else None,
            n_contenders=torch.empty(B, dtype=i32, device=dev),
            pruned=torch.empty(B, n_prune, dtype=i32, device=dev), n_pruned=torch.empty(B, dtype=i32, device=dev),
            score4=torch.empty(B, n_prune, dtype=torch.float32, device=dev))

    def enable_partial(self):
        """Build the token-level posting lists needed by search(..., partial=True)."""
        with torch.cuda.device(self.device):
            _check(lib().chimera_index_enable_partial(self._h, _stream()))
        self._ws = None

    def attach_rabitq(self, rotation: torch.Tensor, bits: torch.Tensor, inv_dot: torch.Tensor):
        """Attach RaBitQ 1-bit codes (kept referenced) for search(..., rabitq=True)."""
        self._rq = (rotation.contiguous().to(torch.float32), bits.contiguous().to(torch.uint8),
                    inv_dot.contiguous().to(torch.float32))
        with torch.cuda.device(self.device):
            _check(lib().chimera_index_attach_rabitq(self._h, _ptr(self._rq[0]), _ptr(self._rq[1]), _ptr(self._rq[2]),
                                                     _stream()))
        self._ws = None

    def build_graph(self, degree: int):
        """Build the proximity graph over the centroids (chimera_index_build_graph) for graph_probes() and
        search(..., rabitq=True, graph=...)."""
        with torch.cuda.device(self.device):
            _check(lib().chimera_index_build_graph(self._h, _ptr(self.centroids), ctypes.c_int32(degree), _stream()))
        self._ws = None

    def graph(self) -> Optional[torch.Tensor]:
        """A copy of the centroid graph, [K, degree] int32 (None before build_graph)."""
        deg = ctypes.c_int32()
        _check(lib().chimera_index_copy_graph(self._h, None, ctypes.byref(deg), _stream()))
        if deg.value == 0:
            return None
        out = torch.empty(self.K, deg.value, dtype=torch.int32, device=self.device)
        with torch.cuda.device(self.device):
            _check(lib().chimera_index_copy_graph(self._h, _ptr(out), ctypes.byref(deg), _stream()))
        return out

    def graph_probes(self, queries: torch.Tensor, nprobe: int, beam: int, n_entries: int, max_expansions: int = 1 << 30):
        """The graph search alone (chimera_graph_probes).  Returns (probes [B, q_len, nprobe] int32, their fixed-point
        scores, visited counts [B, q_len] int32, visited bitmaps [B * q_len, ceil(K / 32)] int32)."""
        assert queries.is_cuda and queries.dtype == torch.float32 and queries.is_contiguous()
        B, q_len, dim = queries.shape
        assert dim == self.dim
        need = ctypes.c_size_t()
        _check(lib().chimera_graph_scratch_bytes(self._h, ctypes.c_int32(B), ctypes.c_int32(q_len), ctypes.byref(need)))
        vis = torch.empty(need.value // 4, dtype=torch.int32, device=self.device)
        probes = torch.empty(B, q_len, nprobe, dtype=torch.int32, device=self.device)
        scores = torch.empty(B, q_len, nprobe, dtype=torch.int32, device=self.device)
        n_vis = torch.empty(B, q_len, dtype=torch.int32, device=self.device)
        with torch.cuda.device(self.device):
            _check(lib().chimera_graph_probes(self._h, _ptr(queries), ctypes.c_int32(B), ctypes.c_int32(q_len),
                                              ctypes.c_int32(nprobe), ctypes.c_int32(beam), ctypes.c_int32(n_entries),
                                              ctypes.c_int32(min(max_expansions, (1 << 31) - 1)), _ptr(vis),
                                              ctypes.c_size_t(need.value), _stream(), _ptr(probes), _ptr(scores),
                                              _ptr(n_vis)))
        return probes, scores, n_vis, vis.view(B * q_len, -1)

    def search(self, queries: torch.Tensor, nprobe: int, n_prune: int, k: int, max_candidates: int = 0,
               taps: Optional[Taps] = None, out=None, partial: bool = False, rabitq: bool = False, graph=None):
        """queries: [B, q_len, dim] float32 CUDA tensor.  Returns (ids [B,k] int32, scores [B,k] float32).
        partial=True prunes with the paper's partial scores (chimera_search_partial); rabitq=True runs the paper's
        pipeline on 1-bit codes, with graph=(beam, n_entries, max_expansions) taking its probes from the centroid graph
        (chimera_search_rabitq_graph)."""
        assert queries.is_cuda and queries.dtype == torch.float32 and queries.is_contiguous()
        B, q_len, dim = queries.shape
        assert dim == self.dim
        nbytes = self.workspace_bytes(B, q_len, nprobe, n_prune, k, max_candidates)
        ws = self._workspace(nbytes)
        if out is None:
            ids = torch.empty(B, k, dtype=torch.int32, device=self.device)
            scores = torch.empty(B, k, dtype=torch.float32, device=self.device)
        else:
            ids, scores = out
        args = (self._h, _ptr(queries), ctypes.c_int32(B), ctypes.c_int32(q_len), ctypes.c_int32(nprobe),
                ctypes.c_int32(n_prune), ctypes.c_int32(k), ctypes.c_int64(max_candidates), _ptr(ws),
                ctypes.c_size_t(ws.numel()), _stream(), _ptr(ids), _ptr(scores))
        if graph is not None:
            assert rabitq, "graph probes belong to the RaBitQ pipeline"
            c = taps._c() if taps is not None else None
            beam, n_entries, max_exp = graph
            _check(lib().chimera_search_rabitq_graph(*args[:8], ctypes.c_int32(beam), ctypes.c_int32(n_entries),
                                                     ctypes.c_int32(min(max_exp, (1 << 31) - 1)), *args[8:],
                                                     ctypes.byref(c) if c is not None else None))
        elif partial or rabitq:
            c = taps._c() if taps is not None else None
            fn = lib().chimera_search_rabitq if rabitq else lib().chimera_search_partial
            _check(fn(*args, ctypes.byref(c) if c is not None else None))
        elif taps is None:
            _check(lib().chimera_search(*args))
        else:
            c = taps._c()
            _check(lib().chimera_search_tapped(*args, ctypes.byref(c)))
        return ids, scores

    def search_host(self, queries_host: torch.Tensor, nprobe: int, n_prune: int, k: int, max_candidates: int = 0,
                    out=None):
        """queries_host: [B, q_len, dim] float32 CPU tensor (pinned for speed).  Synchronous.  Returns CPU tensors."""
        assert (not queries_host.is_cuda) and queries_host.dtype == torch.float32 and queries_host.is_contiguous()
        B, q_len, dim = queries_host.shape
        assert dim == self.dim
        nbytes = self.workspace_bytes(B, q_len, nprobe, n_prune, k, max_candidates)
        ws = self._workspace(nbytes)
        if out is None:
            ids = torch.empty(B, k, dtype=torch.int32).pin_memory()
            scores = torch.empty(B, k, dtype=torch.float32).pin_memory()
        else:
            ids, scores = out
        with torch.cuda.device(self.device):
            _check(lib().chimera_search_host(self._h, _ptr(queries_host), ctypes.c_int32(B), ctypes.c_int32(q_len),
                                             ctypes.c_int32(nprobe), ctypes.c_int32(n_prune), ctypes.c_int32(k),
                                             ctypes.c_int64(max_candidates), _ptr(ws), ctypes.c_size_t(ws.numel()),
                                             _stream(), _ptr(ids), _ptr(scores)))
        return ids, scores

    def run_stages(self, first: int, last: int, queries: Optional[torch.Tensor], B: int, q_len: int, nprobe: int,
                   n_prune: int, k: int, taps: Taps, max_candidates: int = 0):
        """Run stages first..last with the earlier stages' results taken from `taps` (see chimera_run_stages)."""
        nbytes = self.workspace_bytes(B, q_len, nprobe, n_prune, k, max_candidates)
        ws = self._workspace(nbytes)
        ids = torch.empty(B, k, dtype=torch.int32, device=self.device)
        scores = torch.empty(B, k, dtype=torch.float32, device=self.device)
        c = taps._c()
        _check(lib().chimera_run_stages(self._h, ctypes.c_int32(first), ctypes.c_int32(last), _ptr(queries),
                                        ctypes.c_int32(B), ctypes.c_int32(q_len), ctypes.c_int32(nprobe),
                                        ctypes.c_int32(n_prune), ctypes.c_int32(k), ctypes.c_int64(max_candidates),
                                        _ptr(ws), ctypes.c_size_t(ws.numel()), _stream(), ctypes.byref(c),
                                        _ptr(ids), _ptr(scores)))
        return ids, scores

    def probe_plan(self, n_queries, q_len, nprobe) -> int:
        """0 when the probes come from a scan of the finished score table; otherwise the sampling stride of the joint
        form of stages 1 and 2a (chimera_probe_plan)."""
        s = ctypes.c_int32()
        _check(lib().chimera_probe_plan(self._h, ctypes.c_int32(n_queries), ctypes.c_int32(q_len),
                                        ctypes.c_int32(nprobe), ctypes.byref(s)))
        return s.value

    def workspace_check(self, n_queries, q_len, nprobe, n_prune, k, max_candidates=0) -> int:
        """Debug build only: index of the first damaged guard region of the workspace after a search with these
        parameters, -1 if all are intact (chimera_workspace_check)."""
        bad = ctypes.c_int32()
        _check(lib().chimera_workspace_check(self._h, ctypes.c_int32(n_queries), ctypes.c_int32(q_len),
                                             ctypes.c_int32(nprobe), ctypes.c_int32(n_prune), ctypes.c_int32(k),
                                             ctypes.c_int64(max_candidates), _ptr(self._ws), _stream(),
                                             ctypes.byref(bad)))
        return bad.value

    def status(self) -> int:
        """Device-side status of the last search (synchronises the current stream)."""
        st = ctypes.c_int32()
        _check(lib().chimera_workspace_status(_ptr(self._ws), _stream(), ctypes.byref(st)))
        return st.value


class GraphedSearch:
    """A search of fixed shape captured once into a CUDA graph and replayed (removes the per-kernel launch gaps of the
    ~18 small kernels of a batch-1 search).  Plumbing only: the captured work is exactly one Index.search call.
    Profiling must be off while capturing (events cannot be timed inside a graph)."""

    def __init__(self, index: "Index", n_queries: int, q_len: int, nprobe: int, n_prune: int, k: int,
                 max_candidates: int = 0, **mode):
        dev = index.device
        self.queries = torch.zeros(n_queries, q_len, index.dim, dtype=torch.float32, device=dev)
        self.ids = torch.empty(n_queries, k, dtype=torch.int32, device=dev)
        self.scores = torch.empty(n_queries, k, dtype=torch.float32, device=dev)
        self.queries[..., 0] = 1.0                       # valid unit vectors for the warm-up call
        self._index = index
        args = (nprobe, n_prune, k)
        stream = torch.cuda.Stream(device=dev)
        stream.wait_stream(torch.cuda.current_stream(dev))
        with torch.cuda.stream(stream):
            index.search(self.queries, *args, max_candidates=max_candidates, out=(self.ids, self.scores), **mode)
            stream.synchronize()
            self.graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(self.graph, stream=stream):
                index.search(self.queries, *args, max_candidates=max_candidates, out=(self.ids, self.scores), **mode)
        torch.cuda.current_stream(dev).wait_stream(stream)

    def __call__(self, queries: torch.Tensor):
        """Copy `queries` (device or pinned host tensor of the captured shape) into the static input and replay.
        Returns the static output tensors (overwritten by the next call)."""
        self.queries.copy_(queries, non_blocking=True)
        self.graph.replay()
        return self.ids, self.scores


def probes_static(score_table: torch.Tensor, nprobe: int) -> torch.Tensor:
    """Top-nprobe centroids per query token through chimera_probes_static: no workspace and no device allocation
    inside the library (its scratch is a fixed 4 MiB array in the library image).  For callers that must not allocate
    at query time; sizes beyond the built-in array raise ChimeraError(WORKSPACE_TOO_SMALL).

    score_table: [B, K, q_len] int32 CUDA tensor (centroid-major).  Returns probes [B, q_len, nprobe] int32.
    The output tensor is allocated here by torch, outside the library; pass `out=` style buffers through the C ABI
    directly if even that must be avoided."""
    assert score_table.is_cuda and score_table.dtype == torch.int32 and score_table.is_contiguous()
    B, K, q_len = score_table.shape
    out = torch.empty(B, q_len, nprobe, dtype=torch.int32, device=score_table.device)
    with torch.cuda.device(score_table.device):
        _check(lib().chimera_probes_static(_ptr(score_table), ctypes.c_int64(K), ctypes.c_int32(B),
                                           ctypes.c_int32(q_len), ctypes.c_int32(nprobe), _stream(), _ptr(out)))
    return out
