"""CPU oracle: ctypes front end of `chimera_oracle.c` (test infrastructure only).

The oracle is the parity reference of the CUDA library.  It is independent of it: nothing here imports the CUDA
package, and the CUDA package never imports this.  Only tests, the smoke check and the benchmark's CPU-baseline leg
may use it.

`pipeline()` chains the stage functions for one query and returns every intermediate result, in the order
score table -> probes -> candidates -> centroid-interaction scores -> pruned ids -> residual-decode scores -> top-k.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "chimera_oracle.c")
_LIB = os.path.join(_HERE, "libchimera_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain -O2, no -march flags, no OpenMP)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_candidates.restype = ctypes.c_int64
        _lib.oracle_prune.restype = ctypes.c_int64
        _lib.oracle_chamfer.restype = ctypes.c_double
        _lib.oracle_recall.restype = ctypes.c_double
        _lib.oracle_graph_probes.restype = ctypes.c_int64
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _arr(a, dtype) -> np.ndarray:
    if hasattr(a, "detach"):
        a = a.detach().cpu().numpy()
    return np.ascontiguousarray(a, dtype=dtype)


@dataclass
class Index:
    """Host copies of the index arrays, as the oracle reads them."""
    dim: int
    nbits: int
    res_lo: float
    res_hi: float
    centroids: np.ndarray   # [K, D] float32
    cids: np.ndarray        # [T] int32
    codes: np.ndarray       # [T, D*nbits/8] uint8
    doclens: np.ndarray     # [N] int32
    doc_off: np.ndarray     # [N+1] int64

    @property
    def K(self):
        return self.centroids.shape[0]

    @property
    def N(self):
        return self.doclens.shape[0]


def make_index(centroids, cids, codes, doclens, nbits: int, res_lo: float = -0.25, res_hi: float = 0.25) -> Index:
    centroids = _arr(centroids, np.float32)
    doclens = _arr(doclens, np.int32)
    doc_off = np.zeros(doclens.shape[0] + 1, dtype=np.int64)
    np.cumsum(doclens, out=doc_off[1:])
    return Index(centroids.shape[1], nbits, float(res_lo), float(res_hi), centroids, _arr(cids, np.int32),
                 _arr(codes, np.uint8), doclens, doc_off)


def score_table(q, centroids) -> np.ndarray:
    """O-1: [K, nq] int32 Q.24 fixed-point inner products (centroid-major)."""
    q = _arr(q, np.float32)
    c = _arr(centroids, np.float32)
    S = np.empty((c.shape[0], q.shape[0]), dtype=np.int32)
    lib().oracle_score_table(_p(q), ctypes.c_int32(q.shape[0]), _p(c), ctypes.c_int64(c.shape[0]),
                             ctypes.c_int32(c.shape[1]), _p(S))
    return S


def probes(S: np.ndarray, nprobe: int) -> np.ndarray:
    """O-2: [nq, nprobe] int32, best first."""
    S = _arr(S, np.int32)
    K, nq = S.shape
    assert 1 <= nprobe <= K
    out = np.empty((nq, nprobe), dtype=np.int32)
    lib().oracle_probes(_p(S), ctypes.c_int32(nq), ctypes.c_int64(K), ctypes.c_int32(nprobe), _p(out))
    return out


def candidates(pr: np.ndarray, ix: Index) -> np.ndarray:
    """O-3: ascending int32 ids of the candidate documents."""
    pr = _arr(pr, np.int32)
    cand = np.empty(ix.N, dtype=np.int32)
    n = lib().oracle_candidates(_p(pr), ctypes.c_int32(pr.size), ctypes.c_int64(ix.K), _p(ix.cids), _p(ix.doclens),
                                ctypes.c_int64(ix.N), _p(cand))
    return cand[:n].copy()


def ci_scores(S: np.ndarray, cand: np.ndarray, ix: Index) -> np.ndarray:
    """O-4a: int32 centroid-interaction score of every candidate."""
    S = _arr(S, np.int32)
    cand = _arr(cand, np.int32)
    ci = np.empty(cand.shape[0], dtype=np.int32)
    lib().oracle_ci(_p(S), ctypes.c_int32(S.shape[1]), _p(cand), ctypes.c_int64(cand.shape[0]), _p(ix.cids),
                    _p(ix.doc_off), _p(ci))
    return ci


def prune(cand: np.ndarray, ci: np.ndarray, n_prune: int) -> np.ndarray:
    """O-4b: ascending ids of the n_prune candidates with the largest CI."""
    cand = _arr(cand, np.int32)
    ci = _arr(ci, np.int32)
    out = np.empty(max(1, min(n_prune, cand.shape[0])), dtype=np.int32)
    n = lib().oracle_prune(_p(cand), _p(ci), ctypes.c_int64(cand.shape[0]), ctypes.c_int64(n_prune), _p(out))
    return out[:n].copy()


def partial_scores(S: np.ndarray, q, pr: np.ndarray, cand: np.ndarray, ix: Index) -> np.ndarray:
    """O-8: int32 partial score F' (Algorithm 2) of every candidate, from the retrieved tokens only."""
    S = _arr(S, np.int32)
    q = _arr(q, np.float32)
    pr = _arr(pr, np.int32)
    cand = _arr(cand, np.int32)
    out = np.empty(cand.shape[0], dtype=np.int32)
    lib().oracle_partial_scores(_p(S), _p(q), ctypes.c_int32(q.shape[0]), ctypes.c_int32(ix.dim),
                                ctypes.c_int32(ix.nbits), ctypes.c_float(ix.res_lo), ctypes.c_float(ix.res_hi),
                                _p(pr), ctypes.c_int32(pr.shape[1]), _p(ix.cids), _p(ix.codes), _p(ix.doclens),
                                ctypes.c_int64(ix.N), _p(cand), ctypes.c_int64(cand.shape[0]), _p(out))
    return out


@dataclass
class RabitqCodes:
    """RaBitQ 1-bit codes of the corpus tokens (Sec. 2.2), as the oracle reads them."""
    rotation: np.ndarray   # [D, D] float32
    bits: np.ndarray       # [T, D/8] uint8
    inv_dot: np.ndarray    # [T] float32


def make_rabitq(rotation, bits, inv_dot) -> RabitqCodes:
    return RabitqCodes(_arr(rotation, np.float32), _arr(bits, np.uint8), _arr(inv_dot, np.float32))


def rotate(rotation, q) -> np.ndarray:
    """O-9: q_p = P q per row, as a sequential fp32 fma chain."""
    P = _arr(rotation, np.float32)
    q = _arr(q, np.float32)
    out = np.empty_like(q)
    lib().oracle_rotate(_p(P), _p(q), ctypes.c_int64(q.shape[0]), ctypes.c_int32(q.shape[1]), _p(out))
    return out


def rabitq_score_docs(qp, docs, ix: Index, rq: RabitqCodes) -> np.ndarray:
    """O-9: complete 1-bit Chamfer score of each listed document (qp = rotated query)."""
    qp = _arr(qp, np.float32)
    docs = _arr(docs, np.int32)
    out = np.empty(docs.shape[0], dtype=np.float32)
    lib().oracle_rabitq_score_docs(_p(qp), ctypes.c_int32(qp.shape[0]), ctypes.c_int32(ix.dim), _p(rq.bits),
                                   _p(rq.inv_dot), _p(ix.doc_off), _p(docs), ctypes.c_int64(docs.shape[0]), _p(out))
    return out


def rabitq_partial(qp, pr, cand, ix: Index, rq: RabitqCodes) -> np.ndarray:
    """O-9: float32 partial score F' (Algorithm 2 with the 1-bit estimate) of every candidate."""
    qp = _arr(qp, np.float32)
    pr = _arr(pr, np.int32)
    cand = _arr(cand, np.int32)
    out = np.empty(cand.shape[0], dtype=np.float32)
    lib().oracle_rabitq_partial(_p(qp), ctypes.c_int32(qp.shape[0]), ctypes.c_int32(ix.dim), _p(rq.bits),
                                _p(rq.inv_dot), _p(pr), ctypes.c_int32(pr.shape[1]), _p(ix.cids), _p(ix.doclens),
                                ctypes.c_int64(ix.N), ctypes.c_int64(ix.K), _p(cand), ctypes.c_int64(cand.shape[0]),
                                _p(out))
    return out


def knn_graph(centroids, degree: int) -> np.ndarray:
    """O-10: [K, degree] int32 nearest-neighbour graph over the centroids (best first, self excluded)."""
    c = _arr(centroids, np.float32)
    K, D = c.shape
    assert 1 <= degree <= K - 1
    g = np.empty((K, degree), dtype=np.int32)
    lib().oracle_knn_graph(_p(c), ctypes.c_int64(K), ctypes.c_int32(D), ctypes.c_int32(degree), _p(g))
    return g


def graph_probes(q, centroids, graph: np.ndarray, nprobe: int, beam: int, n_entries: int, max_expansions: int = 1 << 40):
    """O-10: best-first search of the centroid graph for every query token of q [nq, D].
    Returns (probes [nq, nprobe] int32, scores [nq, nprobe] int32, visited [nq, K] bool)."""
    q = _arr(q, np.float32)
    c = _arr(centroids, np.float32)
    g = _arr(graph, np.int32)
    K, D = c.shape
    assert nprobe <= beam and nprobe <= n_entries <= K and g.shape[0] == K
    nq = q.shape[0]
    pr = np.empty((nq, nprobe), dtype=np.int32)
    sc = np.empty((nq, nprobe), dtype=np.int32)
    vis = np.empty((nq, K), dtype=np.uint8)
    for i in range(nq):
        lib().oracle_graph_probes(_p(q[i]), _p(c), ctypes.c_int64(K), ctypes.c_int32(D), _p(g), ctypes.c_int32(g.shape[1]),
                                  ctypes.c_int32(n_entries), ctypes.c_int32(beam), ctypes.c_int64(max_expansions),
                                  ctypes.c_int32(nprobe), _p(pr[i]), _p(sc[i]), _p(vis[i]))
    return pr, sc, vis.astype(bool)


def pipeline_rabitq(q, ix: Index, rq: RabitqCodes, nprobe: int, k_refine: int, k: int, probes_override=None) -> "Result":
    """The paper's GPU pipeline on 1-bit codes (Algorithm 1 without its CPU half): centroid probes and candidates as
    usual, candidate refinement by partial 1-bit scores, complete 1-bit scores of the survivors, top-k.  `ci` holds
    F' (float32); ordering floats >= 0 equals ordering their bit patterns, so O-4b selects on the int32 view.
    probes_override: the probes of a graph search (O-10) in place of the exhaustive top-nprobe."""
    S = score_table(q, ix.centroids)
    pr = probes(S, nprobe) if probes_override is None else _arr(probes_override, np.int32)
    cand = candidates(pr, ix)
    qp = rotate(rq.rotation, q)
    fp = rabitq_partial(qp, pr, cand, ix, rq)
    pruned = prune(cand, fp.view(np.int32), k_refine)
    s4 = rabitq_score_docs(qp, pruned, ix, rq)
    ids, sc = topk(pruned, s4, k)
    return Result(S, pr, cand, fp, pruned, s4, ids, sc)


def score_docs(q, docs: np.ndarray, ix: Index) -> np.ndarray:
    """O-5: float32 Chamfer score of each listed document on its decoded tokens."""
    q = _arr(q, np.float32)
    docs = _arr(docs, np.int32)
    out = np.empty(docs.shape[0], dtype=np.float32)
    lib().oracle_score_docs(_p(q), ctypes.c_int32(q.shape[0]), ctypes.c_int32(ix.dim), ctypes.c_int32(ix.nbits),
                            ctypes.c_float(ix.res_lo), ctypes.c_float(ix.res_hi), _p(ix.centroids), _p(ix.cids),
                            _p(ix.codes), _p(ix.doc_off), _p(docs), ctypes.c_int64(docs.shape[0]), _p(out))
    return out


def topk(docs: np.ndarray, scores: np.ndarray, k: int):
    """O-6: (ids[k] int32, scores[k] float32), best first, padded with (-1, -inf)."""
    docs = _arr(docs, np.int32)
    scores = _arr(scores, np.float32)
    ids = np.empty(k, dtype=np.int32)
    sc = np.empty(k, dtype=np.float32)
    lib().oracle_topk(_p(docs), _p(scores), ctypes.c_int64(docs.shape[0]), ctypes.c_int32(k), _p(ids), _p(sc))
    return ids, sc


def chamfer(q, v) -> float:
    """Def. 1 on raw vectors."""
    q = _arr(q, np.float32)
    v = _arr(v, np.float32)
    return float(lib().oracle_chamfer(_p(q), ctypes.c_int32(q.shape[0]), _p(v), ctypes.c_int64(v.shape[0]),
                                      ctypes.c_int32(q.shape[1])))


def recall(truth: np.ndarray, got: np.ndarray) -> float:
    """Def. 3."""
    truth = _arr(truth, np.int32)
    got = _arr(got, np.int32)
    assert truth.shape == got.shape
    return float(lib().oracle_recall(_p(truth), _p(got), ctypes.c_int32(truth.shape[0])))


def exhaustive(q, ix: Index, k: int):
    """O-7: score every document (O-5) and take the top-k (O-6): the ground truth for Recall@k."""
    docs = np.arange(ix.N, dtype=np.int32)
    sc = score_docs(q, docs, ix)
    ids, top = topk(docs, sc, k)
    return ids, top, sc


@dataclass
class Result:
    S: np.ndarray          # [K, nq] int32
    probes: np.ndarray     # [nq, nprobe] int32
    cand: np.ndarray       # ascending int32
    ci: np.ndarray         # int32, aligned with cand
    pruned: np.ndarray     # ascending int32
    score4: np.ndarray     # float32, aligned with pruned
    ids: np.ndarray        # [k] int32
    scores: np.ndarray     # [k] float32


def pipeline(q, ix: Index, nprobe: int, n_prune: int, k: int, partial: bool = False) -> Result:
    """All stages for one query [nq, D].  partial=True prunes with the paper's partial scores F' (Algorithm 2) instead
    of the full centroid interaction; `ci` then holds F'."""
    S = score_table(q, ix.centroids)
    pr = probes(S, nprobe)
    cand = candidates(pr, ix)
    ci = partial_scores(S, q, pr, cand, ix) if partial else ci_scores(S, cand, ix)
    pruned = prune(cand, ci, n_prune)
    s4 = score_docs(q, pruned, ix)
    ids, sc = topk(pruned, s4, k)
    return Result(S, pr, cand, ci, pruned, s4, ids, sc)
