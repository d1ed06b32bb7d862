"""Comparison rules between the CUDA library's outputs and the CPU oracle's, shared by the GPU tests.

Integer / id outputs must match bit for bit.  Floating-point scores must agree within REL_TOL (1e-3 relative, the
tolerance the benchmark spec states for fp32 accumulation; the observed error is ~1e-6) plus a small absolute allowance for
scores whose terms cancel.  The final top-k ids must be the
oracle's except for swaps between documents whose scores lie within that tolerance of each other.
"""
import numpy as np

import oracle

REL_TOL = 1e-3
# A score is a sum of q_len terms of magnitude <= ~1.3 each, accumulated in fp32: when the terms cancel (score near 0) a
# purely relative bound is meaningless, so each comparison also allows q_len * 2e-6 absolute (about 16 ulp of a term).
ABS_TOL_PER_QUERY_TOKEN = 2e-6


def score_tol(ref, q_len):
    return REL_TOL * np.abs(ref) + ABS_TOL_PER_QUERY_TOKEN * q_len


def check_topk(ids_gpu, sc_gpu, res: "oracle.Result", k: int, q_len: int = 32):
    """Rule for the final ids: with tau = the oracle's k-th score and tol = score_tol(tau), every id the GPU returns
    must have an oracle score >= tau - tol, every oracle id with score > tau + tol must be returned, and each returned
    score must be within score_tol of the oracle's score for that id.  Returns the number of positions where the two
    id lists differ."""
    ids_gpu = np.asarray(ids_gpu)
    sc_gpu = np.asarray(sc_gpu)
    n_valid = int((res.ids >= 0).sum())
    assert int((ids_gpu >= 0).sum()) == n_valid
    assert np.all(ids_gpu[n_valid:] == -1) and np.all(np.isneginf(sc_gpu[n_valid:]))
    if n_valid == 0:
        return 0
    truth = dict(zip(res.pruned.tolist(), res.score4.tolist()))
    tau = float(res.scores[n_valid - 1])
    tol = float(score_tol(tau, q_len))
    got = ids_gpu[:n_valid].tolist()
    assert len(set(got)) == n_valid
    for r, d in enumerate(got):
        assert d in truth, "returned id %d is not a surviving document" % d
        assert truth[d] >= tau - tol
        assert abs(float(sc_gpu[r]) - truth[d]) <= score_tol(truth[d], q_len)
    for d, s in zip(res.ids[:n_valid].tolist(), res.scores[:n_valid].tolist()):
        if s > tau + tol:
            assert d in got
    assert np.all(np.diff(sc_gpu[:n_valid]) <= 0)
    return int((np.asarray(got) != res.ids[:n_valid]).sum())


def check_query(taps_np: dict, b: int, res: "oracle.Result", ids_gpu, sc_gpu, k: int, n_prune: int,
                table: bool = True):
    """All stages of query b of a tapped search against the oracle's pipeline result."""
    if table:
        assert np.array_equal(taps_np["score_table"][b], res.S), "score table differs"
    assert np.array_equal(taps_np["probes"][b], res.probes), "probes differ"
    n = int(taps_np["n_cand"][b])
    assert n == len(res.cand), "candidate count %d != %d" % (n, len(res.cand))
    assert np.array_equal(taps_np["cand"][b, :n], res.cand), "candidate ids differ"
    assert np.array_equal(taps_np["ci"][b, :n], res.ci), "centroid-interaction scores differ"
    m = int(taps_np["n_pruned"][b])
    assert m == len(res.pruned)
    assert np.array_equal(taps_np["pruned"][b, :m], res.pruned), "pruned ids differ"
    assert np.all(taps_np["pruned"][b, m:] == -1)
    s4 = taps_np["score4"][b]
    q_len = taps_np["probes"].shape[1]
    assert np.all(np.abs(s4[:m] - res.score4) <= score_tol(res.score4, q_len)), "stage-4 scores out of tolerance"
    assert np.all(np.isneginf(s4[m:]))
    return check_topk(ids_gpu, sc_gpu, res, k, q_len)


def taps_to_numpy(taps) -> dict:
    out = {}
    for name in ("score_table", "probes", "cand", "n_cand", "ci", "pruned", "n_pruned", "score4"):
        t = getattr(taps, name)
        if t is not None:
            out[name] = t.cpu().numpy()
    return out
