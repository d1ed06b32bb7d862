"""Pins of the oracle's centroid graph (oracle_knn_graph) and graph search (oracle_graph_probes): hand-worked cases,
numpy on exact integers, special cases that reduce to the exhaustive top-nprobe, and the search restated from its
definition with Python sets.  No expectation comes from the function under test."""
import os

import numpy as np
import pytest

import oracle
from helpers import unit_rows

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(tag):
    with open(os.path.join(GOLDEN, "graph_handworked.txt")) as f:
        return [ln.split()[1:] for ln in f if ln.startswith(tag + " ")]


def _fx(q, c):
    """S_fx of every (query token, centroid) pair with numpy int64 (exact: 128 products below 2^44)."""
    xq = np.rint(q.astype(np.float64) * 2 ** 22).astype(np.int64)
    xc = np.rint(c.astype(np.float64) * 2 ** 22).astype(np.int64)
    return ((xq @ xc.T) + 2 ** 19) >> 20          # arithmetic shift = floor


def test_knn_graph_handworked_circle():
    ang = np.deg2rad([0, 10, 30, 65, 105, 170])
    c = np.zeros((6, 8), np.float32)
    c[:, 0], c[:, 1] = np.cos(ang), np.sin(ang)
    g = oracle.knn_graph(c, 2)
    for node, n0, n1 in _rows("knn"):
        assert g[int(node)].tolist() == [int(n0), int(n1)]


def test_knn_graph_ties_go_to_the_smaller_id_and_self_is_excluded():
    c = np.zeros((5, 8), np.float32)
    c[0, 0] = c[1, 1] = c[2, 1] = c[3, 2] = c[4, 2] = 1.0          # c1 == c2 and c3 == c4
    g = oracle.knn_graph(c, 3)
    assert g[0].tolist() == [1, 2, 3]                              # all scores 0: id order
    assert g[1].tolist() == [2, 0, 3] and g[2].tolist() == [1, 0, 3]   # the identical twin first, never itself
    assert all(i not in g[i] for i in range(5))


@pytest.mark.parametrize("K,D,R", [(50, 16, 5), (40, 128, 39), (33, 96, 1)])
def test_knn_graph_equals_numpy_sort_of_exact_integer_scores(K, D, R):
    c = unit_rows(np.random.default_rng(K + D), K, D)
    S = _fx(c, c)
    g = oracle.knn_graph(c, R)
    ids = np.arange(K)
    for i in range(K):
        order = np.lexsort((ids, -S[i]))
        order = order[order != i][:R]
        assert g[i].tolist() == order.tolist()


def _random_graph(rng, K, R):
    return np.stack([rng.choice(np.delete(np.arange(K), i), size=R, replace=False) for i in range(K)]).astype(np.int32)


def test_search_with_every_centroid_as_entry_point_is_the_exhaustive_top_nprobe():
    rng = np.random.default_rng(3)
    K, D, nprobe = 70, 32, 6
    c, q = unit_rows(rng, K, D), unit_rows(rng, 4, D)
    S = _fx(q, c)
    pr, sc, vis = oracle.graph_probes(q, c, _random_graph(rng, K, 3), nprobe, beam=nprobe, n_entries=K)
    for i in range(4):
        order = np.lexsort((np.arange(K), -S[i]))[:nprobe]
        assert pr[i].tolist() == order.tolist() and sc[i].tolist() == S[i, order].tolist()
    assert vis.all()


def test_search_of_a_connected_graph_with_an_unbounded_list_visits_everything():
    rng = np.random.default_rng(4)
    K, D, nprobe = 45, 16, 5
    c, q = unit_rows(rng, K, D), unit_rows(rng, 3, D)
    ring = np.stack([(np.arange(K) + 1) % K, (np.arange(K) - 1) % K], axis=1).astype(np.int32)
    S = _fx(q, c)
    pr, sc, vis = oracle.graph_probes(q, c, ring, nprobe, beam=K, n_entries=nprobe)
    assert vis.all()
    for i in range(3):
        assert pr[i].tolist() == np.lexsort((np.arange(K), -S[i]))[:nprobe].tolist()


def test_search_handworked_trace_with_a_local_maximum():
    s = [0.1, 0.5, 0.3, 0.2, 0.9, 0.05, 0.6, 0.4]
    c = np.zeros((8, 16), np.float32)
    for j, v in enumerate(s):
        c[j, 0], c[j, 1 + j] = v, np.sqrt(1.0 - v * v)
    q = np.zeros((1, 16), np.float32)
    q[0, 0] = 1.0
    graph = np.array([[1, 2], [0, 3], [0, 3], [1, 5], [6, 7], [3, 4], [4, 7], [4, 6]], np.int32)
    for beam, max_exp, want, n_vis in _rows("search"):
        lim = int(max_exp) if int(max_exp) else 1 << 40
        pr, sc, vis = oracle.graph_probes(q, c, graph, 1, beam=int(beam), n_entries=1, max_expansions=lim)
        assert pr[0, 0] == int(want) and int(vis.sum()) == int(n_vis), (beam, max_exp)
        assert sc[0, 0] == int(_fx(q, c)[0, int(want)])


def _search_with_sets(S_row, graph, K, n_entries, beam, max_exp, nprobe):
    """The search restated with sets: the list is the best `beam` of everything it has been offered."""
    key = lambda n: (-int(S_row[n]), n)
    visited, expanded, members = set(), set(), []
    def offer(nodes):
        nonlocal members
        fresh = [n for n in nodes if n not in visited]
        visited.update(fresh)
        members = sorted(set(members) | set(fresh), key=key)[:beam]
    for j in range(n_entries):
        offer([(j * K) // n_entries])
    done = 0
    while done < max_exp:
        todo = [n for n in members if n not in expanded]
        if not todo:
            break
        expanded.add(todo[0])
        done += 1
        offer([int(n) for n in graph[todo[0]]])
    return members[:nprobe], visited


@pytest.mark.parametrize("K,R,E,beam,nprobe,max_exp", [(60, 4, 3, 5, 2, 10 ** 9), (60, 4, 8, 8, 8, 10 ** 9),
                                                      (90, 6, 4, 16, 4, 7), (35, 2, 1, 3, 1, 10 ** 9),
                                                      (64, 8, 64, 4, 4, 2)])
def test_search_equals_its_restatement_with_sets(K, R, E, beam, nprobe, max_exp):
    rng = np.random.default_rng(K * R + E)
    D = 24
    c, q = unit_rows(rng, K, D), unit_rows(rng, 5, D)
    graph = _random_graph(rng, K, R)
    S = _fx(q, c)
    pr, sc, vis = oracle.graph_probes(q, c, graph, nprobe, beam, E, max_exp)
    for i in range(5):
        want, visited = _search_with_sets(S[i], graph, K, E, beam, max_exp, nprobe)
        assert pr[i].tolist() == want
        assert set(np.flatnonzero(vis[i]).tolist()) == visited
        assert sc[i].tolist() == [int(S[i, n]) for n in want]
        assert set(want) <= visited and len(visited) <= E + min(max_exp, K) * R


def test_search_of_the_knn_graph_finds_the_exact_probes_on_well_covered_data():
    # sanity band, not an equality: 1,024 unit vectors on the 4-sphere are dense enough for a nearest-neighbour graph to
    # be navigable, so the graph search must recover nearly all of the exhaustive top-4
    rng = np.random.default_rng(7)
    K, D = 1024, 8
    c = np.zeros((K, D), np.float32)
    c[:, :5] = unit_rows(rng, K, 5)
    q = c[rng.choice(K, 40, replace=False)] + 0.05 * rng.standard_normal((40, D)).astype(np.float32)
    q[:, 5:] = 0
    q /= np.linalg.norm(q, axis=1, keepdims=True)
    g = oracle.knn_graph(c, 16)
    pr, _, vis = oracle.graph_probes(q, c, g, 4, beam=32, n_entries=32)
    S = _fx(q, c)
    hits = sum(len(set(pr[i].tolist()) & set(np.lexsort((np.arange(K), -S[i]))[:4].tolist())) for i in range(40))
    assert hits / 160 >= 0.9
    assert vis.sum(1).max() < K // 2                    # and it scores a fraction of the centroids
