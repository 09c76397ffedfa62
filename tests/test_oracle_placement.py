"""Pins of the placement-stage oracle (oracle/placement.py): Algorithm 2 and Algorithm 3.

With every possible colouring among the trials colour coding is exhaustive, so the threshold that
Algorithm 2's bisection finds must be the widest bottleneck over all simple paths (permutations),
and with one class and one run Algorithm 3 must place the chain on the best such path.  Two
instances are worked by hand; general facts hold for every result."""
from __future__ import annotations

import itertools

import numpy as np

from oracle import placement as P


def all_colourings(n, k):
    """Draws whose colours for a path of k vertices run through all k^n colourings of n nodes."""
    first = [-(-(c << 32) // k) for c in range(k)]  # smallest draw that maps to colour c
    rows = [[first[c] for c in combo] for combo in itertools.product(range(k), repeat=n)]
    for row, combo in zip(rows[:5], itertools.product(range(k), repeat=n)):
        assert P.colours_for(row, k) == list(combo)
    return rows


def widest_path(bw, k, s, u, alive):
    """max over simple paths of k available vertices (from s to u when given) of the smallest link."""
    n = len(bw)
    best = None
    for p in itertools.permutations([v for v in range(n) if alive[v]], k):
        if (s >= 0 and p[0] != s) or (u >= 0 and p[-1] != u):
            continue
        links = [bw[a][b] for a, b in zip(p, p[1:])]
        if any(x == 0 for x in links):
            continue
        width = min(links) if links else None
        if k == 1:
            return "single"
        if best is None or width > best:
            best = width
    return best


def test_classes_and_runs():
    assert P.size_classes([9, 1], 2) == [1, 0]
    assert P.size_classes([1, 9, 9], 2) == [0, 1, 1]
    assert P.size_classes([5, 5, 5], 3) == [0, 0, 0]
    assert P.size_classes([10, 20, 30, 40], 2) == [0, 0, 1, 1]
    assert P.size_classes([10, 20, 30, 40], 4) == [0, 1, 2, 3]
    assert P.size_classes([10, 20, 30], 20) == [0, 6, 13]
    assert P.find_subarrays([1, 1, 0, 1, 0, 0], 1) == [(0, 2), (3, 1)]
    assert P.find_subarrays([1, 1, 0, 1, 0, 0], 0) == [(2, 1), (4, 2)]
    assert P.find_subarrays([2, 2], 1) == []
    assert P.colours_for([0, 2**31, 2**32 - 1, 2**30], 4) == [0, 2, 3, 1]


def test_hand_worked_matchings():
    bw = [[0, 5, 9, 2], [5, 0, 4, 7], [9, 4, 0, 3], [2, 7, 3, 0]]
    draws = all_colourings(4, 2)
    # two cuts, sizes 9 and 1, two classes: the large cut goes on the widest link 0 - 2 (the path ends at
    # the lower vertex: N = 2, 0), then from node 0 the best link to an unused node is 0 - 1 (5, not 2)
    got = P.k_path_matching(bw, [9, 1], 2, draws)
    assert got.status == P.OK and got.nodes == (2, 0, 1)
    assert got.thresholds == ((0, 1, 1, 9), (1, 1, 0, 5))
    # the other way round the small cut comes second and is anchored at its right end: N[1] = 2, N[2] = 0
    # first; then a link into node 2 from an unused node: 1 -> 2 (4) beats 3 -> 2 (3)
    got = P.k_path_matching(bw, [1, 9], 2, draws)
    assert got.nodes == (1, 2, 0) and got.thresholds == ((1, 1, 1, 9), (0, 1, 0, 4))
    # one class: both cuts form one run of three nodes; widest 3-path: 1 - 3? no: 2 - 0 - 1 has width 5,
    # 0 - 2 - 1 width 4, 3 - 1 - 0 width 5, 1 - 0 - 2 width 5: the bisection stops at 5
    got = P.k_path_matching(bw, [9, 1], 1, all_colourings(4, 3))
    assert got.thresholds == ((0, 2, 0, 5),) and min(bw[a][b] for a, b in zip(got.nodes, got.nodes[1:])) == 5
    # no cut: node 0; more partitions than nodes: the stage fails
    assert P.k_path_matching(bw, [], 3, draws).nodes == (0,)
    assert P.k_path_matching(bw, [1, 1, 1, 1], 1, all_colourings(4, 5)).status == P.INFEASIBLE


def test_bisection_finds_the_widest_path():
    rng = np.random.default_rng(41)
    for trial in range(120):
        n = int(rng.integers(2, 6))
        k = int(rng.integers(2, min(n, 4) + 1))
        bw = rng.integers(0, 9, size=(n, n))
        if trial % 2:
            bw = np.triu(bw, 1) + np.triu(bw, 1).T
        bw = bw.tolist()
        alive = [bool(x) for x in rng.random(n) < 0.9]
        s = int(rng.integers(0, n)) if trial % 3 == 0 else -1
        u = int(rng.integers(0, n)) if trial % 4 == 0 else -1
        if s >= 0:
            alive[s] = True
        if u >= 0:
            alive[u] = True
        t, path = P.subgraph_k_path(bw, k, s, u, alive, all_colourings(n, k))
        want = widest_path(bw, k, s, u, alive)
        assert t == want, (trial, bw, k, s, u, alive)
        if t is not None:
            assert len(path) == k and len(set(path)) == k and all(alive[v] for v in path)
            assert (s < 0 or path[0] == s) and (u < 0 or path[-1] == u)
            assert min(bw[a][b] for a, b in zip(path, path[1:])) == t  # the bottleneck link is the threshold


def test_matching_facts():
    rng = np.random.default_rng(42)
    ok = 0
    for trial in range(60):
        n = int(rng.integers(4, 8))
        cuts = int(rng.integers(1, min(n - 1, 4) + 1))
        bw = rng.integers(1, 50, size=(n, n))
        bw = (np.triu(bw, 1) + np.triu(bw, 1).T).tolist()
        sizes = [int(x) for x in rng.integers(1, 100, cuts)]
        n_classes = int(rng.integers(1, 4))
        draws = rng.integers(0, 2**32, size=(40, n), dtype=np.uint64).tolist()
        got = P.k_path_matching(bw, sizes, n_classes, draws)
        if got.status != P.OK:
            continue
        ok += 1
        assert len(got.nodes) == cuts + 1 and len(set(got.nodes)) == cuts + 1
        classes = P.size_classes(sizes, n_classes)
        for first, run, X, t in got.thresholds:
            assert all(classes[first + i] == X for i in range(run))
            assert all(bw[got.nodes[first + i]][got.nodes[first + i + 1]] >= t for i in range(run))
        # the highest class is served first, every cut belongs to exactly one served run
        assert got.thresholds[0][2] == max(classes)
        assert sorted(c for first, run, _, _ in got.thresholds for c in range(first, first + run)) == list(range(cuts))
        # one class, one run, exhaustive colourings: the chain sits on a widest path
        if cuts <= 3 and n <= 5:
            ex = P.k_path_matching(bw, sizes, 1, all_colourings(n, cuts + 1))
            assert ex.thresholds[0][3] == widest_path(bw, cuts + 1, -1, -1, [True] * n)
    assert ok > 40
