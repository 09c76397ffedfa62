"""Pins of the k-path oracle (oracle/kpath.py): Eq. 8's classifier and Algorithm 2's K-PATH call.

The table over colour sets is checked against the exhaustive walk over simple paths, against
hand-worked graphs, and against facts that hold for any graph: a path coloured 0..k-1 along its
vertices is found; in a complete graph a colourful path exists exactly when k different colours
are available; raising the threshold never creates a path; a found path is valid by an independent
check; without the colour constraint (k = n, all colours different) the question is the plain
Hamiltonian-path question answered by itertools.permutations."""
from __future__ import annotations

import itertools

import numpy as np

from oracle import kpath as K


def test_classifier_of_eq8():
    bw = [[0, 5, 9], [5, 0, 2], [9, 2, 0]]
    assert K.classify(bw, 3, 5) == [[2, 3, 3], [3, 2, 2], [3, 2, 2]]  # >= t is class X, below is X - 1
    adj = K.class_subgraph(bw, 5, [True] * 3)
    assert adj == [[False, True, True], [True, False, False], [True, False, False]]
    assert K.class_subgraph(bw, 0, [True, True, False])[0] == [False, True, False]  # deleted nodes, 0 = no link


def test_hand_worked_graphs():
    # a chain 0 - 1 - 2 - 3 with a chord 0 - 2; every link 10 except 2 - 3 which is 4
    n = 4
    bw = [[0] * n for _ in range(n)]
    for a, b, x in ((0, 1, 10), (1, 2, 10), (2, 3, 4), (0, 2, 10)):
        bw[a][b] = bw[b][a] = x
    alive = [True] * n
    # at threshold 4 the path 0 1 2 3 exists; coloured along the path it is found, from 0 to 3
    assert K.colour_coding(bw, 4, 4, 0, 3, alive, [0, 1, 2, 3]) == (True, [0, 1, 2, 3])
    # at threshold 5 the link 2 - 3 is class X - 1: no 4-path, but the 3-path 0 1 2 or 1 0 2
    assert K.colour_coding(bw, 5, 4, -1, -1, alive, [0, 1, 2, 3])[0] is False
    # (walking back from 2 the lowest-numbered predecessor is 0, before it 1)
    assert K.colour_coding(bw, 5, 3, -1, 2, alive, [0, 1, 2, 0]) == (True, [1, 0, 2])
    # two nodes of one colour cannot both be on the path: 1 and 2 share a colour, so no 3-path ends at 2
    assert K.colour_coding(bw, 5, 3, -1, 2, alive, [0, 1, 1, 2])[0] is False
    # the end vertex may not be passed early: from 0 to 2 with 3 vertices the only walk is 0 1 2;
    # 0 2 ... would reach the end too soon and is not continued
    assert K.colour_coding(bw, 5, 3, 0, 2, alive, [0, 1, 2, 0]) == (True, [0, 1, 2])
    assert K.colour_coding(bw, 5, 2, 0, 2, alive, [0, 1, 1, 0]) == (True, [0, 2])
    # a deleted node breaks the chain
    assert K.colour_coding(bw, 4, 4, 0, 3, [True, False, True, True], [0, 1, 2, 3])[0] is False
    # a single vertex is a 1-path
    assert K.colour_coding(bw, 99, 1, 2, 2, alive, [0, 0, 0, 0]) == (True, [2])
    assert K.colour_coding(bw, 99, 1, 1, 2, alive, [0, 0, 0, 0])[0] is False


def test_table_equals_exhaustive_walk():
    rng = np.random.default_rng(21)
    found = 0
    for trial in range(400):
        n = int(rng.integers(2, 9))
        k = int(rng.integers(1, min(n, 6) + 1))
        bw = rng.integers(0, 10, size=(n, n))
        if trial % 2:
            bw = np.triu(bw, 1) + np.triu(bw, 1).T
        bw = bw.tolist()
        t = int(rng.integers(1, 9))
        alive = [bool(x) for x in rng.random(n) < 0.85]
        colours = [int(x) for x in rng.integers(0, k, n)]
        s = int(rng.integers(0, n)) if trial % 3 == 0 else -1
        u = int(rng.integers(0, n)) if trial % 5 < 2 else -1
        want = K.colourful_path_exists(bw, t, k, s, u, alive, colours)
        got, path = K.colour_coding(bw, t, k, s, u, alive, colours)
        assert got == want, (trial, n, k, t, s, u)
        if got:
            found += 1
            assert K.path_is_valid(path, bw, t, k, s, u, alive, colours)
    assert 40 < found < 360


def test_general_facts():
    rng = np.random.default_rng(22)
    for _ in range(60):
        n = int(rng.integers(3, 8))
        bw = rng.integers(1, 10, size=(n, n)).tolist()
        alive = [True] * n
        # complete graph at threshold 1: a colourful k-path exists exactly when k colours occur
        k = int(rng.integers(2, n + 1))
        colours = [int(x) for x in rng.integers(0, k, n)]
        assert K.colour_coding(bw, 1, k, -1, -1, alive, colours)[0] == (len(set(colours)) == k)
        # all colours different and k = n: the Hamiltonian-path question
        t = int(rng.integers(3, 8))
        ident = list(range(n))
        ham = any(all(bw[a][b] >= t for a, b in zip(p, p[1:])) for p in itertools.permutations(range(n)))
        assert K.colour_coding(bw, t, n, -1, -1, alive, ident)[0] == ham
        # raising the threshold never creates a path
        lo_t, hi_t = sorted(int(x) for x in rng.integers(1, 10, 2))
        if K.colour_coding(bw, hi_t, k, -1, -1, alive, colours)[0]:
            assert K.colour_coding(bw, lo_t, k, -1, -1, alive, colours)[0]
        # a path coloured 0..k-1 along its vertices is found whatever the other colours are
        perm = [int(x) for x in rng.permutation(n)[:k]]
        planted = [int(x) for x in rng.integers(0, k, n)]
        for i, v in enumerate(perm):
            planted[v] = i
        tt = min(bw[a][b] for a, b in zip(perm, perm[1:])) if k > 1 else 1
        ok, path = K.colour_coding(bw, tt, k, perm[0], perm[-1], alive, planted)
        assert ok and K.path_is_valid(path, bw, tt, k, perm[0], perm[-1], alive, planted)
