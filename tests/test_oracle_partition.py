"""Pins of the partition-stage oracle (oracle/partition.py): Section 3.2.1, Eq. 6-7, Algorithm 1.

The oracle is checked against things that are not itself: instances worked by hand, the adjacency
example the paper gives for Eq. 7, an exhaustive enumeration of every way to cut a short chain, the
textbook greedy bound on the number of partitions, monotonicity in the capacity, and planted
mistakes that must break a hand-worked line."""
from __future__ import annotations

import itertools
import os

import numpy as np
import pytest

from oracle import partition as P

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hand_worked_partitions.txt")


def golden_cases():
    out = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            w, mem, kappa, res = [x.split() for x in line.split("|")]
            res = [int(x) for x in res]
            out.append(([int(x) for x in w], [int(x) for x in mem], int(kappa[0]), res[0], res[1], tuple(res[2:])))
    return out


def enumerate_all(weights, mem, kappa):
    """Every subset of cut positions; feasibility and cost written out directly."""
    L = len(mem)
    best = None
    for r in range(L):
        for cuts in itertools.combinations(range(L - 1), r):
            bounds = [-1] + list(cuts) + [L - 1]
            if any(sum(mem[a + 1:b + 1]) > kappa for a, b in zip(bounds, bounds[1:])):
                continue
            key = (sum(weights[c] for c in cuts), r + 1, tuple(cuts))
            if best is None or key < best:
                best = key
    return best


def test_hand_worked_partitions():
    cases = golden_cases()
    assert len(cases) >= 7
    for w, mem, kappa, cost, m, cuts in cases:
        got = P.minsum_partition(w, mem, kappa)
        if m == 0:
            assert got.status == P.INFEASIBLE and got.m == 0
        else:
            assert (got.status, got.cost, got.m, got.cuts) == (P.OK, cost, m, cuts), (w, mem, kappa)
            assert got.sizes == tuple(w[c] for c in cuts)


def test_edge_rule_example_of_eq7():
    # the paper's example: P = (1, 2, 3, 4), u = [1, 2], v = [3, 4] are joined; as 0-based runs
    # u = (0, 1), v = (2, 3)
    verts = P.vertices([1, 1, 1, 1], 4)
    assert len(verts) == 10  # every contiguous run of four points
    e = P.edges(verts)
    assert ((0, 1), (2, 3)) in e
    assert ((0, 1), (3, 3)) not in e and ((0, 0), (2, 3)) not in e and ((2, 3), (0, 1)) not in e
    # a run is a vertex only when it fits (Eq. 6, inclusive)
    assert P.vertices([2, 2, 2], 4) == [(0, 0), (0, 1), (1, 1), (1, 2), (2, 2)]


def test_against_exhaustive_enumeration():
    rng = np.random.default_rng(11)
    n_inf = 0
    for trial in range(300):
        L = int(rng.integers(1, 12))
        mem = [int(x) for x in rng.integers(1, 10, L)]
        w = [int(x) for x in rng.integers(0, 6 if trial % 2 else 1000, L)]
        kappa = int(rng.integers(5, 30))
        want = enumerate_all(w, mem, kappa)
        got = P.minsum_partition(w, mem, kappa)
        if want is None:
            n_inf += 1
            assert got.status == P.INFEASIBLE
        else:
            assert (got.cost, got.m, got.cuts) == want, (w, mem, kappa)
    assert n_inf >= 5


def test_invariants_and_closed_forms():
    rng = np.random.default_rng(12)
    for _ in range(60):
        L = int(rng.integers(2, 60))
        mem = [int(x) for x in rng.integers(1, 50, L)]
        w = [int(x) for x in rng.integers(1, 10**6, L)]
        kappa = int(rng.integers(50, 200))
        got = P.minsum_partition(w, mem, kappa)
        assert got.status == P.OK
        # every partition fits, the cost is the sum over the cuts
        bounds = [-1] + list(got.cuts) + [L - 1]
        assert all(sum(mem[a + 1:b + 1]) <= kappa for a, b in zip(bounds, bounds[1:]))
        assert got.cost == sum(w[c] for c in got.cuts) and got.m == len(got.cuts) + 1
        # more capacity never costs more; enough capacity for the chain costs nothing
        assert P.minsum_partition(w, mem, kappa + 17).cost <= got.cost
        assert P.minsum_partition(w, mem, sum(mem)).cuts == ()
        # equal weights: the cost is (fewest partitions - 1) * weight, fewest partitions = greedy packing
        parts, held = 1, 0
        for x in mem:
            if held + x > kappa:
                parts, held = parts + 1, 0
            held += x
        uni = P.minsum_partition([7] * L, mem, kappa)
        assert uni.m == parts and uni.cost == 7 * (parts - 1)
        # doubling every weight doubles the cost and keeps the plan
        dbl = P.minsum_partition([2 * x for x in w], mem, kappa)
        assert dbl.cost == 2 * got.cost and dbl.cuts == got.cuts


def test_planted_mistakes_break_a_hand_worked_line(monkeypatch):
    cases = golden_cases()

    def broken(fn):
        bad = 0
        for w, mem, kappa, cost, m, cuts in cases:
            got = fn(w, mem, kappa)
            bad += (got.cost, got.m, got.cuts) != (cost, m, cuts) and m != 0
        return bad

    # exclusive memory test (< kappa instead of <=)
    assert broken(lambda w, mem, kappa: P.minsum_partition(w, mem, kappa - 1)) >= 1
    # weight of the point after the cut instead of the point before it
    assert broken(lambda w, mem, kappa: P.minsum_partition(w[1:] + [0], mem, kappa)) >= 1
    # maximum instead of sum: the min-bottleneck objective gives another plan on case B's data
    w, mem, kappa = [5, 1, 9, 4], [2, 2, 2, 2], 4
    assert P.minsum_partition(w, mem, kappa).cuts == (1,)
