"""GPU parity of the colour-coding k-path search (pp_kpath_colour_batch) against oracle/kpath.py.
Whether a path exists under a given colouring is unique and must match; which path is returned is
not, so the returned path is checked for validity instead."""
from __future__ import annotations

import numpy as np
import pytest

import paper_2210_12219_b200 as pp
from oracle import kpath as OK
from paper_2210_12219_b200 import build
from paper_2210_12219_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    pp.lib()


def _alive_bits(mask):
    return [bool((int(mask) >> v) & 1) for v in range(64)]


def _run_and_check(bw, kk, thr, start, end, alive, colours, exhaustive):
    found, path = pp.kpath_colour_batch(bw, kk, thr, start, end, alive, colours)
    n = bw.shape[0]
    hits = 0
    for q in range(len(thr)):
        al = _alive_bits(alive[q])[:n]
        args = (bw.tolist(), int(thr[q]), kk, int(start[q]), int(end[q]), al, colours[q].tolist())
        want = OK.colourful_path_exists(*args) if exhaustive else OK.colour_coding(*args)[0]
        assert bool(found[q]) == want, q
        if want:
            hits += 1
            assert OK.path_is_valid(path[q].tolist(), *args), (q, path[q])
        else:
            assert (path[q] == -1).all()
    return hits


def test_small_graphs_against_the_exhaustive_walk():
    rng = np.random.default_rng(31)
    total = 0
    for n, kk in ((2, 1), (3, 2), (5, 3), (7, 4), (8, 5), (8, 6), (6, 6)):
        Q = 80
        bw = rng.integers(0, 10, size=(n, n)).astype(np.uint32)
        if n % 2:
            bw = (np.triu(bw, 1) + np.triu(bw, 1).T).astype(np.uint32)
        thr = rng.integers(1, 9, Q).astype(np.uint32)
        start = np.where(rng.random(Q) < 0.4, rng.integers(0, n, Q), -1).astype(np.int32)
        end = np.where(rng.random(Q) < 0.4, rng.integers(0, n, Q), -1).astype(np.int32)
        alive = np.array([sum(1 << v for v in range(n) if rng.random() < 0.9) for _ in range(Q)], dtype=np.uint64)
        colours = rng.integers(0, kk + (1 if n > 5 else 0), size=(Q, n)).astype(np.uint8)  # some colours out of range
        total += _run_and_check(bw, kk, thr, start, end, alive, colours, exhaustive=True)
    assert total > 60


def test_paper_sized_graphs_against_the_table():
    # the paper's graphs: up to 50 devices, Shannon-capacity links (Section 4); thresholds taken from
    # the sorted list of bandwidths as Algorithm 2's binary search does; path lengths up to 13
    rng = np.random.default_rng(32)
    for n, kk in ((20, 6), (50, 9), (50, 13), (64, 11)):
        bw, _ = W.geometric_bandwidths(n, seed=n + kk, link="pairwise")
        Q = 48
        edges = np.sort(bw[np.triu_indices(n, 1)])[::-1]
        thr = edges[rng.integers(0, len(edges), Q)].astype(np.uint32)
        start = np.where(rng.random(Q) < 0.3, rng.integers(0, n, Q), -1).astype(np.int32)
        end = np.where(rng.random(Q) < 0.3, rng.integers(0, n, Q), -1).astype(np.int32)
        alive = np.array([sum(1 << v for v in range(n) if rng.random() < 0.9) for _ in range(Q)], dtype=np.uint64)
        colours = rng.integers(0, kk, size=(Q, n)).astype(np.uint8)
        hits = _run_and_check(bw, kk, thr, start, end, alive, colours, exhaustive=False)
        assert 0 < hits < Q


def test_binary_search_over_the_threshold_and_limits():
    # Algorithm 2: the largest threshold for which some colouring finds a path, by bisection over the
    # sorted bandwidths, every probe a batch of colourings; the same bisection on the oracle
    rng = np.random.default_rng(33)
    n, kk, trials = 16, 5, 24
    bw, _ = W.geometric_bandwidths(n, seed=5, link="pairwise")
    edges = np.sort(np.unique(bw[np.triu_indices(n, 1)]))[::-1]
    colours = rng.integers(0, kk, size=(trials, n)).astype(np.uint8)
    alive = np.full(trials, (1 << n) - 1, dtype=np.uint64)
    anyv = np.full(trials, -1, dtype=np.int32)

    def gpu_probe(t):
        return bool(pp.kpath_colour_batch(bw, kk, np.full(trials, t, np.uint32), anyv, anyv, alive, colours)[0].any())

    def cpu_probe(t):
        return any(OK.colour_coding(bw.tolist(), int(t), kk, -1, -1, [True] * n, colours[i].tolist())[0]
                   for i in range(trials))

    def bisect(probe):
        low, high, best = 0, len(edges), None
        while low < high:
            mid = (low + high) // 2
            if probe(edges[mid]):
                high, best = mid, int(edges[mid])
            else:
                low = mid + 1
        return best

    assert bisect(gpu_probe) == bisect(cpu_probe) is not None
    # limits and empty input
    with pytest.raises(pp.PPError):
        pp.kpath_colour_batch(np.zeros((65, 65), np.uint32), 3, np.ones(1, np.uint32), anyv[:1], anyv[:1], alive[:1],
                              np.zeros((1, 65), np.uint8))
    with pytest.raises(pp.PPError):
        pp.kpath_colour_batch(bw, 14, np.ones(1, np.uint32), anyv[:1], anyv[:1], alive[:1], np.zeros((1, n), np.uint8))
    f, p = pp.kpath_colour_batch(bw, 3, np.zeros(0, np.uint32), anyv[:0], anyv[:0], alive[:0], np.zeros((0, n), np.uint8))
    assert f.shape == (0,) and p.shape == (0, 3)
