"""CPU oracle (test infrastructure only) for the placement stage of the paper's heuristic:
Section 3.2.2, Algorithm 2 (SUBGRAPH-K-PATH) and Algorithm 3 (K-PATH-MATCHING), on top of the
k-path search of oracle/kpath.py.

Plain Python.  Nothing in the product package imports this module; it shares no code with the
CUDA path.

What it computes.  The partition stage has left m - 1 cuts with transfer sizes S; node j and node
j + 1 of the sought node sequence N (m nodes, all different) are joined by cut j.  The sizes are put
into classes (the paper: as many transfer-size classes as bandwidth classes, assigned "based on the
distribution"); the classes are served from the highest down, and within a class the maximal runs
of consecutive cuts of that class, longest first.  A run of l cuts needs a path of l + 1 nodes; its
first and last node are fixed when a neighbouring run has been placed already.  For each run
Algorithm 2 sorts the link bandwidths in descending order and bisects for the largest threshold at
which the subgraph of links >= threshold (Eq. 8: the class-X links) still holds such a path among
the nodes not used yet; the path found at that threshold is written into N and its nodes are
deleted from the graph.  The k-path search is colour coding: here it runs over a list of colourings
that the caller derives from its random draws, and takes the first colouring that finds a path.

Readings where the paper is silent or inconsistent:
  * class of a size = floor(rank * classes / count) over the distinct sizes: rank = number of distinct
    sizes below it, count = number of distinct sizes (equal sizes share a class, the largest size is
    in the highest class that is used);
  * Algorithm 2 calls the classifier twice, once with a threshold that is never set: one threshold
    per bisection step, the bandwidth of the median entry of the sorted list;
  * Algorithm 3 sets the path length from the length of the list of runs and reads the end vertex
    one past the run: a run that starts at cut i and has l cuts places nodes N[i .. i + l], its
    start vertex is N[i] and its end vertex N[i + l] when they are set;
  * runs of equal length are served in order of their first cut;
  * a colour is floor(draw * k / 2^32) for a 32-bit draw and a path of k vertices;
  * a chain with no cut takes node 0;
  * if some run finds no path at any threshold the stage fails (the paper: run again with fewer
    classes; that loop is the caller's).
"""
from __future__ import annotations

from dataclasses import dataclass

from oracle import kpath

OK, INFEASIBLE = 0, 1


@dataclass
class Placement:
    status: int
    nodes: tuple       # N: node of every partition, () if the stage failed
    thresholds: tuple  # per served run, in serving order: (first cut, cuts in the run, class, threshold found)


def size_classes(sizes, n_classes: int):
    """Class 0 .. n_classes - 1 of every transfer size by its rank among the distinct sizes."""
    distinct = sorted(set(int(x) for x in sizes))
    return [distinct.index(int(x)) * n_classes // len(distinct) for x in sizes]


def find_subarrays(classes, X: int):
    """Maximal runs of consecutive cuts of class X: (first cut, number of cuts)."""
    runs, i = [], 0
    while i < len(classes):
        if classes[i] == X:
            j = i
            while j < len(classes) and classes[j] == X:
                j += 1
            runs.append((i, j - i))
            i = j
        else:
            i += 1
    return runs


def colours_for(draws_row, k: int):
    return [(int(d) * k) >> 32 for d in draws_row]


def subgraph_k_path(bw, k: int, s: int, u: int, alive, draws):
    """Algorithm 2: the largest threshold among the link bandwidths at which a path of k vertices from
    s to u (-1 = any) exists over available nodes, and the path found there; (None, []) if none."""
    n = len(bw)
    edge_list = sorted((bw[v][w] for v in range(n) for w in range(n) if v != w and bw[v][w] > 0), reverse=True)
    low, high = 0, len(edge_list)
    best_path, best_t = [], None

    def k_path(t):
        for row in draws:
            found, path = kpath.colour_coding(bw, t, k, s, u, alive, colours_for(row, k))
            if found:
                return path
        return None

    while low < high:
        median = (low + high) // 2
        result = k_path(edge_list[median])
        if result is None:
            low = median + 1
        else:
            high = median
            best_path, best_t = result, edge_list[median]
    return best_t, best_path


def k_path_matching(bw, sizes, n_classes: int, draws) -> Placement:
    """Algorithm 3: nodes for the m = len(sizes) + 1 partitions."""
    n = len(bw)
    m = len(sizes) + 1
    if m == 1:
        return Placement(OK, (0,), ())
    classes = size_classes(sizes, n_classes)
    N = [-1] * m
    used = [False] * n
    served = []
    for X in range(n_classes - 1, -1, -1):
        runs = sorted(find_subarrays(classes, X), key=lambda r: (-r[1], r[0]))
        for first, cuts in runs:
            s, u = N[first], N[first + cuts]
            alive = [not used[v] or v == s or v == u for v in range(n)]
            t, path = subgraph_k_path(bw, cuts + 1, s, u, alive, draws)
            if not path:
                return Placement(INFEASIBLE, (), tuple(served))
            N[first:first + cuts + 1] = path
            for v in path:
                used[v] = True
            served.append((first, cuts, X, t))
    return Placement(OK, tuple(N), tuple(served))
