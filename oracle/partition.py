"""CPU oracle (test infrastructure only) for the partition stage of the paper's heuristic:
Section 3.2.1, the partition graph (vertex rule Eq. 6, edge rule Eq. 7) and Algorithm 1.

Plain Python, exact integers.  Nothing in the product package imports this module; it shares no
code with the CUDA path.

What it computes.  The chain's cut points 0..L-1 are split into contiguous, non-empty partitions.
A partition is a vertex of the partition graph when the memory of its layers is within the
capacity kappa of a compute node (Eq. 6, read as <=, like everywhere in this build; one capacity
for all nodes, the paper's homogeneous case).  Two vertices are joined by an edge when the second
starts right after the first ends (Eq. 7); the edge weighs what crosses that cut: the weight of the
first partition's last point (the paper uses the transfer-size class of the point; the caller
supplies one non-negative integer per point, raw sizes or class numbers).  A plan is a path from a
vertex that starts at point 0 to a vertex that ends at point L-1, and Algorithm 1 returns the path
with the smallest sum of edge weights, memoising, per last point of a partition, the best way on
from there.  The cut list Q is the last point of every partition but the final one, S their weights.

Where the paper is silent: among paths of equal cost the one with fewer partitions wins, then the
lexicographically smaller cut list (earlier first cut, then earlier second cut, ...).
"""
from __future__ import annotations

import sys
from dataclasses import dataclass

OK, INFEASIBLE = 0, 1


@dataclass
class Partition:
    status: int
    cost: int          # sum of the weights of the cuts; 0 with a single partition
    m: int             # number of partitions, 0 if infeasible
    cuts: tuple        # Q: last point of every partition but the final one
    sizes: tuple       # S: their weights


def vertices(mem, kappa):
    """Eq. 6: every contiguous run of points (first, last) whose memory fits."""
    L = len(mem)
    out = []
    for i in range(L):
        total = 0
        for j in range(i, L):
            total += int(mem[j])
            if total <= int(kappa):
                out.append((i, j))
    return out


def edges(verts):
    """Eq. 7: (u, v) when v starts at the point after u's last one."""
    return [(u, v) for u in verts for v in verts if v[0] == u[1] + 1]


def minsum_partition(weights, mem, kappa) -> Partition:
    """Algorithm 1 on the explicit partition graph, memoised per last point of a partition."""
    L = len(mem)
    weights = [int(x) for x in weights]
    verts = vertices(mem, kappa)
    starting_at = {}
    for v in verts:
        starting_at.setdefault(v[0], []).append(v)
    children = {u: starting_at.get(u[1] + 1, []) for u in verts}  # the edge rule of Eq. 7, by lookup
    path_from = {}  # last point of a partition -> best (cost, partitions, cuts) over its children

    def min_cost_path(v):
        """Best path that starts with vertex v: (cost, partitions, cuts) or None if no leaf is reachable."""
        if v[1] == L - 1:
            return (0, 1, ())
        last = v[1]
        if last not in path_from:
            found = [r for r in (min_cost_path(c) for c in children[v]) if r is not None]
            path_from[last] = min(found) if found else None
        best = path_from[last]
        if best is None:
            return None
        cost, parts, cuts = best
        return (cost + weights[last], parts + 1, (last,) + cuts)

    limit = sys.getrecursionlimit()
    sys.setrecursionlimit(max(limit, 4 * L + 100))
    try:
        found = [r for r in (min_cost_path(v) for v in verts if v[0] == 0) if r is not None]
    finally:
        sys.setrecursionlimit(limit)
    if not found:
        return Partition(INFEASIBLE, 0, 0, (), ())
    cost, parts, cuts = min(found)
    return Partition(OK, cost, parts, cuts, tuple(weights[c] for c in cuts))
