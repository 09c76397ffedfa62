"""CPU oracle (test infrastructure only) for the inner step of the paper's placement stage:
Section 3.2.2, the threshold classifier of Eq. 8 and the K-PATH call of Algorithm 2 (the
colour-coding k-path search the paper takes from Alon, Yuster and Zwick, with the paper's fixed
start and end vertices).

Plain Python.  Nothing in the product package imports this module; it shares no code with the
CUDA path.

What it computes.  The communication graph has n nodes and a bandwidth per ordered pair.  The
classifier of Eq. 8 puts a link into class X when its bandwidth is at least the threshold t, and
into the class below otherwise; the subgraph Algorithm 2 searches keeps the class-X links.  In that
subgraph the search looks for a simple path of k vertices (k counts vertices, as in the paper) that
starts at s and ends at u when those are given, uses only nodes that are still available
(Algorithm 2 deletes the nodes of every path it has placed), and does not pass through u before its
last vertex (the paper stops a walk that reaches u early).  Colour coding: every node carries one
of k colours, and only paths whose k vertices show k different colours are looked for; a table
over (set of colours used, last vertex) finds one if it exists.  The colours are an input here:
the random draw belongs to the caller, so both sides see the same colouring.

Two functions answer the same question in two ways: `colourful_path_exists` walks every simple
path (the definition), `colour_coding` fills the table over colour sets (the algorithm).
"""
from __future__ import annotations


def classify(bw, X: int, t: int):
    """Eq. 8: class of every link under threshold t: X if bandwidth >= t, else the class below."""
    return [[(X if b >= t else X - 1) for b in row] for row in bw]


def class_subgraph(bw, t: int, alive):
    """Adjacency of the class-X subgraph: link v -> w with v != w, both available, bandwidth >= t
    (a bandwidth of 0 is no link, whatever the threshold)."""
    n = len(bw)
    return [[v != w and alive[v] and alive[w] and bw[v][w] > 0 and bw[v][w] >= t for w in range(n)]
            for v in range(n)]


def path_is_valid(path, bw, t, k, s, u, alive, colours) -> bool:
    """A returned path must be simple, k vertices long, on available nodes, over class-X links, with
    k different colours, from s to u when those are given."""
    if len(path) != k or len(set(path)) != k:
        return False
    if any(not (0 <= v < len(bw)) or not alive[v] for v in path):
        return False
    if len({colours[v] for v in path}) != k or any(colours[v] >= k for v in path):
        return False
    if s >= 0 and path[0] != s:
        return False
    if u >= 0 and path[-1] != u:
        return False
    return all(bw[a][b] > 0 and bw[a][b] >= t for a, b in zip(path, path[1:]))


def colourful_path_exists(bw, t, k, s, u, alive, colours) -> bool:
    """Every simple path of k vertices, by depth-first walk."""
    n = len(bw)
    adj = class_subgraph(bw, t, alive)

    def walk(v, used_nodes, used_colours, length):
        if length == k:
            return u < 0 or v == u
        if v == u:
            return False  # u may only be the last vertex
        for w in range(n):
            if adj[v][w] and w not in used_nodes and colours[w] < k and colours[w] not in used_colours:
                if walk(w, used_nodes | {w}, used_colours | {colours[w]}, length + 1):
                    return True
        return False

    starts = [s] if s >= 0 else range(n)
    return any(alive[v] and colours[v] < k and walk(v, {v}, {colours[v]}, 1) for v in starts)


def colour_coding(bw, t, k, s, u, alive, colours):
    """The table over colour sets: reach[C] = vertices at which a colourful path ends that uses
    exactly the colours of C.  Returns (found, path); the path is rebuilt by taking, step by step
    from the end, the lowest-numbered predecessor."""
    n = len(bw)
    adj = class_subgraph(bw, t, alive)
    full = (1 << k) - 1
    reach = [set() for _ in range(full + 1)]
    for v in range(n):
        if alive[v] and colours[v] < k and (s < 0 or v == s):
            reach[1 << colours[v]].add(v)
    for C in range(1, full + 1):  # a transition adds a colour, so sets only feed larger numbers
        for v in sorted(reach[C]):
            if v == u and C != full:
                continue  # a walk that reaches u early stops
            for w in range(n):
                if adj[v][w] and colours[w] < k and not (C >> colours[w]) & 1:
                    reach[C | (1 << colours[w])].add(w)
    ends = sorted(v for v in reach[full] if u < 0 or v == u)
    if not ends:
        return False, []
    path = [ends[0]]
    C = full
    while len(path) < k:
        v = path[-1]
        C &= ~(1 << colours[v])
        prev = min(x for x in reach[C] if adj[x][v] and not (x == u))
        path.append(prev)
    path.reverse()
    return True, path
