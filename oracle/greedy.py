"""CPU oracle (test infrastructure only) for the greedy comparison baseline of Section 4
("Joint-Optimization Algorithm" in the list of algorithms the paper compares against).

Plain Python, exact integers for the memory sums and one binary64 division per transfer.
Nothing in the product package imports this module; it shares no code with the CUDA path.

What it computes (Section 4, second comparison algorithm).  A walk starts on one node and
repeats two choices until the chain is used up:
  * segment choice: among the segments that start at the next unassigned layer and fit the
    memory of the node the walk stands on, the one that sends the fewest bits onward;
  * next-node choice: among the nodes not used yet, the one reached from the current node over
    the link of highest bandwidth; the segment choice is then made there.
One walk is made from every start node, and the result is the walk with the smallest
bottleneck latency (Eq. 2).

Where the paper is silent, the readings are:
  * a segment that reaches the last layer transfers nothing, so it is taken as soon as it fits;
  * equal transfer sizes: the longer segment; equal bandwidths: the lower node index;
    equal bottlenecks: the lower start node;
  * a link of bandwidth 0 is no link; a start node whose walk gets stuck (no segment fits, no
    unused neighbour left) contributes no plan; if every start node gets stuck there is no plan.
"""
from __future__ import annotations

from dataclasses import dataclass

OK, INFEASIBLE = 0, 1


@dataclass
class GreedyPlan:
    status: int
    beta_ms: float
    m: int
    cuts: tuple
    placement: tuple
    start: int = -1

    def plan(self):
        return (self.m, tuple(self.cuts), tuple(self.placement))


def walk_from(inst, start: int):
    """One walk (segment choice, next-node choice, repeated) from one start node: (beta_ms, cuts, nodes) or None when stuck."""
    L, k = int(inst.L), int(inst.k)
    bits = [int(x) for x in inst.layer_out_bits]
    mem = [int(x) for x in inst.layer_mem_bytes]
    cap = [int(x) for x in inst.node_mem_bytes]
    bw = [[int(x) for x in row] for row in inst.bw_kbps]
    used = [False] * k
    used[start] = True
    node, first = start, 0
    cuts, nodes, beta = [], [start], 0.0
    while True:
        # segment choice: smallest outgoing transfer among the segments [first, e] that fit `node`
        chosen, held = -1, 0
        for e in range(first, L):
            held += mem[e]
            if held > cap[node]:
                break
            if e == L - 1 or chosen < 0 or bits[e] <= bits[chosen]:
                chosen = e
        if chosen < 0:
            return None
        if chosen == L - 1:
            return beta, tuple(cuts), tuple(nodes)
        # next-node choice: highest-bandwidth link from `node` to a node not used yet
        nxt = -1
        for w in range(k):
            if used[w] or bw[node][w] == 0:
                continue
            if nxt < 0 or bw[node][w] > bw[node][nxt]:
                nxt = w
        if nxt < 0:
            return None
        beta = max(beta, float(bits[chosen]) / float(bw[node][nxt]))  # Eq. 3, then Eq. 2
        cuts.append(chosen)
        nodes.append(nxt)
        used[nxt] = True
        node, first = nxt, chosen + 1


def greedy_joint(inst) -> GreedyPlan:
    """The best walk over all start nodes."""
    best = None
    for n in range(int(inst.k)):
        got = walk_from(inst, n)
        if got is not None and (best is None or got[0] < best[1][0]):
            best = (n, got)
    if best is None:
        return GreedyPlan(INFEASIBLE, float("inf"), 0, (), (), -1)
    n, (beta, cuts, nodes) = best
    return GreedyPlan(OK, beta, len(nodes), cuts, nodes, n)
