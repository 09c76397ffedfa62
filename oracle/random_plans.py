"""CPU oracle (test infrastructure only) for the random comparison baseline of Section 4
("Random Algorithm" in the list of algorithms the paper compares against): choose a random node
and a random segment that the node can hold, until the chain is used up.

Plain Python on exact integers.  Nothing in the product package imports this module; it shares no
code with the CUDA path.  The random numbers are inputs: 2 k draws of 32 bits per plan, draw 2 s
choosing the node of step s and draw 2 s + 1 its segment.

Where the paper is silent, the readings are:
  * both choices are uniform: the node among the nodes not used yet, the segment among those that
    start at the next unassigned layer and fit the node's memory (by their last layer);
  * a draw d picks index floor(d * n / 2^32) among n candidates listed in ascending order;
  * bandwidths play no part (the plan is scored afterwards, Eq. 2; over a missing link it scores
    +inf);
  * there is no plan when the chosen node holds not even the next layer, or when all k nodes are
    used and layers are left over.
"""
from __future__ import annotations


def pick(draw: int, n: int) -> int:
    """Index in [0, n) from a 32-bit draw."""
    return (int(draw) * int(n)) >> 32


def random_plan(inst, draws):
    """(cuts, nodes) of one random plan, or None; `draws` holds 2 k integers in [0, 2^32)."""
    L, k = int(inst.L), int(inst.k)
    mem = [int(x) for x in inst.layer_mem_bytes]
    cap = [int(x) for x in inst.node_mem_bytes]
    used = [False] * k
    first, cuts, nodes = 0, [], []
    for step in range(k):
        free = [w for w in range(k) if not used[w]]
        node = free[pick(draws[2 * step], len(free))]
        fits, held = [], 0
        for e in range(first, L):
            held += mem[e]
            if held > cap[node]:
                break
            fits.append(e)
        if not fits:
            return None
        last = fits[pick(draws[2 * step + 1], len(fits))]
        used[node] = True
        nodes.append(node)
        if last == L - 1:
            return tuple(cuts), tuple(nodes)
        cuts.append(last)
        first = last + 1
    return None


def random_plans(inst, draws):
    """Rows shaped like the batched evaluator's inputs: (nseg [P], ends [P][k], nodes [P][k]) as lists;
    nseg = 0 and rows of -1 where there is no plan.  `draws` is [P][2 k]."""
    k = int(inst.k)
    nseg, ends, nodes = [], [], []
    for row in draws:
        got = random_plan(inst, [int(x) for x in row])
        c, n = got if got is not None else ((), ())
        nseg.append(len(n))
        ends.append(list(c) + [-1] * (k - len(c)))
        nodes.append(list(n) + [-1] * (k - len(n)))
    return nseg, ends, nodes
