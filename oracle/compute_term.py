"""CPU oracle (test infrastructure only) for the exact search under the paper's full objective,
Eq. 1: the bottleneck of a plan is the largest of the compute times of its partitions and the
transfer latencies of its cuts,   beta = max_k { c_k, gamma_k }.
(Eq. 2, which the rest of this build optimises, is Eq. 1 with the compute times dropped.)

Plain Python and numpy, binary64.  Nothing in the product package imports this module; it shares
no code with the CUDA path.

Model.  Layer i costs work[i] units of computation; node n performs speed[n] units per
millisecond.  The compute time of a partition is ONE correctly rounded division of the exact
integer sum of its layers' work by the node's speed (like gamma, Eq. 3, it is in milliseconds);
a node of speed 0 cannot compute.  Everything else is the problem of oracle/pp_oracle.c: contiguous
non-empty partitions, pairwise different nodes, memory within capacity (<=), gamma_j = bits of the
last layer before cut j over the bandwidth of the link it crosses, 0 kbps = no link.

Canonical optimum: among all plans with beta == beta*, the smallest key
(m, mask, n_m, e_{m-1}, n_{m-1}, ..., e_1, n_1), as for Eq. 2.

Two routes to the same answer: `bruteforce` walks every cut set times every injective placement
(the definition), `dp` fills the table over (used-node set, last node, last layer) with the compute
time of the segment inside the minimum (the recurrence), and walks back by the threshold rule.
"""
from __future__ import annotations

import itertools
import math
from dataclasses import dataclass

import numpy as np

OK, INFEASIBLE = 0, 1
INF = math.inf


@dataclass
class Plan:
    status: int
    beta_ms: float
    m: int
    cuts: tuple
    placement: tuple

    def plan(self):
        return (self.m, tuple(self.cuts), tuple(self.placement))


def compute_ms(work_sum: int, speed: int) -> float:
    return INF if speed == 0 else float(int(work_sum)) / float(int(speed))


def gamma_ms(bits: int, kbps: int) -> float:
    return INF if kbps == 0 else float(int(bits)) / float(int(kbps))


def eval_plan(inst, work, speed, cuts, nodes) -> float:
    """Eq. 1 for one plan (cuts = last layers of all partitions but the final one); +inf if invalid."""
    L, k = inst.L, inst.k
    m = len(nodes)
    if m < 1 or m > min(k, L) or len(cuts) != m - 1 or len(set(nodes)) != m:
        return INF
    ends = list(cuts) + [L - 1]
    if any(not (0 <= n < k) for n in nodes) or any(b <= a for a, b in zip(ends, ends[1:])) or ends[0] < 0:
        return INF
    beta, first = 0.0, 0
    for j, (last, n) in enumerate(zip(ends, nodes)):
        if sum(int(x) for x in inst.layer_mem_bytes[first:last + 1]) > int(inst.node_mem_bytes[n]):
            return INF
        beta = max(beta, compute_ms(sum(int(x) for x in work[first:last + 1]), int(speed[n])))
        if j + 1 < m:
            beta = max(beta, gamma_ms(int(inst.layer_out_bits[last]), int(inst.bw_kbps[n, nodes[j + 1]])))
        first = last + 1
    return beta


def _key(m, nodes, ends):
    mask = sum(1 << n for n in nodes)
    tail = []
    for j in range(m - 2, -1, -1):
        tail += [ends[j], nodes[j]]
    return (m, mask, nodes[m - 1], *tail)


def bruteforce(inst, work, speed) -> Plan:
    L, k = inst.L, inst.k
    best = None
    for m in range(1, min(k, L) + 1):
        for cuts in itertools.combinations(range(L - 1), m - 1):
            for nodes in itertools.permutations(range(k), m):
                b = eval_plan(inst, work, speed, cuts, nodes)
                if math.isinf(b):
                    continue
                cand = (b, _key(m, nodes, list(cuts) + [L - 1]), cuts, nodes)
                if best is None or cand[:2] < best[:2]:
                    best = cand
    if best is None:
        return Plan(INFEASIBLE, INF, 0, (), ())
    return Plan(OK, best[0], len(best[3]), tuple(best[2]), tuple(best[3]))


def dp(inst, work, speed) -> Plan:
    """dp[S][v][c] = smallest bottleneck (Eq. 1) of a partial plan that covers layers 0..c with exactly
    the nodes of S, the last partition on v ending at c, that partition's compute time included."""
    L, k = inst.L, inst.k
    M = np.concatenate([[0], np.cumsum([int(x) for x in inst.layer_mem_bytes], dtype=object)])
    Wp = np.concatenate([[0], np.cumsum([int(x) for x in work], dtype=object)])
    cap = [int(x) for x in inst.node_mem_bytes]
    gam = np.full((k, k, L), INF)
    for v in range(k):
        for w in range(k):
            if v != w:
                gam[v, w] = [gamma_ms(int(inst.layer_out_bits[c]), int(inst.bw_kbps[v, w])) for c in range(L)]
    # seg[w][c][c2] = compute time of layers c+1..c2 on w if they fit there, else +inf (c < c2)
    seg = np.full((k, L, L), INF)
    for w in range(k):
        for c2 in range(L):
            for c in range(c2):
                if M[c2 + 1] - M[c + 1] <= cap[w]:
                    seg[w, c, c2] = compute_ms(Wp[c2 + 1] - Wp[c + 1], int(speed[w]))
    table = {}
    for v in range(k):
        table[(1 << v, v)] = np.array([compute_ms(Wp[c + 1], int(speed[v])) if M[c + 1] <= cap[v] else INF
                                       for c in range(L)])
    by_pop = sorted(range(1, 1 << k), key=lambda S: (bin(S).count("1"), S))
    for S in by_pop:
        if bin(S).count("1") < 2:
            continue
        for w in range(k):
            if not (S >> w) & 1:
                continue
            P = S & ~(1 << w)
            g = np.full(L, INF)
            for v in range(k):
                if (P >> v) & 1:
                    g = np.minimum(g, np.maximum(table[(P, v)], gam[v, w]))
            # out[c2] = min over c < c2 of max(g[c], seg[w][c][c2])
            table[(S, w)] = np.maximum(g[:, None], seg[w]).min(axis=0)
    finals = [(table[(S, v)][L - 1], bin(S).count("1"), S, v) for (S, v) in table if not math.isinf(table[(S, v)][L - 1])]
    if not finals:
        return Plan(INFEASIBLE, INF, 0, (), ())
    beta, m, S, w = min(finals)
    ends, nodes, c2 = [L - 1], [w], L - 1
    for _ in range(m - 1):
        P = S & ~(1 << w)
        step = None
        for c in range(c2):
            for v in range(k):
                if (P >> v) & 1 and max(table[(P, v)][c], gam[v, w][c], seg[w, c, c2]) <= beta:
                    step = (c, v)
                    break
            if step:
                break
        c2, w, S = step[0], step[1], P
        ends.append(c2)
        nodes.append(w)
    ends.reverse()
    nodes.reverse()
    return Plan(OK, float(beta), m, tuple(ends[:-1]), tuple(nodes))
