"""Helpers shared by the tests: an exact-rational plan enumerator and fixture parsing.

The enumerator is an independent statement of the problem in Python with
fractions.Fraction; it knows nothing about the oracle's C code or the CUDA library.
"""
from __future__ import annotations

import itertools
import os
from fractions import Fraction

import numpy as np

from paper_2210_12219_b200.workloads import Instance

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def make_instance(bits, mem, cap, bw, name="") -> Instance:
    bits = np.asarray(bits, dtype=np.uint64)
    mem = np.asarray(mem, dtype=np.uint64)
    cap = np.asarray(cap, dtype=np.uint64)
    k = len(cap)
    bw = np.asarray(bw, dtype=np.uint32).reshape(k, k)
    return Instance(len(bits), k, bits, mem, cap, np.ascontiguousarray(bw), name)


def plan_beta_exact(inst: Instance, cuts, nodes):
    """Exact beta of a structurally valid plan, or None when a segment does not fit or a
    link is dead.  Eq. 2 / Eq. 3 in rationals."""
    L = inst.L
    ends = list(cuts) + [L - 1]
    first = 0
    beta = Fraction(0)
    for j, last in enumerate(ends):
        need = sum(int(x) for x in inst.layer_mem_bytes[first:last + 1])
        if need > int(inst.node_mem_bytes[nodes[j]]):
            return None
        if j + 1 < len(ends):
            link = int(inst.bw_kbps[nodes[j], nodes[j + 1]])
            if link == 0:
                return None
            beta = max(beta, Fraction(int(inst.layer_out_bits[last]), link))
        first = last + 1
    return beta


def canonical_key(m, cuts, nodes):
    mask = sum(1 << n for n in nodes)
    key = [m, mask, nodes[m - 1]]
    for j in range(m - 2, -1, -1):
        key += [cuts[j], nodes[j]]
    return tuple(key)


def enumerate_optimum(inst: Instance):
    """(beta Fraction, (m, cuts, nodes)) of the canonical optimum, or (None, None)."""
    L, k = inst.L, inst.k
    best = None
    for m in range(1, min(k, L) + 1):
        for cuts in itertools.combinations(range(L - 1), m - 1):
            for nodes in itertools.permutations(range(k), m):
                b = plan_beta_exact(inst, cuts, nodes)
                if b is None:
                    continue
                cand = (b, canonical_key(m, cuts, nodes), (m, tuple(cuts), tuple(nodes)))
                if best is None or cand[:2] < best[:2]:
                    best = cand
    if best is None:
        return None, None
    return best[0], best[2]


def parse_golden(path=None):
    """Parse hand_worked_plans.txt -> (gamma_lines, [(instance, plans, optimum)])."""
    path = path or os.path.join(GOLDEN, "hand_worked_plans.txt")
    gammas, cases = [], []
    cur = None

    def val(tok):
        return float("inf") if tok == "inf" else float(tok)

    with open(path) as f:
        for raw in f:
            line = raw.split("#")[0].strip()
            if not line:
                continue
            t = line.split()
            if t[0] == "gamma":
                gammas.append((int(t[1]), int(t[2]), float(t[3])))
            elif t[0] == "instance":
                cur = {"name": t[1], "plans": [], "optimum": None}
                cases.append(cur)
            elif t[0] in ("L", "k"):
                cur[t[0]] = int(t[1])
            elif t[0] in ("bits", "mem", "cap", "bw"):
                cur[t[0]] = [int(x) for x in t[1:]]
            elif t[0] == "plan":
                bar, arrow = t.index("|"), t.index("->")
                nseg = int(t[1])
                cuts = [int(x) for x in t[2:bar]]
                nodes = [int(x) for x in t[bar + 1:arrow]]
                cur["plans"].append((nseg, cuts, nodes, val(t[arrow + 1]), int(t[arrow + 2])))
            elif t[0] == "optimum":
                bar = t.index("|")
                cur["optimum"] = (val(t[1]), int(t[2]), [int(x) for x in t[3:bar]],
                                  [int(x) for x in t[bar + 1:]])
    out = []
    for c in cases:
        inst = make_instance(c["bits"], c["mem"], c["cap"], c["bw"], c["name"])
        assert inst.L == c["L"] and inst.k == c["k"]
        out.append((inst, c["plans"], c["optimum"]))
    return gammas, out
