"""Pins of the greedy comparison baseline's oracle (Section 4): hand-worked walks, properties
that hold for any heuristic plan, and mutants that the fixtures must catch."""
from __future__ import annotations

import os

import numpy as np
import pytest

import oracle
from oracle import greedy
from paper_2210_12219_b200 import workloads as W
from tests.helpers import GOLDEN, make_instance


def parse_greedy_golden():
    out, cur = [], None
    for raw in open(os.path.join(GOLDEN, "hand_worked_greedy.txt")):
        line = raw.split("#")[0].strip()
        if not line:
            continue
        tok = line.split()
        if tok[0] == "instance":
            cur = {"name": tok[1], "walks": {}, "best": None}
            out.append(cur)
        elif tok[0] in ("L", "k"):
            cur[tok[0]] = int(tok[1])
        elif tok[0] in ("bits", "mem", "cap", "bw"):
            cur[tok[0]] = [int(x) for x in tok[1:]]
        elif tok[0] in ("walk", "best"):
            arrow = tok.index("->")
            rhs = tok[arrow + 1:]
            if rhs[0] in ("stuck", "none"):
                val = None
            else:
                if tok[0] == "best":
                    start, rhs = int(rhs[0]), rhs[1:]
                bar = rhs.index("|")
                beta, nseg = float(rhs[0]), int(rhs[1])
                cuts = tuple(int(x) for x in rhs[2:bar])
                nodes = tuple(int(x) for x in rhs[bar + 1:])
                assert len(cuts) == nseg - 1 and len(nodes) == nseg
                val = (beta, cuts, nodes) if tok[0] == "walk" else (start, beta, cuts, nodes)
            if tok[0] == "walk":
                cur["walks"][int(tok[1])] = val
            else:
                cur["best"] = val
    insts = []
    for c in out:
        k = c["k"]
        inst = make_instance(c["bits"], c["mem"], c["cap"], np.array(c["bw"]).reshape(k, k), c["name"])
        assert inst.L == c["L"]
        insts.append((inst, c["walks"], c["best"]))
    return insts


def test_hand_worked_walks():
    cases = parse_greedy_golden()
    assert len(cases) == 6
    for inst, walks, best in cases:
        assert sorted(walks) == list(range(inst.k))
        for start, want in walks.items():
            assert greedy.walk_from(inst, start) == want, (inst.name, start)
        got = greedy.greedy_joint(inst)
        if best is None:
            assert got.status == greedy.INFEASIBLE and got.m == 0 and np.isinf(got.beta_ms)
        else:
            assert (got.start, got.beta_ms, got.cuts, got.placement) == best, inst.name


def _random(seed, L, k):
    return W.random_small(seed, L, k, tight=(seed % 3 == 1), ties=(seed % 3 == 2),
                          dead_links=0.25 if seed % 4 == 3 else 0.0)


def test_greedy_plans_are_valid_and_never_beat_the_optimum():
    # whatever the heuristic returns is a plan of the problem: the evaluator (pinned on its own)
    # accepts it with the same beta, and the exhaustive optimum is not larger
    n_ok = n_worse = n_missed = 0
    for seed in range(120):
        L, k = 3 + seed % 6, 2 + seed % 4
        inst = _random(9000 + seed, L, k)
        got = greedy.greedy_joint(inst)
        best = oracle.bruteforce(inst)
        if got.status == greedy.OK:
            beta, flags = oracle.eval_plan(inst, got.m, got.cuts, got.placement)
            assert flags == 0 and beta == got.beta_ms
            assert best.status == oracle.OK and best.beta_ms <= got.beta_ms
            assert len(set(got.placement)) == got.m and got.placement[0] == got.start
            n_ok += 1
            n_worse += best.beta_ms < got.beta_ms
        else:
            n_missed += best.status == oracle.OK
    # the heuristic is a heuristic: it is beaten somewhere and gets stuck somewhere
    assert n_ok > 40 and n_worse > 0 and n_missed > 0


def test_every_walk_is_a_valid_plan_from_its_start_node():
    for seed in range(60):
        inst = _random(9500 + seed, 4 + seed % 5, 2 + seed % 3)
        walks = [greedy.walk_from(inst, n) for n in range(inst.k)]
        done = [(w[0], n) for n, w in enumerate(walks) if w is not None]
        for n, w in enumerate(walks):
            if w is None:
                continue
            beta, cuts, nodes = w
            assert nodes[0] == n
            b2, flags = oracle.eval_plan(inst, len(nodes), cuts, nodes)
            assert flags == 0 and b2 == beta
        got = greedy.greedy_joint(inst)
        if done:
            assert (got.beta_ms, got.start) == min(done)
        else:
            assert got.status == greedy.INFEASIBLE


def test_one_roomy_node_means_no_transfer():
    inst = make_instance([7, 9, 3], [1, 1, 1], [1, 1, 3], np.array([[0, 4, 4], [4, 0, 4], [4, 4, 0]]))
    got = greedy.greedy_joint(inst)
    assert got.plan() == (1, (), (2,)) and got.beta_ms == 0.0


@pytest.mark.parametrize("mutant", ["slowest_link", "largest_transfer", "shorter_on_tie", "ignore_used"])
def test_fixtures_catch_planted_mistakes(monkeypatch, mutant):
    # a wrong rule planted in a copy of the walk must disagree with at least one hand-worked line
    import inspect
    src = inspect.getsource(greedy.walk_from)
    swaps = {
        "slowest_link": ("bw[node][w] > bw[node][nxt]", "bw[node][w] < bw[node][nxt]"),
        "largest_transfer": ("bits[e] <= bits[chosen]", "bits[e] >= bits[chosen]"),
        "shorter_on_tie": ("bits[e] <= bits[chosen]", "bits[e] < bits[chosen]"),
        "ignore_used": ("if used[w] or bw[node][w] == 0", "if w == node or bw[node][w] == 0"),
    }
    old, new = swaps[mutant]
    assert old in src
    ns = {}
    exec(src.replace(old, new), vars(greedy).copy(), ns)
    wrong = ns["walk_from"]
    misses = 0
    for inst, walks, _ in parse_greedy_golden():
        for start, want in walks.items():
            try:
                misses += wrong(inst, start) != want
            except Exception:
                misses += 1
    assert misses > 0
