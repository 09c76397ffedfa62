"""Pins of the random comparison baseline's oracle (Section 4): hand-worked draws, the index rule,
validity of every plan, coverage of every valid plan, and mutants the fixtures must catch."""
from __future__ import annotations

import inspect
import itertools
import os

import numpy as np
import pytest

import oracle
from oracle import random_plans as rp
from paper_2210_12219_b200 import workloads as W
from tests.helpers import GOLDEN, make_instance


def parse_random_golden():
    out, cur = [], None
    for raw in open(os.path.join(GOLDEN, "hand_worked_random_plans.txt")):
        line = raw.split("#")[0].strip()
        if not line:
            continue
        tok = line.split()
        if tok[0] == "instance":
            cur = {"name": tok[1], "cases": []}
            out.append(cur)
        elif tok[0] in ("L", "k"):
            cur[tok[0]] = int(tok[1])
        elif tok[0] in ("bits", "mem", "cap", "bw"):
            cur[tok[0]] = [int(x) for x in tok[1:]]
        elif tok[0] == "draws":
            arrow = tok.index("->")
            draws = [int(x, 16) for x in tok[1:arrow]]
            rhs = tok[arrow + 1:]
            if rhs[0] == "none":
                want = None
            else:
                bar = rhs.index("|")
                want = (tuple(int(x) for x in rhs[1:bar]), tuple(int(x) for x in rhs[bar + 1:]))
                assert len(want[1]) == int(rhs[0]) and len(want[0]) == int(rhs[0]) - 1
            cur["cases"].append((draws, want))
    res = []
    for c in out:
        k = c["k"]
        inst = make_instance(c["bits"], c["mem"], c["cap"], np.array(c["bw"]).reshape(k, k), c["name"])
        assert all(len(d) == 2 * k for d, _ in c["cases"])
        res.append((inst, c["cases"]))
    return res


def test_hand_worked_draws():
    cases = parse_random_golden()
    assert sum(len(c) for _, c in cases) == 8
    for inst, rows in cases:
        for draws, want in rows:
            assert rp.random_plan(inst, draws) == want, (inst.name, draws)


def test_index_rule_splits_the_draws_evenly():
    # floor(d * n / 2^32): candidate j owns the draws from ceil(j * 2^32 / n) up to the next one's first
    for n in (1, 2, 3, 5, 7, 20, 1024):
        for j in range(n):
            lo = -((-j << 32) // n)
            assert rp.pick(lo, n) == j
            if j:
                assert rp.pick(lo - 1, n) == j - 1
        assert rp.pick(0, n) == 0 and rp.pick(2**32 - 1, n) == n - 1


def _draw_rows(seed, P, k):
    return np.random.default_rng(seed).integers(0, 2**32, size=(P, 2 * k), dtype=np.uint64)


def test_every_plan_is_a_plan_of_the_problem():
    n_plan = n_none = 0
    for seed in range(40):
        L, k = 3 + seed % 7, 2 + seed % 4
        inst = W.random_small(8100 + seed, L, k, tight=(seed % 3 == 1), dead_links=0.3 if seed % 2 else 0.0)
        for row in _draw_rows(seed, 25, k):
            got = rp.random_plan(inst, row)
            if got is None:
                n_none += 1
                continue
            cuts, nodes = got
            beta, flags = oracle.eval_plan(inst, len(nodes), cuts, nodes)
            assert flags in (0, oracle.PLAN_DEAD_LINK)  # distinct nodes, increasing cuts, memory fits
            n_plan += 1
    assert n_plan > 200 and n_none > 20


def test_a_grid_of_draws_reaches_exactly_the_valid_plans():
    # tiny instance: draws on a grid fine enough to hit every candidate index produce every plan the
    # evaluator accepts (dead links aside), and nothing else
    inst = make_instance([5, 9, 2, 0], [2, 3, 1, 2], [5, 4, 8], np.array([[0, 3, 1], [3, 0, 2], [1, 2, 0]]))
    L, k = inst.L, inst.k
    grid = [((2 * j + 1) << 32) // 12 for j in range(6)]  # hits every index of 1..4 candidates
    reached = set()
    for combo in itertools.product(grid, repeat=2 * k):
        got = rp.random_plan(inst, combo)
        if got is not None:
            reached.add(got)
    valid = set()
    for m in range(1, k + 1):
        for cuts in itertools.combinations(range(L - 1), m - 1):
            for nodes in itertools.permutations(range(k), m):
                _, flags = oracle.eval_plan(inst, m, cuts, nodes)
                if flags in (0, oracle.PLAN_DEAD_LINK):
                    valid.add((tuple(cuts), tuple(nodes)))
    assert reached == valid and len(valid) > 10


@pytest.mark.parametrize("mutant", ["node_among_all", "segment_off_by_one", "draws_swapped", "exclusive_memory"])
def test_fixtures_catch_planted_mistakes(mutant):
    src = inspect.getsource(rp.random_plan)
    swaps = {
        "node_among_all": ("free = [w for w in range(k) if not used[w]]", "free = list(range(k))"),
        "segment_off_by_one": ("last = fits[pick(draws[2 * step + 1], len(fits))]",
                               "last = fits[min(pick(draws[2 * step + 1], len(fits)) + 1, len(fits) - 1)]"),
        "draws_swapped": ("node = free[pick(draws[2 * step], len(free))]",
                          "node = free[pick(draws[2 * step + 1], len(free))]"),
        "exclusive_memory": ("if held > cap[node]:", "if held >= cap[node]:"),
    }
    old, new = swaps[mutant]
    assert old in src
    ns = {}
    exec(src.replace(old, new), vars(rp).copy(), ns)
    wrong = ns["random_plan"]
    misses = 0
    for inst, rows in parse_random_golden():
        for draws, want in rows:
            misses += wrong(inst, draws) != want
    assert misses > 0
