"""Pins of the Eq. 1 oracle (oracle/compute_term.py): bottleneck = max over compute times and
transfer latencies.  Checked against hand-worked plans, the exhaustive walk against the table,
the reduction to the Eq. 2 oracle (the C library, pinned on its own) when nothing costs compute,
a closed form for pure load balancing, and monotonicity."""
from __future__ import annotations

import numpy as np

import oracle
from oracle import compute_term as CT
from paper_2210_12219_b200 import workloads as W
from tests.helpers import make_instance


def _inst(bits, mem, cap, bw):
    return make_instance(np.array(bits, np.uint64), np.array(mem, np.uint64), np.array(cap, np.uint64),
                         np.array(bw, np.uint32))


def test_hand_worked_plans():
    # three layers, two nodes; node 0 does 2 units per ms, node 1 does 4; links 3000 kbps both ways
    inst = _inst([6000, 12000, 999], [1, 1, 1], [3, 3], [[0, 3000], [3000, 0]])
    work, speed = [10, 20, 30], [2, 4]
    # all on node 0: 60 / 2 = 30 ms; all on node 1: 60 / 4 = 15 ms
    assert CT.eval_plan(inst, work, speed, (), (0,)) == 30.0
    assert CT.eval_plan(inst, work, speed, (), (1,)) == 15.0
    # cut after layer 0, nodes 0 then 1: compute 10/2 = 5 and 50/4 = 12.5, transfer 6000/3000 = 2 -> 12.5
    assert CT.eval_plan(inst, work, speed, (0,), (0, 1)) == 12.5
    # cut after layer 1, nodes 1 then 0: compute 30/4 = 7.5 and 30/2 = 15, transfer 12000/3000 = 4 -> 15
    assert CT.eval_plan(inst, work, speed, (1,), (1, 0)) == 15.0
    # cut after layer 1, nodes 0 then 1: 30/2 = 15, 30/4 = 7.5, 4 -> 15
    assert CT.eval_plan(inst, work, speed, (1,), (0, 1)) == 15.0
    # invalid plans
    assert CT.eval_plan(inst, work, speed, (0,), (0, 0)) == CT.INF
    assert CT.eval_plan(inst, work, speed, (2,), (0, 1)) == CT.INF
    # optimum: (0,) on (0, 1) with 12.5; no other plan is as good
    for solve in (CT.bruteforce, CT.dp):
        got = solve(inst, work, speed)
        assert (got.beta_ms, got.plan()) == (12.5, (2, (0,), (0, 1)))
    # a slow link makes the single fast node the optimum: transfer 6000 / 100 = 60 ms
    slow = _inst([6000, 12000, 999], [1, 1, 1], [3, 3], [[0, 100], [100, 0]])
    assert CT.dp(slow, work, speed).plan() == (1, (), (1,)) and CT.dp(slow, work, speed).beta_ms == 15.0
    # a node of speed 0 cannot compute; no node can: infeasible
    assert CT.dp(inst, work, [0, 4]).plan() == (1, (), (1,))
    assert CT.dp(inst, work, [0, 0]).status == CT.INFEASIBLE == CT.bruteforce(inst, work, [0, 0]).status


def test_exhaustive_walk_equals_table():
    rng = np.random.default_rng(61)
    n_inf = 0
    for trial in range(70):
        L, k = int(rng.integers(1, 8)), int(rng.integers(1, 5))
        inst = W.random_small(61000 + trial, L, k, tight=trial % 3 == 0, ties=trial % 4 == 1,
                              dead_links=0.3 if trial % 5 == 2 else 0.0)
        work = [int(x) for x in rng.integers(0, 60, L)]
        speed = [int(x) for x in rng.integers(0 if trial % 7 == 0 else 1, 9, k)]
        if trial % 4 == 1:
            work = [int(x) * 1000 for x in rng.integers(1, 4, L)]  # many equal compute times
        a, b = CT.bruteforce(inst, work, speed), CT.dp(inst, work, speed)
        assert a.status == b.status and (a.beta_ms == b.beta_ms or a.status == CT.INFEASIBLE), trial
        assert a.plan() == b.plan(), trial
        n_inf += a.status == CT.INFEASIBLE
        if a.status == CT.OK:
            assert CT.eval_plan(inst, work, speed, a.cuts, a.placement) == a.beta_ms
    assert n_inf >= 3


def test_without_compute_cost_it_is_the_eq2_optimum():
    for trial in range(40):
        L, k = 3 + trial % 9, 2 + trial % 4
        inst = W.random_small(62000 + trial, L, k, tight=trial % 3 == 0, dead_links=0.2 if trial % 4 == 0 else 0.0)
        got = CT.dp(inst, [0] * L, [1] * k)
        want = oracle.dp_naive(inst)
        assert got.status == want.status
        if want.status == oracle.OK:
            assert got.beta_ms == want.beta_ms and got.plan() == want.plan()
    # and the compute term can only raise the optimum
    rng = np.random.default_rng(62)
    for trial in range(20):
        inst = W.random_small(62100 + trial, 8, 4)
        work = [int(x) for x in rng.integers(1, 10**6, 8)]
        speed = [int(x) for x in rng.integers(1, 50, 4)]
        with_c, without = CT.dp(inst, work, speed), oracle.dp_naive(inst)
        if with_c.status == CT.OK:
            assert with_c.beta_ms >= without.beta_ms
            faster = CT.dp(inst, work, [2 * s for s in speed])
            assert faster.beta_ms <= with_c.beta_ms  # faster nodes never hurt


def test_pure_load_balancing_closed_form():
    # nothing is transferred (bits 0), memory never binds, k identical nodes of speed s: the optimum is
    # the textbook "split a chain into at most k runs minimising the largest run", over s
    rng = np.random.default_rng(63)
    for trial in range(25):
        L, k, s = int(rng.integers(2, 9)), int(rng.integers(1, 4)), int(rng.integers(1, 7))
        work = [int(x) for x in rng.integers(1, 40, L)]
        inst = _inst([0] * L, [1] * L, [L] * k, (np.ones((k, k), int) - np.eye(k, dtype=int)) * 5)
        best = None
        for m in range(1, min(k, L) + 1):
            import itertools
            for cuts in itertools.combinations(range(L - 1), m - 1):
                ends = [-1] + list(cuts) + [L - 1]
                biggest = max(sum(work[a + 1:b + 1]) for a, b in zip(ends, ends[1:]))
                best = biggest if best is None else min(best, biggest)
        assert CT.dp(inst, work, [s] * k).beta_ms == best / s
