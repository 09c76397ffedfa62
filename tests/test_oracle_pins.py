"""Pins for the CPU oracle: everything here checks oracle/ against something that is not
itself -- numbers printed in the paper, hand-worked fixtures, an exact-rational enumerator
written independently in Python, closed forms, invariants and symmetries."""
from __future__ import annotations

import math
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2210_12219_b200 import workloads as W
from tests.helpers import (canonical_key, enumerate_optimum, make_instance, parse_golden,
                           plan_beta_exact)

INF = float("inf")


# ---------------------------------------------------------------- paper's numbers

def test_gamma_section1_example():
    # Section 1: 10.2 Mbit over a 6 Mbps link takes 1.7 s.
    assert oracle.gamma(10_200_000, 6000) == 1700.0
    assert oracle.gamma(10_200_000, 6000) / 1000.0 == 1.7
    for bits, kbps, want in parse_golden()[0]:
        assert oracle.gamma(bits, kbps) == want


def test_gamma_is_one_rounded_division():
    rng = np.random.default_rng(1)
    for _ in range(2000):
        a = int(rng.integers(1, 1 << 40))
        b = int(rng.integers(1, 1 << 24))
        assert oracle.gamma(a, b) == a / b  # Python int/int is correctly rounded
    assert oracle.gamma(123, 0) == INF


def test_gamma_order_matches_rational_order():
    # with bits < 2^25 and kbps < 2^16 distinct ratios are distinct doubles in the same order
    rng = np.random.default_rng(2)
    a = rng.integers(1, 1 << 25, size=(3000, 2))
    b = rng.integers(1, 1 << 16, size=(3000, 2))
    for (a0, a1), (b0, b1) in zip(a.tolist(), b.tolist()):
        x, y = oracle.gamma(a0, b0), oracle.gamma(a1, b1)
        lhs, rhs = a0 * b1, a1 * b0
        assert (x < y) == (lhs < rhs) and (x == y) == (lhs == rhs)


# ---------------------------------------------------------------- hand-worked fixtures

def test_hand_worked_plans_and_optima():
    _, cases = parse_golden()
    assert len(cases) == 3
    for inst, plans, optimum in cases:
        for nseg, cuts, nodes, want_beta, want_flags in plans:
            beta, flags = oracle.eval_plan(inst, nseg, cuts, nodes)
            assert flags == want_flags, (inst.name, nseg, cuts, nodes)
            assert beta == want_beta, (inst.name, nseg, cuts, nodes)
        want_beta, m, cuts, nodes = optimum
        for sol in (oracle.bruteforce(inst), oracle.dp_naive(inst), oracle.dp_fact(inst)):
            assert sol.beta_ms == want_beta
            assert sol.m == m
            assert sol.plan() == (m, tuple(cuts), tuple(nodes))
            assert sol.status == (oracle.INFEASIBLE if m == 0 else oracle.OK)
            assert (sol.cuts[max(m - 1, 0):] == -1).all() and (sol.placement[m:] == -1).all()


def test_consecutive_segments_share_a_cut():
    # Section 3.2.1 edge example: u = [1,2], v = [3,4] in P = (1,2,3,4) are adjacent, and the
    # edge carries the transfer of u's last point.  Here: cut after layer 1 moves bits[1].
    inst = make_instance([111, 222, 333, 444], [1, 1, 1, 1], [2, 2], [0, 7, 7, 0])
    beta, flags = oracle.eval_plan(inst, 2, [1], [0, 1])
    assert flags == 0 and beta == 222 / 7


# ---------------------------------------------------------------- exact enumeration

def _small_cases():
    cases = []
    seed = 0
    for L, k, n in ((1, 1, 2), (1, 3, 2), (2, 2, 6), (3, 2, 8), (4, 3, 30), (5, 3, 40),
                    (6, 4, 50), (7, 4, 40), (3, 5, 10)):
        for i in range(n):
            kind = i % 4
            cases.append(W.random_small(seed, L, k, tight=(kind == 1), ties=(kind == 2),
                                        dead_links=0.3 if kind == 3 else 0.0))
            seed += 1
    return cases


def test_oracle_matches_exact_rational_enumeration():
    cases = _small_cases()
    assert len(cases) >= 180
    n_inf = n_single = n_multi = 0
    for inst in cases:
        want_beta, want_plan = enumerate_optimum(inst)
        sols = [oracle.bruteforce(inst), oracle.dp_naive(inst), oracle.dp_fact(inst, 2)]
        for sol in sols:
            if want_plan is None:
                assert sol.status == oracle.INFEASIBLE and sol.m == 0 and sol.beta_ms == INF
            else:
                assert sol.status == oracle.OK
                assert sol.beta_ms == float(want_beta), inst.name
                assert sol.plan() == want_plan, inst.name
        if want_plan is None:
            n_inf += 1
        elif want_plan[0] == 1:
            n_single += 1
        else:
            n_multi += 1
    assert n_inf >= 5 and n_single >= 5 and n_multi >= 60


def test_larger_enumeration_few():
    for seed in range(6):
        inst = W.random_small(1000 + seed, 9, 5, tight=(seed % 2 == 1), ties=(seed % 3 == 2))
        want_beta, want_plan = enumerate_optimum(inst)
        for sol in (oracle.bruteforce(inst), oracle.dp_naive(inst), oracle.dp_fact(inst)):
            if want_plan is None:
                assert sol.status == oracle.INFEASIBLE
            else:
                assert sol.beta_ms == float(want_beta) and sol.plan() == want_plan


def test_bruteforce_equals_dp_on_tiny_config():
    inst = W.config_tiny()
    bf = oracle.bruteforce(inst)
    assert bf.plans_visited > 10_000
    for sol in (oracle.dp_naive(inst), oracle.dp_fact(inst)):
        assert sol.status == bf.status == oracle.OK
        assert sol.beta_ms == bf.beta_ms and sol.plan() == bf.plan()
    for seed in range(40):
        inst = W.random_small(2000 + seed, 10 + seed % 3, 5 + seed % 2, tight=(seed % 2 == 0),
                              ties=(seed % 5 == 0), dead_links=0.2 if seed % 7 == 0 else 0.0)
        bf, dn, df = oracle.bruteforce(inst), oracle.dp_naive(inst), oracle.dp_fact(inst, 2)
        assert bf.status == dn.status == df.status
        assert bf.beta_ms == dn.beta_ms == df.beta_ms
        assert bf.plan() == dn.plan() == df.plan()


# ---------------------------------------------------------------- closed forms

def test_two_nodes_closed_form():
    # k = 2: either one node holds everything (beta 0) or the best single cut over both orders
    for seed in range(40):
        inst = W.random_small(3000 + seed, 8, 2, tight=(seed % 2 == 0))
        mem = [int(x) for x in inst.layer_mem_bytes]
        cap = [int(x) for x in inst.node_mem_bytes]
        best = None
        if sum(mem) <= max(cap):
            best = Fraction(0)
        else:
            for c in range(inst.L - 1):
                for a, b in ((0, 1), (1, 0)):
                    if sum(mem[:c + 1]) <= cap[a] and sum(mem[c + 1:]) <= cap[b]:
                        g = Fraction(int(inst.layer_out_bits[c]), int(inst.bw_kbps[a, b]))
                        best = g if best is None or g < best else best
        sol = oracle.dp_naive(inst)
        if best is None:
            assert sol.status == oracle.INFEASIBLE
        else:
            assert sol.beta_ms == float(best)


def test_uniform_data_closed_form():
    # every layer emits T bits and every link runs at b kbps: once two segments are forced,
    # beta* = T / b no matter where the cuts fall.
    L, k, T, b = 9, 4, 7_654_321, 5432
    inst = make_instance([T] * L, [10] * L, [40, 30, 35, 25], np.full((k, k), b) - np.eye(k) * b)
    sol = oracle.dp_fact(inst)
    assert sol.beta_ms == T / b and sol.m == 3  # 90 bytes need three nodes (40 + 35 + 30)
    inst2 = make_instance([T] * L, [10] * L, [90, 30, 35, 25], inst.bw_kbps)
    assert oracle.dp_fact(inst2).beta_ms == 0.0 and oracle.dp_fact(inst2).plan() == (1, (), (0,))


def _chain_minmax(weights, mem, kappa, kmax):
    """Textbook 1-D problem: cut a chain into <= kmax chunks of <= kappa bytes minimising the
    largest cut weight.  f[c][j] = best for layers 0..c in exactly j chunks."""
    L = len(mem)
    f = [[None] * (kmax + 1) for _ in range(L)]
    for c in range(L):
        if sum(mem[:c + 1]) <= kappa:
            f[c][1] = 0
        for j in range(2, kmax + 1):
            for p in range(c):
                if f[p][j - 1] is not None and sum(mem[p + 1:c + 1]) <= kappa:
                    cand = max(f[p][j - 1], weights[p])
                    if f[c][j] is None or cand < f[c][j]:
                        f[c][j] = cand
    vals = [x for x in f[L - 1][1:] if x is not None]
    return min(vals) if vals else None


def test_homogeneous_nodes_constant_bandwidth_reduces_to_chain_partition():
    # identical nodes and links: placement is irrelevant and beta* * b is the 1-D min-max cut
    for seed in range(25):
        base = W.random_small(4000 + seed, 10, 4, tight=True)
        kappa, b = 50_000_000, 4000
        bw = np.full((4, 4), b) - np.eye(4) * b
        inst = make_instance(base.layer_out_bits, base.layer_mem_bytes, [kappa] * 4, bw)
        want = _chain_minmax([int(x) for x in inst.layer_out_bits],
                             [int(x) for x in inst.layer_mem_bytes], kappa, 4)
        sol = oracle.dp_naive(inst)
        if want is None:
            assert sol.status == oracle.INFEASIBLE
        else:
            assert sol.beta_ms == want / b


# ---------------------------------------------------------------- invariants

def _check_plan_consistency(inst, sol):
    assert sol.status == oracle.OK
    m, cuts, nodes = sol.plan()
    assert len(set(nodes)) == m  # a different device per partition (Section 1)
    exact = plan_beta_exact(inst, cuts, nodes)
    assert exact is not None and float(exact) == sol.beta_ms  # every segment fits; Eq. 2
    beta, flags = oracle.eval_plan(inst, m, cuts, nodes)
    assert flags == 0 and beta == sol.beta_ms
    if m > 1:
        gam = {oracle.gamma(int(inst.layer_out_bits[c]), int(inst.bw_kbps[v, w]))
               for c in range(inst.L) for v in range(inst.k) for w in range(inst.k) if v != w}
        assert sol.beta_ms in gam  # min/max only select values
        # Theorem 1 for the plan's own transfer sizes: beta >= max S / max E_c
        maxbw = int(inst.bw_kbps.max())
        assert sol.beta_ms >= max(int(inst.layer_out_bits[c]) for c in cuts) / maxbw
    else:
        assert sol.beta_ms == 0.0


def test_returned_plan_is_consistent_on_named_configs():
    for inst in (W.config_tiny(), W.config_resnet50_shaped(), W.config_deeper_cnn()):
        sol = oracle.dp_fact(inst, 4)
        _check_plan_consistency(inst, sol)
    # config 2's capacities force at least three segments
    assert oracle.dp_fact(W.config_resnet50_shaped()).m >= 3


def test_theorem1_bound_on_random_plans():
    inst = W.config_tiny()
    nseg, ends, nodes = W.random_plans(inst, 300, seed=5, invalid_fraction=0.0)
    maxbw = int(inst.bw_kbps.max())
    for b in range(300):
        beta, flags = oracle.eval_plan(inst, int(nseg[b]), ends[b], nodes[b])
        if flags == 0 and nseg[b] > 1:
            cut_bits = [int(inst.layer_out_bits[c]) for c in ends[b, :nseg[b] - 1]]
            assert beta >= max(cut_bits) / maxbw
        if flags == 0:
            assert beta >= oracle.dp_fact(inst).beta_ms  # nothing beats the optimum


def test_monotone_in_nodes_memory_and_bandwidth():
    for seed in range(30):
        inst = W.random_small(5000 + seed, 9, 4, tight=(seed % 2 == 0))
        base = oracle.dp_fact(inst).beta_ms
        cap2 = inst.node_mem_bytes.copy()
        cap2[seed % 4] += np.uint64(20_000_000)
        more_mem = make_instance(inst.layer_out_bits, inst.layer_mem_bytes, cap2, inst.bw_kbps)
        assert oracle.dp_fact(more_mem).beta_ms <= base
        bw2 = inst.bw_kbps.copy()
        bw2[0, 1] += 5000
        bw2[1, 0] += 5000
        faster = make_instance(inst.layer_out_bits, inst.layer_mem_bytes, inst.node_mem_bytes, bw2)
        assert oracle.dp_fact(faster).beta_ms <= base
        big = W.random_small(5000 + seed, 9, 5, tight=(seed % 2 == 0))
        bwx = big.bw_kbps.copy()
        bwx[:4, :4] = inst.bw_kbps
        capx = big.node_mem_bytes.copy()
        capx[:4] = inst.node_mem_bytes
        extra_node = make_instance(inst.layer_out_bits, inst.layer_mem_bytes, capx, bwx)
        assert oracle.dp_fact(extra_node).beta_ms <= base
        # the paper's homogeneous reading (every node at the smallest capacity) is never better
        homog = make_instance(inst.layer_out_bits, inst.layer_mem_bytes,
                              [int(inst.node_mem_bytes.min())] * 4, inst.bw_kbps)
        assert oracle.dp_fact(homog).beta_ms >= base


def test_power_of_two_scalings_are_exact():
    for seed in range(15):
        inst = W.random_small(6000 + seed, 8, 4)
        s0 = oracle.dp_fact(inst)
        twice_bits = make_instance(inst.layer_out_bits * np.uint64(2), inst.layer_mem_bytes,
                                   inst.node_mem_bytes, inst.bw_kbps)
        s1 = oracle.dp_fact(twice_bits)
        assert s1.beta_ms == 2 * s0.beta_ms and s1.plan() == s0.plan()
        twice_bw = make_instance(inst.layer_out_bits, inst.layer_mem_bytes, inst.node_mem_bytes,
                                 inst.bw_kbps * np.uint32(2))
        s2 = oracle.dp_fact(twice_bw)
        assert s2.beta_ms == s0.beta_ms / 2 and s2.plan() == s0.plan()


def test_relabelling_and_reversal_symmetry():
    rng = np.random.default_rng(7)
    for seed in range(20):
        inst = W.random_small(7000 + seed, 8, 4, tight=(seed % 2 == 0))
        base = oracle.dp_fact(inst).beta_ms
        perm = rng.permutation(4)
        relabelled = make_instance(inst.layer_out_bits, inst.layer_mem_bytes,
                                   inst.node_mem_bytes[perm], inst.bw_kbps[np.ix_(perm, perm)])
        assert oracle.dp_fact(relabelled).beta_ms == base
        # reversed chain: boundary i (between layers i and i+1) keeps its weight bits[i], so
        # the reversed chain's layer j carries old boundary L-2-j; bandwidths are transposed
        L = inst.L
        rbits = np.empty(L, dtype=np.uint64)
        rbits[:L - 1] = inst.layer_out_bits[:L - 1][::-1]
        rbits[L - 1] = 1
        rev = make_instance(rbits, inst.layer_mem_bytes[::-1].copy(), inst.node_mem_bytes,
                            inst.bw_kbps.T.copy())
        assert oracle.dp_fact(rev).beta_ms == base


def test_memory_test_is_inclusive():
    # a segment whose bytes equal the capacity fits ("within the memory capacity")
    inst = make_instance([100, 100], [10, 10], [10, 10], [0, 5, 5, 0])
    sol = oracle.dp_naive(inst)
    assert sol.status == oracle.OK and sol.beta_ms == 20.0 and sol.plan() == (2, (0,), (1, 0))  # tie: lower last node
    tight = make_instance([100, 100], [10, 11], [10, 10], [0, 5, 5, 0])
    assert oracle.dp_naive(tight).status == oracle.INFEASIBLE


def test_directed_bandwidth_reads_sender_row():
    inst = make_instance([1000, 1], [10, 10], [10, 10], [0, 4, 8, 0])
    # 0 -> 1 runs at 4 kbps, 1 -> 0 at 8 kbps: sending from node 1 is faster
    sol = oracle.dp_naive(inst)
    assert sol.beta_ms == 125.0 and sol.plan() == (2, (0,), (1, 0))


def test_more_nodes_than_layers():
    inst = W.random_small(8000, 3, 5, tight=True)
    sol = oracle.dp_naive(inst)
    want_beta, want_plan = enumerate_optimum(inst)
    assert (sol.plan() == want_plan) if want_plan else (sol.status == oracle.INFEASIBLE)
    assert sol.m <= 3


# ---------------------------------------------------------------- the two DP forms agree

def test_naive_and_factorised_tables_are_identical():
    for inst in (W.config_tiny(), W.config_resnet50_shaped(), W.random_small(9000, 11, 6, tight=True),
                 W.random_small(9001, 7, 7, dead_links=0.3)):
        a = oracle.dp_naive(inst, want_table=True)
        b = oracle.dp_fact(inst, 3, want_table=True)
        assert a.table.shape == (1 << inst.k, inst.k, inst.L)
        assert np.array_equal(a.table, b.table)
        assert a.plan() == b.plan() and a.beta_ms == b.beta_ms
        # states that cannot exist are +inf: fewer layers than segments
        for S in range(1, 1 << inst.k):
            pc = bin(S).count("1")
            for v in range(inst.k):
                if S >> v & 1:
                    assert np.isinf(a.table[S, v, :pc - 1]).all()


# ---------------------------------------------------------------- evaluator flags

def test_evaluator_flags_one_per_kind():
    inst = W.config_tiny()
    sol = oracle.dp_fact(inst)
    m, cuts, nodes = sol.plan()
    assert oracle.eval_plan(inst, m, cuts, nodes) == (sol.beta_ms, 0)
    assert oracle.eval_plan(inst, 0, [], [])[1] == oracle.PLAN_BAD_NSEG
    assert oracle.eval_plan(inst, 7, [0, 1, 2, 3, 4, 5], [0, 1, 2, 3, 4, 5, 0])[1] == oracle.PLAN_BAD_NSEG
    assert oracle.eval_plan(inst, 3, [5, 5], [0, 1, 2])[1] == oracle.PLAN_BAD_ENDS
    assert oracle.eval_plan(inst, 3, [1, 11], [0, 1, 2])[1] == oracle.PLAN_BAD_ENDS
    assert oracle.eval_plan(inst, 3, [1, 5], [0, 1, 0])[1] == oracle.PLAN_BAD_NODE
    assert oracle.eval_plan(inst, 3, [1, 5], [0, 6, 1])[1] == oracle.PLAN_BAD_NODE
    assert oracle.eval_plan(inst, 3, [5, 1], [0, 0, 1])[1] == oracle.PLAN_BAD_ENDS | oracle.PLAN_BAD_NODE
    beta, flags = oracle.eval_plan(inst, 1, [], [int(np.argmin(inst.node_mem_bytes))])
    assert flags == oracle.PLAN_MEMORY and beta == INF
    dead = make_instance(inst.layer_out_bits, inst.layer_mem_bytes, inst.node_mem_bytes,
                         inst.bw_kbps * np.uint32(0))
    beta, flags = oracle.eval_plan(dead, m, cuts, nodes)
    assert flags == oracle.PLAN_DEAD_LINK and beta == INF


def test_random_plans_against_exact_rationals():
    inst = W.random_small(9100, 10, 5, dead_links=0.15)
    nseg, ends, nodes = W.random_plans(inst, 400, seed=11, invalid_fraction=0.0)
    beta, status = oracle.eval_plans(inst, nseg, ends, nodes)
    seen_ok = 0
    for b in range(400):
        m = int(nseg[b])
        exact = plan_beta_exact(inst, list(ends[b, :m - 1]), list(nodes[b, :m]))
        if exact is None:
            assert status[b] & (oracle.PLAN_MEMORY | oracle.PLAN_DEAD_LINK) and math.isinf(beta[b])
        else:
            assert status[b] == 0 and beta[b] == float(exact)
            seen_ok += 1
    assert seen_ok >= 10
