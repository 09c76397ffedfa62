"""GPU parity of the placement stage (pp_kpath_matching: Algorithms 2 and 3 on top of the k-path
kernel) against oracle/placement.py, and the paper's whole heuristic end to end: partition stage,
placement stage, bottleneck latency of the result against the exact optimum and Theorem 1's bound.
The colourings are the same on both sides and both take the first colouring that finds a path and
rebuild it by the same rule, so the node sequences are compared exactly."""
from __future__ import annotations

import numpy as np
import pytest

import oracle
import paper_2210_12219_b200 as pp
from oracle import partition as OP
from oracle import placement as OPL
from paper_2210_12219_b200 import build
from paper_2210_12219_b200 import workloads as W
from tests.helpers import make_instance

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    pp.lib()


def test_matching_equals_the_oracle():
    rng = np.random.default_rng(51)
    n_ok = n_fail = 0
    for trial in range(40):
        n = int(rng.integers(4, 25))
        cuts = int(rng.integers(1, min(n - 1, 9) + 1)) if trial % 8 else n + 1  # every 8th: too many partitions
        if trial % 3 == 0:
            bw, _ = W.geometric_bandwidths(n, seed=trial, link="pairwise")
        else:
            bw = rng.integers(0, 40, size=(n, n)).astype(np.uint32)
            if trial % 2:
                bw = (np.triu(bw, 1) + np.triu(bw, 1).T).astype(np.uint32)
        sizes = rng.integers(1, 10**7, cuts).astype(np.uint64)
        if trial % 4 == 1:
            sizes = rng.integers(1, 4, cuts).astype(np.uint64)  # few distinct sizes: long runs
        n_classes = int(rng.integers(1, 6))
        draws = rng.integers(0, 2**32, size=(12, n), dtype=np.uint64).astype(np.uint32)
        if cuts > 12 and n_classes == 1:
            continue
        want = OPL.k_path_matching(bw.tolist(), [int(x) for x in sizes], n_classes, draws.tolist())
        longest = max((r[1] for X in range(n_classes) for r in OPL.find_subarrays(OPL.size_classes(sizes, n_classes), X)),
                      default=0)
        if longest > 12:
            continue
        st, nodes, thr = pp.kpath_matching(bw, sizes, n_classes, draws)
        if want.status == OPL.INFEASIBLE:
            n_fail += 1
            assert st == pp.PP_INFEASIBLE and (nodes == -1).all()
            continue
        n_ok += 1
        assert st == pp.PP_OK and tuple(nodes.tolist()) == want.nodes, trial
        for first, run, _, t in want.thresholds:
            assert (thr[first:first + run] == t).all()
    assert n_ok >= 20 and n_fail >= 3
    # no cut: node 0; limits
    st, nodes, _ = pp.kpath_matching(np.ones((3, 3), np.uint32), np.zeros(0, np.uint64), 2, np.zeros((1, 3), np.uint32))
    assert st == pp.PP_OK and nodes.tolist() == [0]
    with pytest.raises(pp.PPError):
        pp.kpath_matching(np.ones((65, 65), np.uint32), np.ones(2, np.uint64), 1, np.zeros((1, 65), np.uint32))
    with pytest.raises(pp.PPError):  # one run of 13 cuts needs a path of 14 vertices
        pp.kpath_matching(np.ones((20, 20), np.uint32), np.ones(13, np.uint64), 1, np.zeros((1, 20), np.uint32))


def test_the_papers_heuristic_end_to_end():
    # Section 3.2 as a whole on the paper's kind of setting: a chain, devices of equal memory, the
    # random geometric graph of Section 4.  Partition stage (Algorithm 1, weights = transfer sizes),
    # placement stage (Algorithms 2 and 3), bottleneck latency by the evaluator (Eq. 2, Eq. 3).
    rng = np.random.default_rng(52)
    ratios = []
    for seed, (k, cap_mb, n_classes) in enumerate(((10, 32, 2), (12, 32, 3), (14, 48, 2), (12, 24, 5), (14, 40, 8))):
        inst = W.config_geometric(k, cap_mb, seed, link="pairwise")
        kappa = int(inst.node_mem_bytes[0])
        part = pp.partition_minsum_batch(inst.layer_out_bits[None, :], inst.layer_mem_bytes[None, :],
                                         np.array([kappa], np.uint64), inst.L)
        want_part = OP.minsum_partition(inst.layer_out_bits.tolist(), inst.layer_mem_bytes.tolist(), kappa)
        m = int(part.m[0])
        assert part.status[0] == pp.PP_OK and m == want_part.m and tuple(part.cuts[0, :m - 1].tolist()) == want_part.cuts
        assert 2 <= m <= k
        sizes = part.sizes[0, :m - 1]
        draws = rng.integers(0, 2**32, size=(24, k), dtype=np.uint64).astype(np.uint32)
        st, nodes, thr = pp.kpath_matching(inst.bw_kbps, sizes, n_classes, draws)
        want = OPL.k_path_matching(inst.bw_kbps.tolist(), [int(x) for x in sizes], n_classes, draws.tolist())
        assert (st == pp.PP_OK) == (want.status == OPL.OK)
        if st != pp.PP_OK:
            continue
        assert tuple(nodes.tolist()) == want.nodes and len(set(nodes.tolist())) == m
        # score the plan: cuts from the partition stage, nodes from the placement stage
        ends = np.full((1, k), -1, np.int32)
        nd = np.full((1, k), -1, np.int32)
        ends[0, :m - 1] = part.cuts[0, :m - 1]
        nd[0, :m] = nodes
        with pp.Problem.from_instance(inst) as p:
            beta, flags = p.eval_plans(np.array([m], np.uint8), ends, nd)
            exact = p.solve_exact()
        wb, wf = oracle.eval_plans(inst, np.array([m], np.uint8), ends, nd)
        assert flags[0] == 0 == wf[0] and beta[0] == wb[0]
        # the exact search can only be better; Theorem 1 bounds the heuristic from below for its own S
        assert exact.status == pp.PP_OK and exact.beta_ms <= beta[0]
        assert beta[0] >= float(sizes.max()) / float(inst.bw_kbps.max())
        # every cut's link is at least the threshold its run was placed at
        for j in range(m - 1):
            assert inst.bw_kbps[nodes[j], nodes[j + 1]] >= thr[j] > 0
        ratios.append(beta[0] / exact.beta_ms)
    assert len(ratios) >= 3 and min(ratios) >= 1.0
