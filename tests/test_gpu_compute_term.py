"""GPU parity of the exact search under Eq. 1 (pp_solve_exact_compute) against
oracle/compute_term.py: beta is an fp64 quotient selected by min/max on both sides and the plan is
integers, so every comparison is exact equality."""
from __future__ import annotations

import numpy as np
import pytest

import paper_2210_12219_b200 as pp
from oracle import compute_term as CT
from paper_2210_12219_b200 import build
from paper_2210_12219_b200 import workloads as W
from tests.helpers import make_instance

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    pp.lib()


def _same(got, want, k):
    assert got.status == want.status
    if want.status == CT.INFEASIBLE:
        assert np.isinf(got.beta_ms) and got.m == 0
    else:
        assert got.beta_ms == want.beta_ms and got.plan() == want.plan()
    assert (got.cuts[max(got.m - 1, 0):] == -1).all() and (got.placement[got.m:] == -1).all()
    assert len(got.cuts) == k - 1 and len(got.placement) == k


def test_hand_worked_instance():
    inst = make_instance(np.array([6000, 12000, 999], np.uint64), np.array([1, 1, 1], np.uint64),
                         np.array([3, 3], np.uint64), np.array([[0, 3000], [3000, 0]], np.uint32))
    got = pp.solve_exact_compute(inst, [10, 20, 30], [2, 4])
    assert got.beta_ms == 12.5 and got.plan() == (2, (0,), (0, 1))
    assert pp.solve_exact_compute(inst, [10, 20, 30], [0, 0]).status == pp.PP_INFEASIBLE


def test_random_instances_against_the_oracle():
    rng = np.random.default_rng(71)
    n_inf = 0
    for trial, (L, k) in enumerate([(1, 1), (1, 3), (2, 2), (5, 3), (7, 4), (12, 6), (9, 5), (17, 5), (33, 4), (16, 7),
                                    (40, 3), (24, 8)] * 4):
        inst = W.random_small(71000 + trial, L, k, tight=trial % 4 == 1, ties=trial % 4 == 2,
                              dead_links=0.3 if trial % 4 == 3 else 0.0)
        work = rng.integers(0, 10**6, L).astype(np.uint64)
        if trial % 5 == 0:
            work = (rng.integers(1, 4, L) * 1000).astype(np.uint64)
        # speeds that make compute times comparable to the transfer latencies (hundreds of ms)
        speed = rng.integers(0 if trial % 6 == 0 else 1, 4000, k).astype(np.uint32)
        want = CT.dp(inst, work.tolist(), speed.tolist())
        _same(pp.solve_exact_compute(inst, work, speed), want, k)
        n_inf += want.status == CT.INFEASIBLE
    assert n_inf >= 2


def test_named_shapes_and_the_reduction_to_eq2():
    rng = np.random.default_rng(72)
    for inst in (W.config_tiny(), W.config_resnet50_shaped(), W.config_geometric(10, 32, 3)):
        # layers cost work in proportion to their memory, nodes differ threefold in speed
        work = (inst.layer_mem_bytes // 1000).astype(np.uint64)
        speed = rng.integers(200, 600, inst.k).astype(np.uint32)
        want = CT.dp(inst, work.tolist(), speed.tolist())
        got = pp.solve_exact_compute(inst, work, speed)
        _same(got, want, inst.k)
        assert CT.eval_plan(inst, work.tolist(), speed.tolist(), got.plan()[1], got.plan()[2]) == got.beta_ms
        # nothing costs compute: the optimum of Eq. 2, plan and all
        with pp.Problem.from_instance(inst) as p:
            eq2 = p.solve_exact()
        free = pp.solve_exact_compute(inst, np.zeros(inst.L, np.uint64), np.ones(inst.k, np.uint32))
        assert free.beta_ms == eq2.beta_ms and free.plan() == eq2.plan()
        assert got.beta_ms >= eq2.beta_ms
    # limits
    big = W.config_large()
    with pytest.raises(pp.PPError) as e:
        pp.solve_exact_compute(big, np.ones(big.L, np.uint64), np.ones(big.k, np.uint32))
    assert e.value.status == pp.PP_ERR_LIMIT
