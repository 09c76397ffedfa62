"""GPU parity of the random comparison baseline (Section 4): plans generated on the device from
caller-supplied draws, through the C-ABI, against the CPU oracle fed the same draws, entry by
entry (integers only)."""
from __future__ import annotations

import numpy as np
import pytest
import torch

import paper_2210_12219_b200 as pp
from oracle import random_plans as rp
from paper_2210_12219_b200 import build
from paper_2210_12219_b200 import workloads as W
from tests.test_oracle_random_plans import parse_random_golden

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    pp.lib()


def _draws(seed, P, k):
    d = np.random.default_rng(seed).integers(0, 2**32, size=(P, 2 * k), dtype=np.uint64).astype(np.uint32)
    d[0, :] = 0  # the extreme draws are always in
    d[1, :] = 0xFFFFFFFF
    return d


def _check(inst, draws, got):
    nseg, ends, nodes = got
    w_nseg, w_ends, w_nodes = rp.random_plans(inst, draws)
    assert nseg.tolist() == w_nseg
    assert ends.tolist() == w_ends
    assert nodes.tolist() == w_nodes
    return sum(1 for x in w_nseg if x == 0)


def test_hand_worked_draws_on_the_device():
    for inst, rows in parse_random_golden():
        draws = np.array([d for d, _ in rows], dtype=np.uint32)
        with pp.Problem.from_instance(inst) as p:
            nseg, ends, nodes = p.random_plans(draws)
        for i, (_, want) in enumerate(rows):
            if want is None:
                assert nseg[i] == 0 and (ends[i] == -1).all() and (nodes[i] == -1).all()
            else:
                cuts, nd = want
                assert nseg[i] == len(nd) and tuple(nodes[i, :len(nd)]) == nd and tuple(ends[i, :len(cuts)]) == cuts
                assert (ends[i, len(cuts):] == -1).all() and (nodes[i, len(nd):] == -1).all()


def test_random_instances_of_many_shapes():
    none = 0
    for L, k, P in ((1, 1, 5), (2, 2, 40), (7, 3, 300), (13, 5, 257), (30, 7, 100), (100, 12, 64), (200, 20, 33)):
        inst = W.random_small(83000 + L, L, k, tight=(L % 2 == 1))
        draws = _draws(L, P, k)
        with pp.Problem.from_instance(inst) as p:
            none += _check(inst, draws, p.random_plans(draws))
    assert none > 0


def test_named_configs_and_scoring_by_the_evaluator():
    for inst in (W.config_resnet50_shaped(), W.config_large()):
        draws = _draws(5, 2000, inst.k)
        with pp.Problem.from_instance(inst) as p:
            got = p.random_plans(draws)
            none = _check(inst, draws, got)
            beta, flags = p.eval_plans(*got)
            best = p.solve_exact()
        nseg = got[0]
        assert 0 < none < len(nseg)
        # generated plans are plans of the problem: the evaluator flags only the rows without a plan
        # (and plans over missing links), and none beats the exact optimum
        assert ((flags == 0) | (flags == pp.PP_PLAN_DEAD_LINK))[nseg > 0].all()
        assert (flags[nseg == 0] == pp.PP_PLAN_BAD_NSEG).all()
        assert (beta[nseg > 0] >= best.beta_ms).all()


def test_device_pointer_form():
    inst = W.config_deeper_cnn()
    P, k = 1000, inst.k
    draws = _draws(9, P, k)
    d = torch.from_numpy(draws.view(np.int32)).cuda()
    nseg = torch.empty(P, dtype=torch.uint8, device="cuda")
    ends = torch.empty(P * k, dtype=torch.int32, device="cuda")
    nodes = torch.empty(P * k, dtype=torch.int32, device="cuda")
    stream = torch.cuda.Stream()
    with pp.Problem.from_instance(inst) as p:
        p.set_stream(stream.cuda_stream)
        p.random_plans_dev(P, d.data_ptr(), nseg.data_ptr(), ends.data_ptr(), nodes.data_ptr())
        stream.synchronize()
        host = p.random_plans(draws)
    assert (nseg.cpu().numpy() == host[0]).all()
    assert (ends.cpu().numpy().reshape(P, k) == host[1]).all()
    assert (nodes.cpu().numpy().reshape(P, k) == host[2]).all()
    _check(inst, draws, host)
