"""GPU parity of the greedy comparison baseline (Section 4): the CUDA entry point, through the
C-ABI, against its CPU oracle, bit for bit (beta is one fp64 quotient chosen by max and min on
both sides; plans are integers)."""
from __future__ import annotations

import ctypes

import numpy as np
import pytest
import torch

import paper_2210_12219_b200 as pp
from oracle import greedy
from paper_2210_12219_b200 import build
from paper_2210_12219_b200 import workloads as W
from tests.test_oracle_greedy import parse_greedy_golden

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    pp.lib()


def _stack(insts):
    f = lambda g: np.stack([g(i) for i in insts])
    return (f(lambda i: i.layer_out_bits), f(lambda i: i.layer_mem_bytes), f(lambda i: i.node_mem_bytes),
            f(lambda i: i.bw_kbps))


def _check(insts, got):
    k = insts[0].k
    n_stuck = 0
    for b, inst in enumerate(insts):
        want = greedy.greedy_joint(inst)
        assert got.status[b] == want.status, (inst.name, b)
        if want.status == greedy.OK:
            assert got.beta_ms[b] == want.beta_ms, (inst.name, b)
        else:
            assert np.isinf(got.beta_ms[b]) and got.m[b] == 0
            n_stuck += 1
        assert got.plan(b) == want.plan(), (inst.name, b)
        assert (got.cuts[b, max(want.m - 1, 0):] == -1).all() and (got.placement[b, want.m:] == -1).all()
        assert got.cuts.shape[1] == k - 1 and got.placement.shape[1] == k
    return n_stuck


def test_hand_worked_walks_on_the_device():
    for inst, _, best in parse_greedy_golden():
        got = pp.greedy_batch(inst.L, inst.k, *_stack([inst]))
        if best is None:
            assert got.status[0] == pp.PP_INFEASIBLE and got.m[0] == 0 and np.isinf(got.beta_ms[0])
        else:
            start, beta, cuts, nodes = best
            assert got.status[0] == pp.PP_OK and got.beta_ms[0] == beta
            assert got.plan(0) == (len(nodes), cuts, nodes) and nodes[0] == start


def test_random_instances_of_many_shapes():
    stuck = 0
    for L, k, n in ((1, 1, 3), (2, 2, 9), (5, 3, 40), (13, 5, 60), (3, 6, 12), (30, 7, 40), (64, 12, 20),
                    (200, 20, 9)):
        insts = [W.random_small(71000 + 100 * L + i, L, k, tight=(i % 3 == 1), ties=(i % 3 == 2),
                                dead_links=0.25 if i % 4 == 3 else 0.0) for i in range(n)]
        stuck += _check(insts, pp.greedy_batch(L, k, *_stack(insts)))
    assert stuck > 0


def test_full_batched_config_and_ratio_to_the_optimum():
    insts = W.config_batched()
    arrays = _stack(insts)
    got = pp.greedy_batch(24, 8, *arrays)
    stuck = _check(insts, got)
    assert 0 <= stuck < len(insts)
    # against the exact search on the same arrays: never better, and a plan whenever the greedy has one
    best = pp.solve_exact_batch(24, 8, *arrays)
    found = got.status == pp.PP_OK
    assert (best.status[found] == pp.PP_OK).all()
    assert (best.beta_ms[found] <= got.beta_ms[found]).all()
    assert (best.beta_ms[found] < got.beta_ms[found]).any()


def test_device_pointer_form_on_a_stream_and_argument_checks():
    insts = [W.random_small(72000 + i, 9, 4) for i in range(33)]  # a ragged last block of warps
    bits, mem, cap, bw = (torch.from_numpy(a).cuda() for a in
                          (x.view(np.int64) if x.dtype == np.uint64 else x.view(np.int32) for x in _stack(insts)))
    B, L, k = len(insts), 9, 4
    beta = torch.empty(B, dtype=torch.float64, device="cuda")
    m = torch.empty(B, dtype=torch.int32, device="cuda")
    cuts = torch.empty(B * (k - 1), dtype=torch.int32, device="cuda")
    place = torch.empty(B * k, dtype=torch.int32, device="cuda")
    status = torch.empty(B, dtype=torch.int8, device="cuda")
    stream = torch.cuda.Stream()
    pp.greedy_batch_dev(B, L, k, bits.data_ptr(), mem.data_ptr(), cap.data_ptr(), bw.data_ptr(), beta.data_ptr(),
                        m.data_ptr(), cuts.data_ptr(), place.data_ptr(), status.data_ptr(), stream.cuda_stream)
    stream.synchronize()
    host = pp.greedy_batch(L, k, *_stack(insts))
    assert (beta.cpu().numpy() == host.beta_ms).all() and (m.cpu().numpy() == host.m).all()
    assert (cuts.cpu().numpy().reshape(B, k - 1) == host.cuts).all()
    assert (place.cpu().numpy().reshape(B, k) == host.placement).all()
    assert (status.cpu().numpy() == host.status).all()
    lib = pp.lib()
    assert lib.pp_greedy_batch(-1, 4, 2, *([None] * 9)) == pp.PP_ERR_ARG
    assert lib.pp_greedy_batch(1, 4, 30, *([None] * 9)) == pp.PP_ERR_LIMIT
    assert lib.pp_greedy_batch(0, 4, 2, *([None] * 9)) == pp.PP_OK
    assert lib.pp_greedy_batch(1, 4, 2, *([None] * 9)) == pp.PP_ERR_ARG
