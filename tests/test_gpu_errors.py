"""Error reporting on a healthy device: the bounds-checking build of the library (every index into
the state and rank tables checked, a violation recorded instead of trapping) runs the parity cases
clean, and allocation failures injected by the library's test hook come back as PP_ERR_NOMEM."""
from __future__ import annotations

import contextlib

import numpy as np
import pytest

import oracle
import paper_2210_12219_b200 as pp
import paper_2210_12219_b200.binding as binding
from paper_2210_12219_b200 import build
from paper_2210_12219_b200 import workloads as W

pytestmark = pytest.mark.gpu


@contextlib.contextmanager
def library(path):
    old_path, old_lib = binding.LIB_PATH, binding._lib
    binding.LIB_PATH, binding._lib = path, None
    try:
        yield
    finally:
        binding.LIB_PATH, binding._lib = old_path, old_lib


def test_bounds_checking_build_runs_the_parity_cases_clean():
    build.build()
    dbg = build.build_debug()
    cases = [W.config_tiny(), W.config_resnet50_shaped(), W.random_small(81000, 1, 1), W.random_small(81001, 3, 6),
             W.random_small(81002, 17, 5, tight=True), W.random_small(81003, 33, 4, dead_links=0.3),
             W.uniform_memory_small(81004, 24, 7, 8, 16), W.uniform_memory_small(81005, 40, 9, 8, 30),
             W.uniform_memory_small(81006, 200, 8, 21, 85), W.config_geometric(9, 64, 4)]
    with library(dbg):
        for inst in cases:
            want = oracle.dp_fact(inst, 4)
            for mode in (-1, 1, 2, 3):
                with pp.Problem.from_instance(inst) as p:
                    p.force_generic(mode)
                    got = p.solve_exact()  # a recorded violation would raise PP_ERR_CUDA here
                    assert got.status == want.status and got.plan() == want.plan(), (inst.name, mode)
                    assert got.beta_ms == want.beta_ms or np.isinf(want.beta_ms)
        # the other entry points of the debug build answer like the normal one
        inst = W.config_resnet50_shaped()
        nseg, ends, nodes = W.random_plans(inst, 500, seed=2)
        with pp.Problem.from_instance(inst) as p:
            assert np.array_equal(p.eval_plans(nseg, ends, nodes)[0], oracle.eval_plans(inst, nseg, ends, nodes)[0])
        # the batched search, both device paths (64 instances and more take the instance-per-lane
        # kernels); a recorded violation would come back as PP_ERR_CUDA in the instance's status
        for L, k, n in ((24, 8, 70), (7, 8, 65), (32, 4, 66), (13, 5, 20)):
            insts = [W.random_small(82000 + 100 * L + i, L, k, tight=(i % 3 == 1), dead_links=0.25 if i % 4 == 3 else 0.0)
                     for i in range(n)]
            got = pp.solve_exact_batch(L, k, np.stack([i.layer_out_bits for i in insts]),
                                       np.stack([i.layer_mem_bytes for i in insts]),
                                       np.stack([i.node_mem_bytes for i in insts]),
                                       np.stack([i.bw_kbps for i in insts]))
            for b, inst in enumerate(insts):
                want = oracle.dp_naive(inst)
                assert got.status[b] == want.status and got.plan(b) == want.plan(), (L, k, b)
    assert binding.LIB_PATH.endswith("libpp.so")


def test_injected_allocation_failures_come_back_as_nomem():
    build.build()
    inst = W.config_resnet50_shaped()
    with pp.Problem.from_instance(inst) as warm:  # per-k tables and pools exist from here on
        warm.solve_exact()
    # the input upload of pp_problem_create
    pp.debug_fail_alloc(1)
    with pytest.raises(pp.PPError) as e:
        pp.Problem.from_instance(inst)
    assert e.value.status == pp.PP_ERR_NOMEM
    # the search scratch, allocated at the first solve; the problem stays usable
    with pp.Problem.from_instance(inst) as p:
        pp.debug_fail_alloc(1)
        with pytest.raises(pp.PPError) as e:
            p.solve_exact()
        assert e.value.status == pp.PP_ERR_NOMEM
        want = oracle.dp_fact(inst, 4)
        got = p.solve_exact()
        assert got.beta_ms == want.beta_ms and got.plan() == want.plan()
        # the staging buffer of a host-pointer entry point
        nseg, ends, nodes = W.random_plans(inst, 100, seed=3)
        pp.debug_fail_alloc(1)
        with pytest.raises(pp.PPError) as e:
            p.eval_plans(nseg, ends, nodes)
        assert e.value.status == pp.PP_ERR_NOMEM
        assert p.eval_plans(nseg, ends, nodes)[0].shape == (100,)
    # the second allocation from now on: create succeeds, the solve does not
    pp.debug_fail_alloc(2)
    with pp.Problem.from_instance(inst) as p:
        with pytest.raises(pp.PPError) as e:
            p.solve_exact()
        assert e.value.status == pp.PP_ERR_NOMEM
        assert p.solve_exact().status == pp.PP_OK
    pp.debug_fail_alloc(0)
    # a workspace that is too small is refused the same way
    import torch
    with pp.Problem.from_instance(inst) as p:
        small = torch.empty(1024, dtype=torch.uint8, device="cuda")
        with pytest.raises(pp.PPError) as e:
            p.set_workspace(small)
        assert e.value.status == pp.PP_ERR_NOMEM
