"""pp_solve_exact_static: the exact search for callers that may not allocate device memory
(for instance a process whose device heap belongs to a framework's allocator, or a serving
loop that cannot take cudaMalloc's device-wide synchronisation).  Its scratch is one array
compiled into the library, shared by all calls and never cleared between them, so the checks
here are: same result record as the allocating entry point (exact equality, like every other
parity test), on consecutive calls with different instances, and a clean refusal of an
instance that does not fit the array."""
from __future__ import annotations

import ctypes

import numpy as np
import pytest

import paper_2210_12219_b200 as pp
from paper_2210_12219_b200 import build
from paper_2210_12219_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _static_solve(inst, torch):
    rec_dev = torch.zeros(ctypes.sizeof(pp.pp_solution) // 8, dtype=torch.float64, device="cuda")
    st = pp.solve_exact_static(inst.L, inst.layer_out_bits, inst.layer_mem_bytes, inst.k,
                               inst.node_mem_bytes, inst.bw_kbps, rec_dev.data_ptr(), 0)
    assert st == pp.PP_OK, pp.status_str(st)
    torch.cuda.synchronize()
    return pp.pp_solution.from_buffer_copy(rec_dev.cpu().numpy().tobytes())


def _same(rec, want, k):
    assert rec.status == want.status
    assert rec.beta_ms == want.beta_ms or (np.isinf(rec.beta_ms) and np.isinf(want.beta_ms))
    assert rec.m == want.m
    assert tuple(rec.cuts[:max(want.m - 1, 0)]) == want.plan()[1]
    assert tuple(rec.placement[:want.m]) == want.plan()[2]
    assert all(x == -1 for x in rec.cuts[max(want.m - 1, 0):]) and all(x == -1 for x in rec.placement[want.m:])


def test_static_scratch_entry_point_matches_allocating_one():
    import torch
    build.build()
    # two calls in a row on different shapes (the second smaller, so stale contents of the
    # first remain in the array), an infeasible instance, then the first shape again
    cases = [W.config_resnet50_shaped(), W.config_tiny(), W.random_small(20001, 5, 3, tight=True),
             W.random_small(70001, 9, 5, tight=True), W.config_resnet50_shaped()]
    statuses = set()
    for inst in cases:
        with pp.Problem.from_instance(inst) as p:
            want = p.solve_exact()
        _same(_static_solve(inst, torch), want, inst.k)
        statuses.add(want.status)
    assert pp.PP_OK in statuses
    # beyond the array (or beyond k = 14): refused with PP_ERR_LIMIT, nothing queued
    big = W.config_large()
    rec_dev = torch.zeros(22, dtype=torch.float64, device="cuda")
    assert pp.solve_exact_static(big.L, big.layer_out_bits, big.layer_mem_bytes, big.k,
                                 big.node_mem_bytes, big.bw_kbps, rec_dev.data_ptr(), 0) == pp.PP_ERR_LIMIT
    deep = W.random_small(70002, 900, 13)
    assert pp.solve_exact_static(deep.L, deep.layer_out_bits, deep.layer_mem_bytes, deep.k,
                                 deep.node_mem_bytes, deep.bw_kbps, rec_dev.data_ptr(), 0) == pp.PP_ERR_LIMIT
    # and the array is still usable afterwards
    inst = W.config_tiny()
    with pp.Problem.from_instance(inst) as p:
        _same(_static_solve(inst, torch), p.solve_exact(), inst.k)
