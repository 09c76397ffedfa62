"""pp_solve_exact_static: the exact search for callers that may not allocate device memory (for
instance a process whose device heap belongs to a framework's allocator, or a plug-in that may
only launch work).  Its scratch is one array compiled into the library, shared by all calls and
never cleared between them.  Checked here: the result record equals the CPU oracle's (exact
equality, like every other parity test) and the allocating entry point's, on consecutive calls
with different shapes, both state-element widths and a shape close to the array's size; the
free device memory does not move across calls; instances beyond the array are refused."""
from __future__ import annotations

import ctypes

import numpy as np
import pytest

import oracle
import paper_2210_12219_b200 as pp
from paper_2210_12219_b200 import build
from paper_2210_12219_b200 import workloads as W
from tests.helpers import make_instance

pytestmark = pytest.mark.gpu


def _static_solve(inst, torch, rec_dev=None):
    if rec_dev is None:
        rec_dev = torch.zeros(ctypes.sizeof(pp.pp_solution) // 8, dtype=torch.float64, device="cuda")
    st = pp.solve_exact_static(inst.L, inst.layer_out_bits, inst.layer_mem_bytes, inst.k,
                               inst.node_mem_bytes, inst.bw_kbps, rec_dev.data_ptr(), 0)
    assert st == pp.PP_OK, pp.status_str(st)
    torch.cuda.synchronize()
    return pp.pp_solution.from_buffer_copy(rec_dev.cpu().numpy().tobytes())


def _same(rec, want):
    assert rec.status == want.status
    assert rec.beta_ms == want.beta_ms or (np.isinf(rec.beta_ms) and np.isinf(want.beta_ms))
    assert rec.m == want.m
    assert tuple(rec.cuts[:max(want.m - 1, 0)]) == want.plan()[1]
    assert tuple(rec.placement[:want.m]) == want.plan()[2]
    assert all(x == -1 for x in rec.cuts[max(want.m - 1, 0):]) and all(x == -1 for x in rec.placement[want.m:])


def _wide_rank_instance():
    """More distinct latencies than 16-bit codes: the static layout then uses 4-byte elements."""
    L, k = 1024, 9
    base = W.random_small(70010, L, k)
    bw = base.bw_kbps.copy()
    bw[np.triu_indices(k, 1)] += np.arange(k * (k - 1) // 2, dtype=np.uint32) + 1  # directed links
    cap = np.full(k, int(base.layer_mem_bytes.sum()) // 3, dtype=np.uint64)
    inst = make_instance(base.layer_out_bits, base.layer_mem_bytes, cap, bw)
    assert len({int(x) for x in inst.bw_kbps.ravel() if x}) * L + 1 > 65534
    return inst


def test_static_scratch_entry_point_matches_oracle_and_allocating_one():
    import torch
    build.build()
    # calls in a row on different shapes (a smaller one after a larger one, so stale contents
    # remain in the array), instances without a plan, both element widths, then the first again
    cases = [W.config_resnet50_shaped(), W.config_tiny(), W.random_small(20001, 5, 3, tight=True),
             W.random_small(70001, 9, 5, tight=True), W.random_small(70003, 6, 4, tight=True),
             _wide_rank_instance(), W.config_deeper_cnn(), W.config_resnet50_shaped()]
    statuses = []
    for inst in cases:
        want = oracle.dp_fact(inst, oracle.max_threads())
        rec = _static_solve(inst, torch)
        _same(rec, want)
        with pp.Problem.from_instance(inst) as p:
            p.force_generic(1)
            _same(rec, p.solve_exact())
        statuses.append(want.status)
    assert pp.PP_OK in statuses and pp.PP_INFEASIBLE in statuses


def test_static_entry_point_leaves_free_device_memory_alone():
    import torch
    build.build()
    rec_dev = torch.zeros(ctypes.sizeof(pp.pp_solution) // 8, dtype=torch.float64, device="cuda")
    shapes = [W.config_tiny(), W.config_resnet50_shaped(), W.random_small(70004, 40, 7)]
    _static_solve(shapes[0], torch, rec_dev)  # first call on the device: looks up the array's address
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for inst in shapes * 2:
        st = pp.solve_exact_static(inst.L, inst.layer_out_bits, inst.layer_mem_bytes, inst.k,
                                   inst.node_mem_bytes, inst.bw_kbps, rec_dev.data_ptr(), 0)
        assert st == pp.PP_OK
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0


def test_static_entry_point_refuses_what_does_not_fit():
    import torch
    build.build()
    rec_dev = torch.zeros(22, dtype=torch.float64, device="cuda")
    big = W.config_large()  # k = 18 is beyond k = 14
    assert pp.solve_exact_static(big.L, big.layer_out_bits, big.layer_mem_bytes, big.k,
                                 big.node_mem_bytes, big.bw_kbps, rec_dev.data_ptr(), 0) == pp.PP_ERR_LIMIT
    deep = W.random_small(70002, 900, 13)  # k is fine, the state table is not
    assert pp.solve_exact_static(deep.L, deep.layer_out_bits, deep.layer_mem_bytes, deep.k,
                                 deep.node_mem_bytes, deep.bw_kbps, rec_dev.data_ptr(), 0) == pp.PP_ERR_LIMIT
    # and the array is still usable afterwards
    inst = W.config_tiny()
    _same(_static_solve(inst, torch), oracle.dp_fact(inst, 2))
