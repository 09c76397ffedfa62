"""CPU-side checks of the C-ABI: the library loads, exports every symbol the header declares,
and rejects bad arguments before touching a device."""
from __future__ import annotations

import ctypes
import math
import os
import re

import numpy as np
import pytest

from paper_2210_12219_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "pp.h")).read()
    declared = set(re.findall(r"\b(pp_[a-z_]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_bounds_checking_build_exports_the_same_symbols():
    dbg = ctypes.CDLL(build.build_debug())
    for name in binding.EXPORTS:
        assert hasattr(dbg, name), name


def test_struct_layouts_match_header():
    assert ctypes.sizeof(binding.pp_solution) == 8 + 4 + 4 + 4 * 20 + 4 * 20
    assert ctypes.sizeof(binding.pp_profile) == 36


def test_status_strings(lib):
    for code in (0, 1, -1, -2, -3, -4, -5):
        assert binding.status_str(code) and "unknown" not in binding.status_str(code)
    assert "unknown" in binding.status_str(77)


def _create(L, bits, mem, k, cap, bw):
    h = ctypes.c_void_p()
    keep = [np.ascontiguousarray(a) for a in (bits, mem, cap, bw)]
    st = binding.lib().pp_problem_create(L, *(ctypes.c_void_p(a.ctypes.data) for a in keep[:2]), k,
                                         *(ctypes.c_void_p(a.ctypes.data) for a in keep[2:]),
                                         ctypes.byref(h))
    return st, h


def test_create_rejects_bad_arguments_without_a_device(lib):
    ok = dict(bits=np.ones(4, np.uint64), mem=np.ones(4, np.uint64), cap=np.ones(2, np.uint64),
              bw=np.ones(4, np.uint32))
    assert _create(0, ok["bits"], ok["mem"], 2, ok["cap"], ok["bw"])[0] == binding.PP_ERR_ARG
    assert _create(4, ok["bits"], ok["mem"], 0, ok["cap"], ok["bw"])[0] == binding.PP_ERR_ARG
    assert _create(2000, np.ones(2000, np.uint64), np.ones(2000, np.uint64), 2, ok["cap"],
                   ok["bw"])[0] == binding.PP_ERR_LIMIT
    assert _create(4, ok["bits"], ok["mem"], 21, np.ones(21, np.uint64),
                   np.ones(441, np.uint32))[0] == binding.PP_ERR_LIMIT
    big = ok["bits"].copy()
    big[1] = 1 << 40
    assert _create(4, big, ok["mem"], 2, ok["cap"], ok["bw"])[0] == binding.PP_ERR_LIMIT
    fat = ok["bw"].copy()
    fat[1] = 1 << 24
    assert _create(4, ok["bits"], ok["mem"], 2, ok["cap"], fat)[0] == binding.PP_ERR_LIMIT
    h = ctypes.c_void_p()
    assert lib.pp_problem_create(4, None, None, 2, None, None, ctypes.byref(h)) == binding.PP_ERR_ARG
    assert lib.pp_problem_create(4, None, None, 2, None, None, None) == binding.PP_ERR_ARG


def test_null_handles_are_rejected(lib):
    lib.pp_problem_destroy(None)  # allowed
    n = ctypes.c_uint64()
    assert lib.pp_problem_workspace_bytes(None, ctypes.byref(n)) == binding.PP_ERR_ARG
    assert lib.pp_solve_exact(None, None, None, None, None) == binding.PP_ERR_ARG
    assert lib.pp_eval_plans(None, 1, None, None, None, None, None) == binding.PP_ERR_ARG
    assert lib.pp_random_plans(None, 1, None, None, None, None) == binding.PP_ERR_ARG
    assert lib.pp_random_plans_dev(None, 1, None, None, None, None) == binding.PP_ERR_ARG
    assert lib.pp_solve_exact_batch(-1, 4, 2, *([None] * 9)) == binding.PP_ERR_ARG
    assert lib.pp_solve_exact_batch(1, 4, 30, *([None] * 9)) == binding.PP_ERR_LIMIT
    assert lib.pp_solve_exact_batch(0, 4, 2, *([None] * 9)) == binding.PP_OK
    assert lib.pp_greedy_batch(-1, 4, 2, *([None] * 9)) == binding.PP_ERR_ARG
    assert lib.pp_greedy_batch(1, 4, 30, *([None] * 9)) == binding.PP_ERR_LIMIT
    assert lib.pp_greedy_batch(0, 4, 2, *([None] * 9)) == binding.PP_OK
    assert lib.pp_greedy_batch_dev(1, 4, 2, *([None] * 10)) == binding.PP_ERR_ARG


def test_no_cpu_fallback_without_device(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    st, _ = _create(4, np.ones(4, np.uint64), np.ones(4, np.uint64), 2, np.ones(2, np.uint64),
                    np.ones(4, np.uint32))
    assert st in (binding.PP_ERR_CUDA, binding.PP_ERR_NOMEM)


def test_mask_order_is_a_revolving_door(lib):
    # the two-mask sweep kernel pairs neighbours of each level: they must differ by one node
    # swapped for another, every non-empty node set must appear exactly once, levels by popcount
    for k in (1, 2, 3, 5, 8, 12, 18):
        masks, level_off = binding.debug_mask_order(k)
        assert level_off[0] == 0 and level_off[k + 1] == (1 << k) - 1
        assert sorted(int(m) for m in masks) == list(range(1, 1 << k))
        for j in range(1, k + 1):
            level = [int(m) for m in masks[level_off[j]:level_off[j + 1]]]
            assert len(level) == math.comb(k, j)
            assert all(bin(m).count("1") == j for m in level)
            for a, b in zip(level, level[1:]):
                assert bin(a ^ b).count("1") == 2, (k, j, a, b)
    bad = np.zeros(4, np.uint32)
    assert binding.lib().pp_debug_mask_order(0, ctypes.c_void_p(bad.ctypes.data),
                                             ctypes.c_void_p(bad.ctypes.data)) == binding.PP_ERR_ARG
    assert binding.lib().pp_debug_mask_order(21, ctypes.c_void_p(bad.ctypes.data),
                                             ctypes.c_void_p(bad.ctypes.data)) == binding.PP_ERR_LIMIT
