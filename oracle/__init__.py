"""CPU oracle (test infrastructure only): ctypes wrapper around pp_oracle.c.

Nothing in the product package imports this module.  It is used by the tests, by the
smoke check and by the benchmark's CPU-baseline leg, never by the CUDA path.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pp_oracle.c")
_LIB = os.path.join(_HERE, "libpp_oracle.so")

OK, INFEASIBLE = 0, 1
PLAN_BAD_NSEG, PLAN_BAD_ENDS, PLAN_BAD_NODE, PLAN_MEMORY, PLAN_DEAD_LINK = 1, 2, 4, 8, 16


def build(force: bool = False) -> str:
    """Compile pp_oracle.c with strict IEEE settings (no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fno-fast-math", "-ffp-contract=off", "-fopenmp",
               "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.orc_gamma.restype = ctypes.c_double
        lib.orc_gamma.argtypes = [ctypes.c_uint64, ctypes.c_uint32]
        _lib = lib
    return _lib


def _p(a, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct))


def _inputs(inst):
    bits = np.ascontiguousarray(inst.layer_out_bits, dtype=np.uint64)
    mem = np.ascontiguousarray(inst.layer_mem_bytes, dtype=np.uint64)
    cap = np.ascontiguousarray(inst.node_mem_bytes, dtype=np.uint64)
    bw = np.ascontiguousarray(inst.bw_kbps, dtype=np.uint32)
    keep = (bits, mem, cap, bw)
    args = (ctypes.c_int(inst.L), _p(bits, ctypes.c_uint64), _p(mem, ctypes.c_uint64),
            ctypes.c_int(inst.k), _p(cap, ctypes.c_uint64), _p(bw, ctypes.c_uint32))
    return keep, args


@dataclass
class Solution:
    status: int
    beta_ms: float
    m: int
    cuts: np.ndarray  # int32 [k-1], -1 padded
    placement: np.ndarray  # int32 [k], -1 padded
    table: np.ndarray | None = None  # float64 [2^k, k, L] when requested
    plans_visited: int = 0

    def plan(self):
        return (self.m, tuple(int(x) for x in self.cuts[: max(self.m - 1, 0)]),
                tuple(int(x) for x in self.placement[: self.m]))


def gamma(bits: int, kbps: int) -> float:
    """Eq. 3 as one fp64 division, in milliseconds (bits / kbps)."""
    return float(_load().orc_gamma(int(bits), int(kbps)))


def eval_plan(inst, nseg: int, cuts, nodes):
    """(beta_ms, plan_status) of one candidate plan (Eq. 2 and Eq. 3)."""
    lib = _load()
    keep, args = _inputs(inst)
    k = inst.k
    c = np.full(max(k, 1), -1, dtype=np.int32)
    n = np.full(max(k, 1), -1, dtype=np.int32)
    cuts = np.asarray(cuts, dtype=np.int32).ravel()
    nodes = np.asarray(nodes, dtype=np.int32).ravel()
    c[: min(len(cuts), k)] = cuts[:k]
    n[: min(len(nodes), k)] = nodes[:k]
    beta = ctypes.c_double()
    st = lib.orc_eval_plan(*args, ctypes.c_int(int(nseg)), _p(c, ctypes.c_int32),
                           _p(n, ctypes.c_int32), ctypes.byref(beta))
    return beta.value, int(st)


def eval_plans(inst, nseg, ends, nodes):
    """Vector form of eval_plan: arrays shaped like the library's batched evaluator."""
    B = len(nseg)
    beta = np.empty(B, dtype=np.float64)
    status = np.empty(B, dtype=np.uint8)
    for b in range(B):
        beta[b], status[b] = eval_plan(inst, int(nseg[b]), ends[b], nodes[b])
    return beta, status


def _solve(fn_name, inst, extra=(), want_table=False, visited=False):
    lib = _load()
    keep, args = _inputs(inst)
    k = inst.k
    beta = ctypes.c_double()
    m = ctypes.c_int32()
    cuts = np.full(max(k - 1, 1), -1, dtype=np.int32)
    placement = np.full(k, -1, dtype=np.int32)
    table = None
    tail = []
    if visited:
        nv = ctypes.c_uint64()
        tail = [ctypes.byref(nv)]
    else:
        if want_table:
            table = np.empty((1 << k, k, inst.L), dtype=np.float64)
            tail = [_p(table, ctypes.c_double)]
        else:
            tail = [ctypes.POINTER(ctypes.c_double)()]
    fn = getattr(lib, fn_name)
    st = fn(*args, *extra, ctypes.byref(beta), ctypes.byref(m), _p(cuts, ctypes.c_int32),
            _p(placement, ctypes.c_int32), *tail)
    if st < 0:
        raise RuntimeError(f"{fn_name} failed with status {st}")
    return Solution(int(st), beta.value, int(m.value), cuts[: max(k - 1, 0)], placement, table,
                    int(nv.value) if visited else 0)


def bruteforce(inst) -> Solution:
    """Enumerate every cut set times every injective placement; canonical optimum."""
    return _solve("orc_bruteforce", inst, visited=True)


def dp_naive(inst, want_table=False) -> Solution:
    """The recurrence with every (v, c) predecessor tested separately."""
    return _solve("orc_dp_naive", inst, want_table=want_table)


def dp_fact(inst, nthreads: int = 1, want_table=False) -> Solution:
    """Same recurrence, min over v first, then a scan over the feasible run of c."""
    return _solve("orc_dp_fact", inst, extra=(ctypes.c_int(int(nthreads)),), want_table=want_table)


def max_threads() -> int:
    return int(_load().orc_max_threads())
