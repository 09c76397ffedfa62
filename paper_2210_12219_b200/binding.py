"""Thin ctypes binding of libpp.so: argument marshalling only, same names as include/pp.h.

Every step of the search and of the evaluator runs inside the library's CUDA kernels.  There is
no Python or CPU fallback: if libpp.so is missing or fails to load, importing the library
handle raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libpp.so")

PP_MAX_K, PP_MAX_L = 20, 1024
PP_OK, PP_INFEASIBLE = 0, 1
PP_ERR_ARG, PP_ERR_LIMIT, PP_ERR_NOMEM, PP_ERR_CUDA, PP_ERR_TIMEOUT = -1, -2, -3, -4, -5
PP_PLAN_BAD_NSEG, PP_PLAN_BAD_ENDS, PP_PLAN_BAD_NODE, PP_PLAN_MEMORY, PP_PLAN_DEAD_LINK = 1, 2, 4, 8, 16

EXPORTS = (
    "pp_problem_create", "pp_problem_destroy", "pp_problem_set_stream",
    "pp_problem_workspace_bytes", "pp_problem_set_workspace", "pp_solve_exact",
    "pp_solve_exact_dev", "pp_eval_plans", "pp_eval_plans_dev", "pp_solve_exact_batch",
    "pp_solve_exact_batch_dev", "pp_last_solve_profile", "pp_debug_read_state_row", "pp_debug_mask_order",
    "pp_problem_force_generic", "pp_solve_exact_static", "pp_status_str", "pp_greedy_batch",
    "pp_greedy_batch_dev", "pp_random_plans", "pp_random_plans_dev", "pp_debug_minmax_rate",
    "pp_problem_set_profiling", "pp_eval_plans_packed", "pp_eval_plans_packed_dev",
    "pp_partition_minsum_batch", "pp_partition_minsum_batch_dev",
    "pp_kpath_colour_batch", "pp_kpath_colour_batch_dev", "pp_debug_fail_alloc",
    "pp_kpath_matching", "pp_solve_exact_compute",
)


class pp_solution(ctypes.Structure):
    _fields_ = [("beta_ms", ctypes.c_double), ("status", ctypes.c_int32), ("m", ctypes.c_int32),
                ("cuts", ctypes.c_int32 * PP_MAX_K), ("placement", ctypes.c_int32 * PP_MAX_K)]


class pp_profile(ctypes.Structure):
    _fields_ = [("ms_rank", ctypes.c_float), ("ms_sweep", ctypes.c_float),
                ("ms_finalize", ctypes.c_float), ("ms_total", ctypes.c_float),
                ("sweep_launches", ctypes.c_int32), ("total_launches", ctypes.c_int32),
                ("state_bytes", ctypes.c_int32), ("fast_path", ctypes.c_int32),
                ("pair_levels", ctypes.c_int32)]


class PPError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_str(status)} ({status})")


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded library.  Raises if it has not been built (run __graft_entry__.build())."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} not found: build the CUDA library first "
                               "(python -m paper_2210_12219_b200.build); there is no CPU fallback")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, i64, u64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_uint64
        L.pp_problem_create.argtypes = [i32, vp, vp, i32, vp, vp, ctypes.POINTER(vp)]
        L.pp_problem_destroy.argtypes = [vp]
        L.pp_problem_destroy.restype = None
        L.pp_problem_set_stream.argtypes = [vp, vp]
        L.pp_problem_workspace_bytes.argtypes = [vp, ctypes.POINTER(u64)]
        L.pp_problem_set_workspace.argtypes = [vp, vp, u64]
        L.pp_solve_exact.argtypes = [vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(i32), vp, vp]
        L.pp_solve_exact_dev.argtypes = [vp, vp]
        L.pp_eval_plans.argtypes = [vp, i64, vp, vp, vp, vp, vp]
        L.pp_eval_plans_dev.argtypes = [vp, i64, vp, vp, vp, vp, vp]
        L.pp_eval_plans_packed.argtypes = [vp, i64, i64, vp, vp, vp, vp, vp, vp]
        L.pp_eval_plans_packed_dev.argtypes = [vp, i64, i64, vp, vp, vp, vp, vp, vp]
        L.pp_solve_exact_batch.argtypes = [i64, i32, i32] + [vp] * 9
        L.pp_solve_exact_batch_dev.argtypes = [i64, i32, i32] + [vp] * 10
        L.pp_greedy_batch.argtypes = [i64, i32, i32] + [vp] * 9
        L.pp_random_plans.argtypes = [vp, i64] + [vp] * 4
        L.pp_random_plans_dev.argtypes = [vp, i64] + [vp] * 4
        L.pp_greedy_batch_dev.argtypes = [i64, i32, i32] + [vp] * 10
        L.pp_last_solve_profile.argtypes = [vp, ctypes.POINTER(pp_profile)]
        L.pp_debug_read_state_row.argtypes = [vp, ctypes.c_uint32, i32, vp]
        L.pp_debug_mask_order.argtypes = [i32, vp, vp]
        L.pp_problem_force_generic.argtypes = [vp, i32]
        L.pp_problem_set_profiling.argtypes = [vp, i32]
        L.pp_solve_exact_static.argtypes = [i32, vp, vp, i32, vp, vp, vp, vp]
        L.pp_debug_minmax_rate.argtypes = [i32, i32, ctypes.POINTER(ctypes.c_double)]
        L.pp_partition_minsum_batch.argtypes = [i64, i32, vp, vp, vp, i32, vp, vp, vp, vp, vp]
        L.pp_partition_minsum_batch_dev.argtypes = [i64, i32, vp, vp, vp, i32, vp, vp, vp, vp, vp, vp]
        L.pp_kpath_colour_batch.argtypes = [i32, vp, i64, i32] + [vp] * 7
        L.pp_kpath_colour_batch_dev.argtypes = [i32, vp, i64, i32] + [vp] * 8
        L.pp_debug_fail_alloc.argtypes = [i32]
        L.pp_kpath_matching.argtypes = [i32, vp, i32, vp, i32, i32, vp, vp, vp, vp]
        L.pp_solve_exact_compute.argtypes = [i32, vp, vp, vp, i32, vp, vp, vp, ctypes.POINTER(ctypes.c_double),
                                             ctypes.POINTER(i32), vp, vp]
        L.pp_status_str.argtypes = [ctypes.c_int]
        L.pp_status_str.restype = ctypes.c_char_p
        for name in EXPORTS:
            if name not in ("pp_problem_destroy", "pp_status_str"):
                getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def status_str(status: int) -> str:
    return lib().pp_status_str(int(status)).decode()


def _host(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a, ctypes.c_void_p(a.ctypes.data)


def _check(status: int, where: str, ok=(PP_OK,)):
    if status not in ok:
        raise PPError(status, where)
    return status


@dataclass
class Solution:
    status: int
    beta_ms: float
    m: int
    cuts: np.ndarray
    placement: np.ndarray

    def plan(self):
        return (self.m, tuple(int(x) for x in self.cuts[: max(self.m - 1, 0)]),
                tuple(int(x) for x in self.placement[: self.m]))


class Problem:
    """Owner of a pp_problem handle.  Methods mirror the C entry points one to one."""

    def __init__(self, L, layer_out_bits, layer_mem_bytes, k, node_mem_bytes, bw_kbps):
        self.L, self.k = int(L), int(k)
        self._h = ctypes.c_void_p()
        keep = [_host(layer_out_bits, np.uint64), _host(layer_mem_bytes, np.uint64),
                _host(node_mem_bytes, np.uint64), _host(bw_kbps, np.uint32)]
        st = lib().pp_problem_create(self.L, keep[0][1], keep[1][1], self.k, keep[2][1], keep[3][1],
                                     ctypes.byref(self._h))
        _check(st, "pp_problem_create")
        self._workspace = None

    @classmethod
    def from_instance(cls, inst):
        return cls(inst.L, inst.layer_out_bits, inst.layer_mem_bytes, inst.k, inst.node_mem_bytes,
                   inst.bw_kbps)

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            lib().pp_problem_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    # -- plumbing ------------------------------------------------------------------------
    def set_stream(self, cuda_stream: int):
        _check(lib().pp_problem_set_stream(self._h, ctypes.c_void_p(cuda_stream)), "pp_problem_set_stream")

    def workspace_bytes(self) -> int:
        n = ctypes.c_uint64()
        _check(lib().pp_problem_workspace_bytes(self._h, ctypes.byref(n)), "pp_problem_workspace_bytes")
        return int(n.value)

    def set_workspace(self, tensor):
        """Use a torch CUDA tensor (uint8) as the search scratch; it is kept alive by this object."""
        _check(lib().pp_problem_set_workspace(self._h, ctypes.c_void_p(tensor.data_ptr()),
                                              tensor.numel() * tensor.element_size()),
               "pp_problem_set_workspace")
        self._workspace = tensor

    def set_profiling(self, on: bool):
        _check(lib().pp_problem_set_profiling(self._h, int(bool(on))), "pp_problem_set_profiling")

    def force_generic(self, mode: int):
        _check(lib().pp_problem_force_generic(self._h, int(mode)), "pp_problem_force_generic")

    # -- exact search --------------------------------------------------------------------
    def solve_exact(self) -> Solution:
        beta = ctypes.c_double()
        m = ctypes.c_int32()
        cuts = np.full(max(self.k - 1, 1), -1, dtype=np.int32)
        placement = np.full(self.k, -1, dtype=np.int32)
        st = lib().pp_solve_exact(self._h, ctypes.byref(beta), ctypes.byref(m),
                                  ctypes.c_void_p(cuts.ctypes.data), ctypes.c_void_p(placement.ctypes.data))
        _check(st, "pp_solve_exact", ok=(PP_OK, PP_INFEASIBLE))
        return Solution(st, beta.value, int(m.value), cuts[: max(self.k - 1, 0)], placement)

    def solve_exact_dev(self, solution_ptr: int):
        """Queue the search; the pp_solution record is written at device address solution_ptr."""
        _check(lib().pp_solve_exact_dev(self._h, ctypes.c_void_p(solution_ptr)), "pp_solve_exact_dev")

    def last_solve_profile(self) -> pp_profile:
        prof = pp_profile()
        _check(lib().pp_last_solve_profile(self._h, ctypes.byref(prof)), "pp_last_solve_profile")
        return prof

    def debug_read_state_row(self, mask: int, v: int) -> np.ndarray:
        row = np.empty(self.L, dtype=np.float64)
        _check(lib().pp_debug_read_state_row(self._h, int(mask), int(v), ctypes.c_void_p(row.ctypes.data)),
               "pp_debug_read_state_row")
        return row

    # -- evaluator -----------------------------------------------------------------------
    def eval_plans(self, nseg, ends, nodes):
        """Host arrays in, host arrays out: (beta_ms float64 [B], plan_status uint8 [B])."""
        nseg, p0 = _host(nseg, np.uint8)
        B = nseg.shape[0]
        ends, p1 = _host(ends, np.int32)
        nodes, p2 = _host(nodes, np.int32)
        assert ends.size == B * self.k and nodes.size == B * self.k
        beta = np.empty(B, dtype=np.float64)
        status = np.empty(B, dtype=np.uint8)
        _check(lib().pp_eval_plans(self._h, B, p0, p1, p2, ctypes.c_void_p(beta.ctypes.data),
                                   ctypes.c_void_p(status.ctypes.data)), "pp_eval_plans")
        return beta, status

    def eval_plans_dev(self, B, nseg_ptr, ends_ptr, nodes_ptr, beta_ptr, status_ptr):
        _check(lib().pp_eval_plans_dev(self._h, int(B), *(ctypes.c_void_p(x) for x in
                                       (nseg_ptr, ends_ptr, nodes_ptr, beta_ptr, status_ptr))),
               "pp_eval_plans_dev")

    def eval_plans_packed(self, nseg, plan_off, ends, nodes, out=None):
        """pp_eval_plans_packed: uint8 [B], uint32 [B + 1], uint16 [total], uint8 [total] (host) ->
        (beta_ms float64 [B], plan_status uint8 [B]).  out = (beta, status): arrays of the caller to
        write into (page-locked ones make the copy back a plain DMA)."""
        nseg, p0 = _host(nseg, np.uint8)
        B = nseg.shape[0]
        plan_off, p1 = _host(plan_off, np.uint32)
        ends, p2 = _host(ends, np.uint16)
        nodes, p3 = _host(nodes, np.uint8)
        assert plan_off.size == B + 1 and ends.size == nodes.size
        beta, status = out if out is not None else (np.empty(B, dtype=np.float64), np.empty(B, dtype=np.uint8))
        assert beta.dtype == np.float64 and status.dtype == np.uint8 and beta.size == B and status.size == B
        assert beta.flags.c_contiguous and status.flags.c_contiguous
        _check(lib().pp_eval_plans_packed(self._h, B, ends.size, p0, p1, p2, p3, ctypes.c_void_p(beta.ctypes.data),
                                          ctypes.c_void_p(status.ctypes.data)), "pp_eval_plans_packed")
        return beta, status

    def eval_plans_packed_dev(self, B, total, nseg_ptr, off_ptr, ends_ptr, nodes_ptr, beta_ptr, status_ptr):
        _check(lib().pp_eval_plans_packed_dev(self._h, int(B), int(total), *(ctypes.c_void_p(x) for x in
                                              (nseg_ptr, off_ptr, ends_ptr, nodes_ptr, beta_ptr, status_ptr))),
               "pp_eval_plans_packed_dev")

    # -- random comparison baseline -------------------------------------------------------
    def random_plans(self, draws):
        """pp_random_plans: uint32 draws [P, 2k] -> (nseg uint8 [P], ends int32 [P, k], nodes int32 [P, k])."""
        draws, p0 = _host(draws, np.uint32)
        assert draws.ndim == 2 and draws.shape[1] == 2 * self.k
        P = draws.shape[0]
        nseg = np.empty(P, dtype=np.uint8)
        ends = np.empty((P, self.k), dtype=np.int32)
        nodes = np.empty((P, self.k), dtype=np.int32)
        _check(lib().pp_random_plans(self._h, P, p0, *(ctypes.c_void_p(a.ctypes.data) for a in (nseg, ends, nodes))),
               "pp_random_plans")
        return nseg, ends, nodes

    def random_plans_dev(self, P, draws_ptr, nseg_ptr, ends_ptr, nodes_ptr):
        _check(lib().pp_random_plans_dev(self._h, int(P), *(ctypes.c_void_p(x) for x in
                                         (draws_ptr, nseg_ptr, ends_ptr, nodes_ptr))), "pp_random_plans_dev")


@dataclass
class BatchSolution:
    beta_ms: np.ndarray  # float64 [B]
    m: np.ndarray  # int32 [B]
    cuts: np.ndarray  # int32 [B, k-1]
    placement: np.ndarray  # int32 [B, k]
    status: np.ndarray  # int8 [B]

    def plan(self, b):
        m = int(self.m[b])
        return (m, tuple(int(x) for x in self.cuts[b, : max(m - 1, 0)]),
                tuple(int(x) for x in self.placement[b, :m]))


def solve_exact_batch(L, k, out_bits, mem, node_mem, bw) -> BatchSolution:
    """Host arrays [B, L], [B, L], [B, k], [B, k, k] -> BatchSolution (synchronous)."""
    return _batch_from_host("pp_solve_exact_batch", L, k, out_bits, mem, node_mem, bw)


def greedy_batch(L, k, out_bits, mem, node_mem, bw) -> BatchSolution:
    """pp_greedy_batch: the greedy comparison baseline on the same host arrays (synchronous)."""
    return _batch_from_host("pp_greedy_batch", L, k, out_bits, mem, node_mem, bw)


def _batch_from_host(entry, L, k, out_bits, mem, node_mem, bw) -> BatchSolution:
    out_bits, p0 = _host(out_bits, np.uint64)
    B = out_bits.shape[0]
    mem, p1 = _host(mem, np.uint64)
    node_mem, p2 = _host(node_mem, np.uint64)
    bw, p3 = _host(bw, np.uint32)
    assert out_bits.size == B * L and mem.size == B * L and node_mem.size == B * k and bw.size == B * k * k
    beta = np.empty(B, dtype=np.float64)
    m = np.empty(B, dtype=np.int32)
    cuts = np.full((B, max(k - 1, 1)), -1, dtype=np.int32)
    placement = np.empty((B, k), dtype=np.int32)
    status = np.empty(B, dtype=np.int8)
    st = getattr(lib(), entry)(B, L, k, p0, p1, p2, p3, *(ctypes.c_void_p(a.ctypes.data) for a in
                                                          (beta, m, cuts, placement, status)))
    _check(st, entry)
    return BatchSolution(beta, m, cuts[:, : max(k - 1, 0)] if k > 1 else cuts[:, :0], placement, status)


def debug_mask_order(k: int):
    """pp_debug_mask_order: (masks uint32 [2^k - 1], level_off uint32 [k + 2]); needs no device."""
    masks = np.zeros((1 << k) - 1, dtype=np.uint32)
    level_off = np.zeros(k + 2, dtype=np.uint32)
    _check(lib().pp_debug_mask_order(int(k), ctypes.c_void_p(masks.ctypes.data),
                                     ctypes.c_void_p(level_off.ctypes.data)), "pp_debug_mask_order")
    return masks, level_off


@dataclass
class PartitionBatch:
    cost: np.ndarray    # uint64 [B]
    m: np.ndarray       # int32 [B]
    cuts: np.ndarray    # int32 [B, cap_seg]
    sizes: np.ndarray   # uint64 [B, cap_seg]
    status: np.ndarray  # int8 [B]


def partition_minsum_batch(cut_weight, mem, kappa, cap_seg: int) -> PartitionBatch:
    """pp_partition_minsum_batch: host arrays [B, L], [B, L], [B] -> PartitionBatch (synchronous)."""
    cut_weight, p0 = _host(cut_weight, np.uint64)
    B, L = cut_weight.shape
    mem, p1 = _host(mem, np.uint64)
    kappa, p2 = _host(kappa, np.uint64)
    assert mem.shape == (B, L) and kappa.shape == (B,)
    cost = np.empty(B, dtype=np.uint64)
    m = np.empty(B, dtype=np.int32)
    cuts = np.full((B, max(cap_seg, 1)), -1, dtype=np.int32)
    sizes = np.zeros((B, max(cap_seg, 1)), dtype=np.uint64)
    status = np.empty(B, dtype=np.int8)
    st = lib().pp_partition_minsum_batch(B, L, p0, p1, p2, int(cap_seg), *(ctypes.c_void_p(a.ctypes.data) for a in
                                         (cost, m, cuts, sizes, status)))
    _check(st, "pp_partition_minsum_batch")
    return PartitionBatch(cost, m, cuts[:, :cap_seg], sizes[:, :cap_seg], status)


def partition_minsum_batch_dev(B, L, weight_ptr, mem_ptr, kappa_ptr, cap_seg, cost_ptr, m_ptr, cuts_ptr, sizes_ptr,
                               status_ptr, cuda_stream: int = 0):
    st = lib().pp_partition_minsum_batch_dev(int(B), int(L), *(ctypes.c_void_p(x) for x in (weight_ptr, mem_ptr, kappa_ptr)),
                                             int(cap_seg), *(ctypes.c_void_p(x) for x in
                                             (cost_ptr, m_ptr, cuts_ptr, sizes_ptr, status_ptr, cuda_stream)))
    _check(st, "pp_partition_minsum_batch_dev")


def kpath_colour_batch(bw, kk: int, threshold, start, end, alive, colours):
    """pp_kpath_colour_batch: bw uint32 [n, n]; per query threshold uint32, start / end int32 (-1 = any),
    alive uint64 bit masks, colours uint8 [Q, n] -> (found uint8 [Q], path int32 [Q, kk])."""
    bw, p0 = _host(bw, np.uint32)
    n = bw.shape[0]
    threshold, p1 = _host(threshold, np.uint32)
    Q = threshold.shape[0]
    start, p2 = _host(start, np.int32)
    end, p3 = _host(end, np.int32)
    alive, p4 = _host(alive, np.uint64)
    colours, p5 = _host(colours, np.uint8)
    assert colours.size == Q * n and start.size == Q and end.size == Q and alive.size == Q
    found = np.zeros(Q, dtype=np.uint8)
    path = np.full((Q, kk), -1, dtype=np.int32)
    st = lib().pp_kpath_colour_batch(n, p0, Q, int(kk), p1, p2, p3, p4, p5, ctypes.c_void_p(found.ctypes.data),
                                     ctypes.c_void_p(path.ctypes.data))
    _check(st, "pp_kpath_colour_batch")
    return found, path


def kpath_colour_batch_dev(n, bw_ptr, Q, kk, threshold_ptr, start_ptr, end_ptr, alive_ptr, colours_ptr, found_ptr,
                           path_ptr, cuda_stream: int = 0):
    st = lib().pp_kpath_colour_batch_dev(int(n), ctypes.c_void_p(bw_ptr), int(Q), int(kk),
                                         *(ctypes.c_void_p(x) for x in (threshold_ptr, start_ptr, end_ptr, alive_ptr,
                                                                       colours_ptr, found_ptr, path_ptr, cuda_stream)))
    _check(st, "pp_kpath_colour_batch_dev")


def kpath_matching(bw, sizes, n_classes: int, draws, cuda_stream: int = 0):
    """pp_kpath_matching: bw uint32 [n, n], sizes uint64 [n_cuts], draws uint32 [trials, n] ->
    (status, nodes int32 [n_cuts + 1], cut_threshold uint32 [n_cuts])."""
    bw, p0 = _host(bw, np.uint32)
    n = bw.shape[0]
    sizes, p1 = _host(sizes, np.uint64)
    draws, p2 = _host(draws, np.uint32)
    assert draws.ndim == 2 and draws.shape[1] == n
    nodes = np.full(sizes.size + 1, -1, dtype=np.int32)
    thr = np.zeros(max(sizes.size, 1), dtype=np.uint32)
    st = lib().pp_kpath_matching(n, p0, int(sizes.size), p1, int(n_classes), int(draws.shape[0]), p2,
                                 ctypes.c_void_p(nodes.ctypes.data), ctypes.c_void_p(thr.ctypes.data),
                                 ctypes.c_void_p(cuda_stream))
    _check(st, "pp_kpath_matching", ok=(PP_OK, PP_INFEASIBLE))
    return st, nodes, thr[: sizes.size]


def solve_exact_compute(inst, layer_work, node_speed) -> Solution:
    """pp_solve_exact_compute: the exact search under Eq. 1 for a workloads.Instance plus per-layer work
    (uint64 [L]) and per-node speed (uint32 [k])."""
    keep = [_host(inst.layer_out_bits, np.uint64), _host(inst.layer_mem_bytes, np.uint64), _host(layer_work, np.uint64),
            _host(inst.node_mem_bytes, np.uint64), _host(inst.bw_kbps, np.uint32), _host(node_speed, np.uint32)]
    k = int(inst.k)
    beta, m = ctypes.c_double(), ctypes.c_int32()
    cuts = np.full(max(k - 1, 1), -1, dtype=np.int32)
    placement = np.full(k, -1, dtype=np.int32)
    st = lib().pp_solve_exact_compute(int(inst.L), keep[0][1], keep[1][1], keep[2][1], k, keep[3][1], keep[4][1],
                                      keep[5][1], ctypes.byref(beta), ctypes.byref(m),
                                      ctypes.c_void_p(cuts.ctypes.data), ctypes.c_void_p(placement.ctypes.data))
    _check(st, "pp_solve_exact_compute", ok=(PP_OK, PP_INFEASIBLE))
    return Solution(st, beta.value, int(m.value), cuts[: max(k - 1, 0)], placement)


def debug_fail_alloc(nth: int):
    """pp_debug_fail_alloc: the nth device allocation from now on reports out of memory (0 clears)."""
    _check(lib().pp_debug_fail_alloc(int(nth)), "pp_debug_fail_alloc")


def debug_minmax_rate(op: int, iters: int = 2048) -> float:
    """pp_debug_minmax_rate: warp instructions per clock per SM of one packed min/max form."""
    rate = ctypes.c_double()
    _check(lib().pp_debug_minmax_rate(int(op), int(iters), ctypes.byref(rate)), "pp_debug_minmax_rate")
    return float(rate.value)


def solve_exact_batch_dev(B, L, k, bits_ptr, mem_ptr, node_mem_ptr, bw_ptr, beta_ptr, m_ptr, cuts_ptr,
                          placement_ptr, status_ptr, cuda_stream: int = 0):
    st = lib().pp_solve_exact_batch_dev(int(B), int(L), int(k), *(ctypes.c_void_p(x) for x in (
        bits_ptr, mem_ptr, node_mem_ptr, bw_ptr, beta_ptr, m_ptr, cuts_ptr, placement_ptr, status_ptr,
        cuda_stream)))
    _check(st, "pp_solve_exact_batch_dev")


def greedy_batch_dev(B, L, k, bits_ptr, mem_ptr, node_mem_ptr, bw_ptr, beta_ptr, m_ptr, cuts_ptr,
                     placement_ptr, status_ptr, cuda_stream: int = 0):
    st = lib().pp_greedy_batch_dev(int(B), int(L), int(k), *(ctypes.c_void_p(x) for x in (
        bits_ptr, mem_ptr, node_mem_ptr, bw_ptr, beta_ptr, m_ptr, cuts_ptr, placement_ptr, status_ptr,
        cuda_stream)))
    _check(st, "pp_greedy_batch_dev")


def solve_exact_static(L, layer_out_bits, layer_mem_bytes, k, node_mem_bytes, bw_kbps,
                       solution_ptr: int, cuda_stream: int = 0) -> int:
    """pp_solve_exact_static: host input arrays, device address of the pp_solution record.
    Returns the status code instead of raising, so callers can test the limit check."""
    keep = [_host(layer_out_bits, np.uint64), _host(layer_mem_bytes, np.uint64),
            _host(node_mem_bytes, np.uint64), _host(bw_kbps, np.uint32)]
    return lib().pp_solve_exact_static(int(L), keep[0][1], keep[1][1], int(k), keep[2][1], keep[3][1],
                                       ctypes.c_void_p(solution_ptr), ctypes.c_void_p(cuda_stream))
