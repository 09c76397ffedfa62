"""Exact min-bottleneck partition-and-placement search on one B200 (sm_100a).

The package is a thin binding over libpp.so (C-ABI in include/pp.h): `Problem` wraps a
pp_problem handle (solve_exact, eval_plans, ...), `solve_exact_batch` solves many small
instances in one launch, `greedy_batch` runs the paper's greedy comparison baseline on the same
arrays.  `workloads` holds the seeded synthetic instance generators.
"""
from .binding import (PP_ERR_ARG, PP_ERR_CUDA, PP_ERR_LIMIT, PP_ERR_NOMEM, PP_INFEASIBLE, PP_MAX_K,
                      PP_MAX_L, PP_OK, PP_PLAN_BAD_ENDS, PP_PLAN_BAD_NODE, PP_PLAN_BAD_NSEG,
                      PP_PLAN_DEAD_LINK, PP_PLAN_MEMORY, BatchSolution, PPError, Problem, Solution,
                      PartitionBatch, debug_fail_alloc, debug_minmax_rate, kpath_colour_batch, kpath_colour_batch_dev, kpath_matching, partition_minsum_batch, partition_minsum_batch_dev, greedy_batch, greedy_batch_dev, lib, pp_profile, pp_solution, solve_exact_batch, solve_exact_batch_dev, solve_exact_compute, solve_exact_static,
                      status_str)

__all__ = [n for n in dir() if not n.startswith("_")]
