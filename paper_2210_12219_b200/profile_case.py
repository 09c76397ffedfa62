"""Small driver for profilers: solves the Large instance restricted to its first --k nodes.

    python -m paper_2210_12219_b200.profile_case --k 16 --solves 2
    python -m paper_2210_12219_b200.profile_case --batch 4096 --solves 1
    python -m paper_2210_12219_b200.profile_case --batch 65536 --greedy --solves 1
    python -m paper_2210_12219_b200.profile_case --k 18 --random-plans 262144 --solves 1

With k = 16 the state table is 0.44 GB (still far above the 126 MB L2), small enough for a
multi-pass counter capture of single sweep launches.
"""
from __future__ import annotations

import argparse
import ctypes

import numpy as np


def main():
    import torch

    import paper_2210_12219_b200 as pp
    from paper_2210_12219_b200 import build
    from paper_2210_12219_b200 import workloads as W

    ap = argparse.ArgumentParser()
    ap.add_argument("--k", type=int, default=16)
    ap.add_argument("--solves", type=int, default=2)
    ap.add_argument("--generic", action="store_true")
    ap.add_argument("--batch", type=int, default=0, help="solve this many batched instances instead")
    ap.add_argument("--greedy", action="store_true", help="with --batch: the greedy comparison baseline")
    ap.add_argument("--random-plans", type=int, default=0,
                    help="generate this many random plans (random comparison baseline) instead of solving")
    args = ap.parse_args()
    build.build()
    if args.batch:
        insts = W.config_batched(args.batch)
        stack = lambda f: np.stack([f(i) for i in insts])
        entry = pp.greedy_batch if args.greedy else pp.solve_exact_batch
        for _ in range(args.solves):
            got = entry(24, 8, stack(lambda i: i.layer_out_bits), stack(lambda i: i.layer_mem_bytes),
                        stack(lambda i: i.node_mem_bytes), stack(lambda i: i.bw_kbps))
        print("batch of %d: %d with a plan" % (args.batch, int((got.status == 0).sum())))
        return
    large = W.config_large()
    k = args.k
    inst = W.Instance(large.L, k, large.layer_out_bits, large.layer_mem_bytes,
                      large.node_mem_bytes[:k].copy(), np.ascontiguousarray(large.bw_kbps[:k, :k]))
    if args.random_plans:
        draws = np.random.default_rng(4242).integers(0, 2**32, size=(args.random_plans, 2 * k), dtype=np.uint64)
        with pp.Problem.from_instance(inst) as p:
            for _ in range(args.solves):
                nseg, _, _ = p.random_plans(draws.astype(np.uint32))
        print("%d random plans: %d rows with a plan" % (args.random_plans, int((nseg > 0).sum())))
        return
    sol = torch.zeros(ctypes.sizeof(pp.pp_solution) // 8, dtype=torch.float64, device="cuda")
    with pp.Problem.from_instance(inst) as p:
        if args.generic:
            p.force_generic(1)
        for _ in range(args.solves):
            p.solve_exact_dev(sol.data_ptr())
        torch.cuda.synchronize()
        prof = p.last_solve_profile()
        rec = pp.pp_solution.from_buffer_copy(sol.cpu().numpy().tobytes())
        print("k=%d L=%d beta=%.6f m=%d sweep=%.3f ms total=%.3f ms fast=%d" %
              (k, inst.L, rec.beta_ms, rec.m, prof.ms_sweep, prof.ms_total, prof.fast_path))


if __name__ == "__main__":
    main()
