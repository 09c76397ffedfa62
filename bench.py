#!/usr/bin/env python
"""Benchmark of the exact partition-and-placement path on B200.

One step = one pass of the whole hot path over one batch of synthetic input:
  1. exact search on the Large instance (k = 18 nodes, L = 200 layers): gamma/rank tables,
     base frontier, every popcount level of the (min,max) sweep, final choice, backtrack;
  2. the batched many-instance search on 4096 instances (k = 8, L = 24);
  3. the batched beta evaluator on 262144 candidate plans of the Large instance (compressed rows:
     16-bit cuts, 8-bit nodes, one offset per plan).
The headline number is DP relaxations per second, where one relaxation is
g = min(g, max(dp, gamma)) and an instance has k(k-1)2^(k-2) L of them (a closed form of
the sizes, not of the data).

`value` is measured with the inputs resident in device memory; `e2e` goes through the
host-pointer C entry points, host<->device copies inside the timed region.
`--impl reference` times the CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import ctypes
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2210_12219_b200 import workloads as W  # noqa: E402

METRIC = "exact-plan DP relaxations/s"
UNIT = "relaxations/s"
# DRAM bytes (read + write) per sweep launch of the Large solve from an ncu capture of the sweep
# kernels as they stand; None whenever those kernels have changed since the counters were taken.
SWEEP_DRAM_BYTES_PER_LAUNCH = 100.40e6
NOMINAL_HBM_GBS = 8000.0  # the "about 8 TB/s" the roofline is also quoted against
N_PLANS = 262144
N_BATCH = 4096
BATCH_L, BATCH_K = 24, 8
WORKLOAD = ("Large: k=18 nodes, L=200 layers (exact search) + Batched: 4096 x (k=8, L=24) + "
            "262144 candidate plans scored")


def n_relax(k: int, L: int) -> int:
    return k * (k - 1) * (1 << (k - 2)) * L if k >= 2 else 0


def n_states(k: int, L: int) -> int:
    return k * (1 << (k - 1)) * L


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "sm_max_mhz": 1965.0}, "fallback"


class ClockSampler:
    """nvidia-smi clock/throttle sampling in the background while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.path = None

    def __enter__(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
            time.sleep(0.3)  # let the first sample land before the timed region starts
        except Exception:
            self.proc = None
        return self

    def __exit__(self, *exc):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()

    def summary(self):
        if self.proc is None or not self.path or not os.path.exists(self.path):
            return None
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        with open(self.path) as f:
            for line in f:
                t = [x.strip() for x in line.split(",")]
                if len(t) < 7:
                    continue
                try:
                    sm.append(float(t[0]))
                    mx.append(float(t[1]))
                except ValueError:
                    continue
                for name, val in zip(names, t[3:7]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        os.unlink(self.path)
        if not sm:
            return None
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "samples": len(sm),
                "reasons": sorted(reasons)}


def aggregate_over_ranks(units_this_rank: float, seconds_this_rank: float, dist=None, device=None):
    """Whole-job throughput of independent replicas: units summed over ranks divided by the
    slowest rank's time.  Works with any initialised torch.distributed backend (NCCL on GPUs,
    gloo on CPU); without one it is the single-rank ratio."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return units_this_rank / seconds_this_rank, seconds_this_rank
    import torch
    t = torch.tensor([seconds_this_rank], dtype=torch.float64, device=device)
    u = torch.tensor([units_this_rank], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(u.item()) / float(t.item()), float(t.item())


def stack(insts):
    return (np.stack([i.layer_out_bits for i in insts]), np.stack([i.layer_mem_bytes for i in insts]),
            np.stack([i.node_mem_bytes for i in insts]), np.stack([i.bw_kbps for i in insts]))


def run_ours(args):
    import torch

    import paper_2210_12219_b200 as pp
    from paper_2210_12219_b200 import build as pp_build

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    pp_build.build()
    pp.lib()
    dev = torch.device("cuda", local)

    # ---- synthetic inputs (every rank works on its own replica of the same workload) ----
    large = W.config_large()
    batch = W.config_batched(N_BATCH, BATCH_L, BATCH_K)
    b_bits, b_mem, b_cap, b_bw = stack(batch)
    nseg, ends, nodes = W.random_plans(large, N_PLANS, seed=77, invalid_fraction=0.05)
    p_off, p_ends, p_nodes = W.pack_plans(nseg, ends, nodes)
    n_entries = int(p_ends.size)
    k, L = large.k, large.L
    relax_large = n_relax(k, L)
    relax_batch = N_BATCH * n_relax(BATCH_K, BATCH_L)
    relax_step = relax_large + relax_batch

    stream = torch.cuda.Stream(device=dev)
    prob = pp.Problem.from_instance(large)
    prob.set_stream(stream.cuda_stream)
    ws = torch.empty(prob.workspace_bytes(), dtype=torch.uint8, device=dev)
    prob.set_workspace(ws)
    tt = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    d_nseg, d_ends, d_nodes = tt(nseg), tt(ends), tt(nodes)
    d_off, d_pends, d_pnodes = tt(p_off.view(np.int32)), tt(p_ends.view(np.int16)), tt(p_nodes)
    d_beta = torch.empty(N_PLANS, dtype=torch.float64, device=dev)
    d_pstat = torch.empty(N_PLANS, dtype=torch.uint8, device=dev)
    d_bb, d_bm, d_bc, d_bbw = tt(b_bits), tt(b_mem), tt(b_cap), tt(b_bw)
    o_beta = torch.empty(N_BATCH, dtype=torch.float64, device=dev)
    o_m = torch.empty(N_BATCH, dtype=torch.int32, device=dev)
    o_cuts = torch.empty(N_BATCH * (BATCH_K - 1), dtype=torch.int32, device=dev)
    o_place = torch.empty(N_BATCH * BATCH_K, dtype=torch.int32, device=dev)
    o_stat = torch.empty(N_BATCH, dtype=torch.int8, device=dev)
    d_sol = torch.zeros(ctypes.sizeof(pp.pp_solution) // 8, dtype=torch.float64, device=dev)
    d_sol2 = torch.zeros_like(d_sol)  # result record of the smaller configurations

    def batch_device():
        pp.solve_exact_batch_dev(N_BATCH, BATCH_L, BATCH_K, d_bb.data_ptr(), d_bm.data_ptr(),
                                 d_bc.data_ptr(), d_bbw.data_ptr(), o_beta.data_ptr(), o_m.data_ptr(),
                                 o_cuts.data_ptr(), o_place.data_ptr(), o_stat.data_ptr(),
                                 stream.cuda_stream)

    def eval_device():
        prob.eval_plans_packed_dev(N_PLANS, n_entries, d_nseg.data_ptr(), d_off.data_ptr(), d_pends.data_ptr(),
                                   d_pnodes.data_ptr(), d_beta.data_ptr(), d_pstat.data_ptr())

    def eval_device_int32():
        prob.eval_plans_dev(N_PLANS, d_nseg.data_ptr(), d_ends.data_ptr(), d_nodes.data_ptr(),
                            d_beta.data_ptr(), d_pstat.data_ptr())

    def step_device():
        prob.solve_exact_dev(d_sol.data_ptr())
        batch_device()
        eval_device()

    def barrier():
        torch.cuda.synchronize(dev)
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(dev)

    def max_over_ranks(x: float) -> float:
        if dist is None:
            return x
        t = torch.tensor([x], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    # ---- warm-up, then the timed region (device-resident inputs) ----
    warmup = max(args.warmup, 3)
    with torch.cuda.stream(stream):
        for _ in range(warmup):
            step_device()
        barrier()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with ClockSampler(local) as clocks:
            ev0.record(stream)
            for _ in range(args.steps):
                step_device()
            ev1.record(stream)
            barrier()
        ms_local = ev0.elapsed_time(ev1)
        ms_total = max_over_ranks(ms_local)
        clk = clocks.summary()
        prof = prob.last_solve_profile()
        # the batched solve of this shape: two preparing passes, one kernel per popcount level from 2 up,
        # the backtrack; the evaluator is one launch
        batch_launches = 2 + (min(BATCH_K, BATCH_L) - 1) + 1
        launches_per_step = prof.total_launches + batch_launches + 1
        if args.step_only:  # for a profiler's launch list: the warm-up and the timed steps, nothing else
            if rank == 0:
                print("step only: %d steps, %.4f ms per step, %d launches per step"
                      % (args.steps, max_over_ranks(ms_local) / args.steps, launches_per_step))
            if dist is not None:
                dist.destroy_process_group()
            return

        # per-part device times (same launch configuration, measured after the timed region): the
        # whole solve as the timed step runs it, then its phases with events between them (which
        # cost a few microseconds: a phase's kernels are then no longer launched under the tail of
        # the previous phase)
        sweep_ms, rank_ms, fin_ms, solve_ms = [], [], [], []
        for _ in range(9):
            prob.solve_exact_dev(d_sol.data_ptr())
            solve_ms.append(prob.last_solve_profile().ms_total)
        prob.set_profiling(True)
        for _ in range(7):
            prob.solve_exact_dev(d_sol.data_ptr())
            pr = prob.last_solve_profile()
            sweep_ms.append(pr.ms_sweep)
            rank_ms.append(pr.ms_rank)
            fin_ms.append(pr.ms_finalize)
        prob.set_profiling(False)
        e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)  # larger than the 126 MB L2
        batch_ms, eval_ms, eval_cold_ms = [], [], []
        for _ in range(7):
            e0.record(stream)
            batch_device()
            e1.record(stream)
            eval_device()
            e2.record(stream)
            stream.synchronize()
            batch_ms.append(e0.elapsed_time(e1))
            eval_ms.append(e1.elapsed_time(e2))
        eval32_cold_ms = []
        for _ in range(7):  # the evaluator alone with its plans evicted from L2 first; both row layouts
            flush.fill_(1)
            e0.record(stream)
            eval_device()
            e1.record(stream)
            stream.synchronize()
            eval_cold_ms.append(e0.elapsed_time(e1))
            flush.fill_(1)
            e0.record(stream)
            eval_device_int32()
            e1.record(stream)
            stream.synchronize()
            eval32_cold_ms.append(e0.elapsed_time(e1))

        # sustained leg: the Large solve back to back for about two seconds, clocks sampled meanwhile
        # (the sweep is bound by an ALU pipe, so its time follows the SM clock the part settles at)
        n_sus = max(50, int(2000.0 / statistics.median(solve_ms)))
        with ClockSampler(local) as sus_clocks:
            e0.record(stream)
            for _ in range(n_sus):
                prob.solve_exact_dev(d_sol.data_ptr())
            e1.record(stream)
            stream.synchronize()
        sus_ms = e0.elapsed_time(e1) / n_sus
        sus_clk = sus_clocks.summary()
        sustained = {"solves": n_sus, "large_solve_ms_sustained": sus_ms,
                     "sm_mhz_median": sus_clk["sm_mhz"] if sus_clk else None,
                     "ms_times_mhz": sus_ms * sus_clk["sm_mhz"] if sus_clk else None,
                     "reasons": sus_clk["reasons"] if sus_clk else None}

        # issue rate of the packed min/max forms the sweep is made of, measured now on this part
        rates = {"minmax_u16x2": pp.debug_minmax_rate(0), "min3_u16x2": pp.debug_minmax_rate(1),
                 "max3_u16x2": pp.debug_minmax_rate(2)}

        # the paper's greedy comparison baseline on the batched instances (not part of the timed
        # step): device time of one launch, and how far its plans are from the exact optimum
        g_beta, g_m, g_stat = torch.empty_like(o_beta), torch.empty_like(o_m), torch.empty_like(o_stat)
        g_cuts, g_place = torch.empty_like(o_cuts), torch.empty_like(o_place)
        greedy_ms = []
        for _ in range(7):
            e0.record(stream)
            pp.greedy_batch_dev(N_BATCH, BATCH_L, BATCH_K, d_bb.data_ptr(), d_bm.data_ptr(), d_bc.data_ptr(),
                                d_bbw.data_ptr(), g_beta.data_ptr(), g_m.data_ptr(), g_cuts.data_ptr(),
                                g_place.data_ptr(), g_stat.data_ptr(), stream.cuda_stream)
            e1.record(stream)
            stream.synchronize()
            greedy_ms.append(e0.elapsed_time(e1))
        both = (g_stat == 0) & (o_stat == 0) & (o_beta > 0)
        ratio = (g_beta[both] / o_beta[both]).cpu().numpy()
        greedy = {"launch_ms": min(greedy_ms[2:]), "instances_per_s": N_BATCH / (min(greedy_ms[2:]) * 1e-3),
                  "plans_found": int((g_stat == 0).sum().item()),
                  "plans_found_by_exact_search": int((o_stat == 0).sum().item()),
                  "beta_over_optimum_median": float(np.median(ratio)) if ratio.size else None,
                  "beta_over_optimum_mean": float(ratio.mean()) if ratio.size else None,
                  "optimal_fraction": float((ratio == 1.0).mean()) if ratio.size else None}

        # the paper's random comparison baseline on the Large instance (not part of the timed step):
        # N_PLANS plans generated on the device from seeded draws, scored by the evaluator
        h_draws = np.random.default_rng(4242).integers(0, 2**32, size=(N_PLANS, 2 * k), dtype=np.uint64)
        d_draws = torch.from_numpy(h_draws.astype(np.uint32).view(np.int32)).to(dev)
        r_nseg = torch.empty(N_PLANS, dtype=torch.uint8, device=dev)
        r_ends = torch.empty(N_PLANS * k, dtype=torch.int32, device=dev)
        r_nodes = torch.empty(N_PLANS * k, dtype=torch.int32, device=dev)
        r_beta, r_stat = torch.empty_like(d_beta), torch.empty_like(d_pstat)
        random_ms = []
        for _ in range(7):
            e0.record(stream)
            prob.random_plans_dev(N_PLANS, d_draws.data_ptr(), r_nseg.data_ptr(), r_ends.data_ptr(),
                                  r_nodes.data_ptr())
            e1.record(stream)
            stream.synchronize()
            random_ms.append(e0.elapsed_time(e1))
        prob.eval_plans_dev(N_PLANS, r_nseg.data_ptr(), r_ends.data_ptr(), r_nodes.data_ptr(),
                            r_beta.data_ptr(), r_stat.data_ptr())
        stream.synchronize()
        r_ok = r_beta[r_stat == 0]
        r_ms = min(random_ms[2:])
        r_bytes = N_PLANS * (2 * k * 4 + 1 + 2 * k * 4)  # draws in, nseg + two rows out
        random_base = {"launch_ms": r_ms, "plans_per_s": N_PLANS / (r_ms * 1e-3),
                       "algorithmic_GBps": r_bytes / (r_ms * 1e-3) / 1e9,
                       "frac_of_hbm_peak": r_bytes / (r_ms * 1e-3) / 1e9 / measured_peaks()[0]["hbm_gbs"],
                       "rows_with_a_plan": int((r_nseg > 0).sum().item()),
                       "plans_scored_finite": int(r_ok.numel()),
                       "best_beta_ms": float(r_ok.min().item()) if r_ok.numel() else None,
                       "median_beta_ms": float(r_ok.median().item()) if r_ok.numel() else None}

        # the smaller named configurations (parity-test cases, not part of the timed step): device
        # time of one exact solve each, for context
        other = {}
        for name, inst in (("tiny_k6_L12", W.config_tiny()), ("resnet50_shaped_k10_L50", W.config_resnet50_shaped()),
                           ("deeper_cnn_k14_L100", W.config_deeper_cnn()),
                           ("large_unequal_layer_memory_k18_L200", W.large_unequal_layers()),
                           ("geometric_graph_k14_64MB_L50", W.config_geometric(14, 64, 0))):
            with pp.Problem.from_instance(inst) as q:
                q.set_stream(stream.cuda_stream)
                if inst.k == k:
                    q.set_workspace(ws)  # the Large problem is idle here
                ts = []
                for _ in range(6):
                    q.solve_exact_dev(d_sol2.data_ptr())
                    ts.append(q.last_solve_profile().ms_total)
                qp = q.last_solve_profile()
                other[name] = {"solve_ms": min(ts[2:]), "relaxations_per_s": n_relax(inst.k, inst.L) / (min(ts[2:]) * 1e-3),
                               "state_bytes": qp.state_bytes, "fast_path": qp.fast_path, "pair_levels": qp.pair_levels}

        # the exact search under the paper's full objective, Eq. 1 (compute times of the partitions in the
        # bottleneck): host-pointer call, fp64 states, wall clock of the whole call; for context
        ct_inst = W.config_geometric(12, 64, 1)
        ct_work = (ct_inst.layer_mem_bytes // np.uint64(1024)).astype(np.uint64)
        ct_speed = (1000 + 37 * np.arange(ct_inst.k)).astype(np.uint32)
        ct_ts = []
        for _ in range(5):
            t_ct = time.perf_counter()
            ct_sol = pp.solve_exact_compute(ct_inst, ct_work, ct_speed)
            ct_ts.append((time.perf_counter() - t_ct) * 1e3)
        other["eq1_compute_term_geometric_k12_L50"] = {
            "call_ms": min(ct_ts[1:]), "relaxations_per_s": n_relax(ct_inst.k, ct_inst.L) / (min(ct_ts[1:]) * 1e-3),
            "state_bytes": 8, "status": int(ct_sol.status), "m": int(ct_sol.m)}

        # the paper's own two-stage heuristic (Algorithm 1, then Algorithms 2 and 3) against the exact
        # optimum on the evaluation setting of its Section 4: 14 devices of 32 MB on a random geometric
        # graph, the ResNet50-shaped chain; not part of the timed step
        h_ratios, h_failed = [], 0
        draws_rng = np.random.default_rng(777)
        for seed in range(8):
            gi = W.config_geometric(14, 32, seed, link="pairwise")
            part = pp.partition_minsum_batch(gi.layer_out_bits[None, :], gi.layer_mem_bytes[None, :],
                                             gi.node_mem_bytes[:1].copy(), gi.L)
            gm = int(part.m[0])
            if part.status[0] != 0 or gm > gi.k:
                h_failed += 1
                continue
            h_draws = draws_rng.integers(0, 2**32, size=(24, gi.k), dtype=np.uint64).astype(np.uint32)
            st, h_nodes, _ = pp.kpath_matching(gi.bw_kbps, part.sizes[0, :gm - 1], 3, h_draws, stream.cuda_stream)
            if st != 0:
                h_failed += 1
                continue
            g_ends = np.full((1, gi.k), -1, np.int32)
            g_nd = np.full((1, gi.k), -1, np.int32)
            g_ends[0, :gm - 1] = part.cuts[0, :gm - 1]
            g_nd[0, :gm] = h_nodes
            with pp.Problem.from_instance(gi) as q:
                q.set_stream(stream.cuda_stream)
                hb, hf = q.eval_plans(np.array([gm], np.uint8), g_ends, g_nd)
                ex = q.solve_exact()
            if hf[0] == 0 and ex.status == 0 and ex.beta_ms > 0:
                h_ratios.append(float(hb[0] / ex.beta_ms))
        heuristic = {"instances": 8, "no_plan": h_failed,
                     "beta_over_optimum_median": float(np.median(h_ratios)) if h_ratios else None,
                     "beta_over_optimum_mean": float(np.mean(h_ratios)) if h_ratios else None,
                     "beta_over_optimum_max": float(np.max(h_ratios)) if h_ratios else None,
                     "setting": "ResNet50-shaped chain, 14 devices of 32 MB, geometric graph (pairwise Eq. 12), "
                                "3 classes, 24 colourings per probe"}

        # the kernels behind the two stages, timed in bulk on the device (not part of the timed step):
        # Algorithm 1 on 4096 copies of the ResNet50-shaped chain with capacities of 16..271 MB, and the
        # colour-coding k-path query (paths of 8 vertices) 4096 times on a 50-node geometric graph
        def timed(fn, reps=7):
            ts = []
            for _ in range(reps):
                a, b2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                fn()
                b2.record(stream)
                b2.synchronize()
                ts.append(a.elapsed_time(b2))
            return statistics.median(ts[2:])

        chain = W.config_resnet50_shaped()
        n_ch, Lc = 4096, chain.L
        c_w = tt(np.tile(chain.layer_out_bits, (n_ch, 1)))
        c_m = tt(np.tile(chain.layer_mem_bytes, (n_ch, 1)))
        c_kap = tt((np.arange(n_ch, dtype=np.uint64) % 256 + 16) * np.uint64(1 << 20))
        c_cost = torch.empty(n_ch, dtype=torch.int64, device=dev)
        c_m_out = torch.empty(n_ch, dtype=torch.int32, device=dev)
        c_cuts = torch.empty(n_ch * Lc, dtype=torch.int32, device=dev)
        c_sizes = torch.empty(n_ch * Lc, dtype=torch.int64, device=dev)
        c_stat = torch.empty(n_ch, dtype=torch.int8, device=dev)
        part_ms = timed(lambda: pp.partition_minsum_batch_dev(
            n_ch, Lc, c_w.data_ptr(), c_m.data_ptr(), c_kap.data_ptr(), Lc, c_cost.data_ptr(), c_m_out.data_ptr(),
            c_cuts.data_ptr(), c_sizes.data_ptr(), c_stat.data_ptr(), stream.cuda_stream))
        g50, _ = W.geometric_bandwidths(50, 5, link="pairwise")
        n_q, kk_path = 4096, 8
        q_rng = np.random.default_rng(4242)
        q_thr = tt(np.full(n_q, int(np.median(g50[g50 > 0])), dtype=np.uint32))
        q_any = tt(np.full(n_q, -1, dtype=np.int32))
        q_alive = tt(np.full(n_q, (1 << 50) - 1, dtype=np.uint64).view(np.int64))
        q_col = tt(q_rng.integers(0, kk_path, size=(n_q, 50), dtype=np.uint8))
        q_bw = tt(g50.astype(np.uint32))
        q_found = torch.empty(n_q, dtype=torch.uint8, device=dev)
        q_path = torch.empty(n_q * kk_path, dtype=torch.int32, device=dev)
        kpath_ms = timed(lambda: pp.kpath_colour_batch_dev(
            50, q_bw.data_ptr(), n_q, kk_path, q_thr.data_ptr(), q_any.data_ptr(), q_any.data_ptr(),
            q_alive.data_ptr(), q_col.data_ptr(), q_found.data_ptr(), q_path.data_ptr(), stream.cuda_stream))
        heuristic["stage_kernels"] = {
            "partition_minsum": {"chains": n_ch, "L": Lc, "ms": part_ms, "chains_per_s": n_ch / (part_ms * 1e-3),
                                 "feasible": int((c_stat == 0).sum().item())},
            "kpath_colour": {"queries": n_q, "nodes": 50, "path_vertices": kk_path, "ms": kpath_ms,
                             "queries_per_s": n_q / (kpath_ms * 1e-3), "found": int(q_found.sum().item())}}

    sol_rec = pp.pp_solution.from_buffer_copy(d_sol.cpu().numpy().tobytes())
    ms_per_step = ms_total / args.steps
    value, _ = aggregate_over_ranks(relax_step * args.steps, ms_local * 1e-3, dist, dev)

    # ---- end to end through the host-pointer entry points ----
    h2d = (large.layer_out_bits.nbytes + large.layer_mem_bytes.nbytes + large.node_mem_bytes.nbytes
           + large.bw_kbps.nbytes + nseg.nbytes + p_off.nbytes + p_ends.nbytes + p_nodes.nbytes
           + b_bits.nbytes + b_mem.nbytes + b_cap.nbytes + b_bw.nbytes)
    d2h = (ctypes.sizeof(pp.pp_solution) + N_PLANS * 9
           + N_BATCH * (8 + 4 + 4 * (BATCH_K - 1) + 4 * BATCH_K + 1))

    # the step's inputs live in pinned host memory; the C entry points copy them to the device
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory().numpy()
    h_bits, h_mem, h_cap, h_bw = (pin(a) for a in (large.layer_out_bits, large.layer_mem_bytes,
                                                    large.node_mem_bytes, large.bw_kbps))
    h_nseg, h_off, h_pends, h_pnodes = pin(nseg), pin(p_off.view(np.int32)).view(np.uint32), \
        pin(p_ends.view(np.int16)).view(np.uint16), pin(p_nodes)
    hb_bits, hb_mem, hb_cap, hb_bw = pin(b_bits), pin(b_mem), pin(b_cap), pin(b_bw)

    h_beta = torch.empty(N_PLANS, dtype=torch.float64).pin_memory().numpy()  # results land in pinned memory too
    h_pstat = torch.empty(N_PLANS, dtype=torch.uint8).pin_memory().numpy()

    def step_host():
        with pp.Problem(L, h_bits, h_mem, k, h_cap, h_bw) as p2:
            p2.set_workspace(ws)
            s = p2.solve_exact()
            bsol = pp.solve_exact_batch(BATCH_L, BATCH_K, hb_bits, hb_mem, hb_cap, hb_bw)
            beta, pstat = p2.eval_plans_packed(h_nseg, h_off, h_pends, h_pnodes, out=(h_beta, h_pstat))
        return s, bsol, beta, pstat

    for _ in range(2):
        host_out = step_host()
    barrier()
    t0 = time.perf_counter()
    e2e_steps = max(2, min(args.steps, 10))
    for _ in range(e2e_steps):
        host_out = step_host()
    barrier()
    e2e_local = (time.perf_counter() - t0) / e2e_steps
    e2e_value, e2e_s = aggregate_over_ranks(relax_step, e2e_local, dist, dev)
    assert host_out[0].beta_ms == sol_rec.beta_ms and host_out[0].m == sol_rec.m

    # ---- roofline ----
    # The DP roofline is the slower of (state bytes at HBM bandwidth) and (min/max element-ops at the
    # ALU rate): every state is written once and read once (2 * states * element bytes); a
    # relaxation is one max and one min, the window step about three more ops per state.  The ALU
    # rate is the packed min/max issue rate measured above x 32 lanes x 2 elements x SMs x max clock.
    peaks, which = measured_peaks()
    med = statistics.median
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    clock_hz = peaks.get("sm_max_mhz", 1965.0) * 1e6
    minmax_rate = min(rates["minmax_u16x2"], rates["min3_u16x2"])  # warp instructions per clock per SM
    alu_peak = minmax_rate * 32 * 2 * sms * clock_hz             # element-ops per second

    def dp_roofline(kk, LL, elem_bytes, solve_ms_):
        bytes_ = 2 * n_states(kk, LL) * elem_bytes
        ops_ = 2 * n_relax(kk, LL) + 3 * n_states(kk, LL)
        t_mem = bytes_ / (peaks["hbm_gbs"] * 1e9) * 1e3
        t_mem_nom = bytes_ / (NOMINAL_HBM_GBS * 1e9) * 1e3
        t_alu = ops_ / alu_peak * 1e3
        return {"algorithmic_bytes": bytes_, "algorithmic_ops": ops_, "t_mem_ms": t_mem, "t_alu_ms": t_alu,
                "t_mem_ms_at_8TBps": t_mem_nom, "bound": "hbm" if t_mem >= t_alu else "alu",
                "solve_ms": solve_ms_, "frac": max(t_mem, t_alu) / solve_ms_,
                "frac_at_8TBps": max(t_mem_nom, t_alu) / solve_ms_}

    elem = prof.state_bytes
    sweep_t = med(sweep_ms) * 1e-3
    whole = dp_roofline(k, L, elem, med(solve_ms))
    alg_bytes = whole["algorithmic_bytes"]
    alu_ops = whole["algorithmic_ops"]
    n_launch = prof.sweep_launches
    if whole["bound"] == "hbm":
        achieved, peak, unit = alg_bytes / sweep_t / 1e9, peaks["hbm_gbs"], "GB/s"
    else:
        achieved, peak, unit = alu_ops / sweep_t / 1e12, alu_peak / 1e12, "Tops/s"
    roofline = {"bound": whole["bound"], "achieved": achieved, "peak": peak, "unit": unit,
                "frac": achieved / peak,
                "traffic": SWEEP_DRAM_BYTES_PER_LAUNCH if prof.fast_path else None,
                "peak_source": (which + " (burst copy figure; the sweep is timed alone)") if whole["bound"] == "hbm"
                               else "measured in this run (packed min/max issue rate x max SM clock)",
                "kernel": "k_sweep_pair + k_sweep_fast (%d launches per solve, one per popcount level)" % n_launch,
                "algorithmic_bytes_per_launch": alg_bytes / n_launch,
                "ms_per_launch": sweep_t * 1e3 / n_launch,
                "algorithmic_bytes_per_solve": alg_bytes, "sweep_ms": sweep_t * 1e3,
                "hbm": {"achieved_GBps": alg_bytes / sweep_t / 1e9, "peak_GBps": peaks["hbm_gbs"],
                        "frac": alg_bytes / sweep_t / 1e9 / peaks["hbm_gbs"], "peak_source": which},
                "alu": {"ops_per_solve": alu_ops, "achieved_ops_per_s": alu_ops / sweep_t,
                        "peak_ops_per_s": alu_peak, "frac": alu_ops / sweep_t / alu_peak,
                        "warp_instr_per_clk_per_sm": rates, "lanes_per_clk_per_sm": minmax_rate * 32,
                        "peak_source": "measured in this run"},
                "whole_solve": whole,
                "sustained": sustained}
    # the other parts of the step against their own bounds
    c3 = W.config_deeper_cnn()
    o3 = other["deeper_cnn_k14_L100"]
    unl = other["large_unequal_layer_memory_k18_L200"]
    # per plan: nseg, its offset, nseg - 1 cuts of 2 bytes, nseg nodes of 1 byte in; beta and flags out
    plan_bytes = 5 * N_PLANS + 3 * n_entries - 2 * int((np.diff(p_off.astype(np.int64)) > 0).sum()) + 9 * N_PLANS
    ev_cold = med(eval_cold_ms) * 1e-3
    batch_ops = N_BATCH * (2 * n_relax(BATCH_K, BATCH_L) + 3 * n_states(BATCH_K, BATCH_L))
    part_rooflines = {
        "deeper_cnn_k14_L100": dp_roofline(c3.k, c3.L, o3["state_bytes"], o3["solve_ms"]),
        "large_unequal_layer_memory_k18_L200": dp_roofline(k, L, unl["state_bytes"], unl["solve_ms"]),
        "evaluator": {"bound": "hbm", "algorithmic_bytes": plan_bytes, "bytes_per_plan": plan_bytes / N_PLANS,
                      "ms_cold": ev_cold * 1e3, "achieved_GBps": plan_bytes / ev_cold / 1e9,
                      "frac": plan_bytes / ev_cold / 1e9 / peaks["hbm_gbs"],
                      "note": "inputs evicted from L2 before each timed launch; eval_ms in the breakdown is "
                              "the launch inside the step, whose inputs may still be L2-resident"},
        "batch": {"bound": "alu", "algorithmic_ops": batch_ops, "t_alu_ms": batch_ops / alu_peak * 1e3,
                  "batch_ms": med(batch_ms), "frac": batch_ops / alu_peak * 1e3 / med(batch_ms)},
    }

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u16" if elem == 2 else "u32",
        "data": "synthetic",
        "config": {"workload": WORKLOAD,
                   "relaxations_per_step": relax_step, "states_large": n_states(k, L),
                   "l2": "state table of %.2f GB per solve exceeds the 126 MB L2; no explicit flush"
                         % (alg_bytes / 2 / 1e9),
                   "parallelism": "replicas only" if world > 1 else "single GPU"},
        "gpu_launches": launches_per_step * args.steps,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(h2d),
                "d2h_bytes_per_step": int(d2h), "ms_per_step": e2e_s * 1e3,
                "workspace": "the %.2f GB search scratch is allocated once by the caller and handed to every "
                             "step's problem (pp_problem_set_workspace); it is not part of the timed copies"
                             % (prob.workspace_bytes() / 1e9)},
        "clocks": clk,
        "roofline": roofline,
        "breakdown": {
            "large_solve_ms": med(solve_ms), "rank_build_ms": med(rank_ms),
            "sweep_ms": med(sweep_ms), "finalize_ms": med(fin_ms),
            "large_relaxations_per_s": relax_large / (med(solve_ms) * 1e-3),
            "batch_ms": med(batch_ms), "instances_per_s": N_BATCH / (med(batch_ms) * 1e-3),
            "eval_ms": med(eval_ms), "plans_per_s": N_PLANS / (med(eval_ms) * 1e-3),
            "eval_cold_ms": med(eval_cold_ms), "plans_per_s_cold": N_PLANS / (med(eval_cold_ms) * 1e-3),
            "eval_int32_rows_cold_ms": med(eval32_cold_ms),
            "batch_roofline": part_rooflines["batch"],
            "part_rooflines": part_rooflines,
            "fast_path": prof.fast_path, "beta_ms": sol_rec.beta_ms, "segments": sol_rec.m,
            "greedy_baseline_batched": greedy,
            "random_baseline_large": random_base,
            "paper_heuristic_geometric": heuristic,
            "other_configs": other,
        },
    }
    if rank == 0 and world == 1 and not args.no_cpu:
        out["cpu_baseline"] = cpu_baseline(large)
    if rank == 0:
        print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


def cpu_baseline(large):
    """The oracle as it stands, timed on the host cores on the Large instance (one full solve)."""
    import oracle
    threads = oracle.max_threads()
    t0 = time.perf_counter()
    sol = oracle.dp_fact(large, threads)
    dt = time.perf_counter() - t0
    return {"value": n_relax(large.k, large.L) / dt, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": "one full factorised-DP solve of the Large instance (k=18, L=200), OpenMP",
            "seconds": dt, "beta_ms": sol.beta_ms}


def run_reference(args):
    """CPU oracle arm: each step is a bounded sample of the step above -- the Large instance
    restricted to its first 15 nodes, 64 of the batched instances, 2048 of the candidate plans."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    large = W.config_large()
    ksub = 15
    sub = W.Instance(large.L, ksub, large.layer_out_bits, large.layer_mem_bytes,
                     large.node_mem_bytes[:ksub].copy(),
                     np.ascontiguousarray(large.bw_kbps[:ksub, :ksub]), "large[:15 nodes]")
    batch = W.config_batched(64, BATCH_L, BATCH_K)
    nseg, ends, nodes = W.random_plans(large, 2048, seed=77, invalid_fraction=0.05)
    threads = oracle.max_threads()
    relax_step = n_relax(ksub, large.L) + 64 * n_relax(BATCH_K, BATCH_L)

    def step():
        oracle.dp_fact(sub, threads)
        for inst in batch:
            oracle.dp_fact(inst, 1)
        oracle.eval_plans(large, nseg, ends, nodes)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = (time.perf_counter() - t0) / args.steps
    value = relax_step / dt
    sample = ("per step: factorised DP on the Large instance restricted to its first 15 nodes, "
              "64 batched instances, 2048 candidate plans")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def run_only(args):
    """Small single-part runs for profilers (no timing, no JSON line): the Large instance restricted
    to its first --k nodes (k = 16: a 0.44 GB state table, far above the L2 and small enough for a
    multi-pass counter capture of single sweep launches), the batched solve, or one of the two
    comparison baselines."""
    import torch

    import paper_2210_12219_b200 as pp
    from paper_2210_12219_b200 import build as pp_build

    pp_build.build()
    if args.only in ("batch", "greedy"):
        insts = W.config_batched(args.batch)
        b_bits, b_mem, b_cap, b_bw = stack(insts)
        entry = pp.greedy_batch if args.only == "greedy" else pp.solve_exact_batch
        for _ in range(args.solves):
            got = entry(BATCH_L, BATCH_K, b_bits, b_mem, b_cap, b_bw)
        print("%s of %d: %d with a plan" % (args.only, args.batch, int((got.status == 0).sum())))
        return
    if args.only == "partition":  # Algorithm 1 on --batch copies of the ResNet50-shaped chain
        chain = W.config_resnet50_shaped()
        kap = (np.arange(args.batch, dtype=np.uint64) % 256 + 16) * np.uint64(1 << 20)
        for _ in range(args.solves):
            got = pp.partition_minsum_batch(np.tile(chain.layer_out_bits, (args.batch, 1)),
                                            np.tile(chain.layer_mem_bytes, (args.batch, 1)), kap, chain.L)
        print("partition of %d chains: %d feasible" % (args.batch, int((got.status == 0).sum())))
        return
    if args.only == "kpath":  # colour-coding k-path, --batch random colourings on a 50-node geometric graph
        g50, _ = W.geometric_bandwidths(50, 5, link="pairwise")
        rng = np.random.default_rng(4242)
        Q, kk = args.batch, 8
        for _ in range(args.solves):
            found, _ = pp.kpath_colour_batch(g50, kk, np.full(Q, int(np.median(g50[g50 > 0])), np.uint32),
                                             np.full(Q, -1, np.int32), np.full(Q, -1, np.int32),
                                             np.full(Q, (1 << 50) - 1, np.uint64),
                                             rng.integers(0, kk, size=(Q, 50), dtype=np.uint8))
        print("k-path of %d queries: %d found" % (Q, int(found.sum())))
        return
    large = W.config_large()
    k = args.k
    inst = W.Instance(large.L, k, large.layer_out_bits, large.layer_mem_bytes,
                      large.node_mem_bytes[:k].copy(), np.ascontiguousarray(large.bw_kbps[:k, :k]))
    if args.only == "unequal":  # same sizes, layers of unequal memory: the general-window kernels
        inst = W.large_unequal_layers(k)
    if args.only == "random":
        draws = np.random.default_rng(4242).integers(0, 2**32, size=(args.plans, 2 * k), dtype=np.uint64)
        with pp.Problem.from_instance(inst) as p:
            for _ in range(args.solves):
                nseg, _, _ = p.random_plans(draws.astype(np.uint32))
        print("%d random plans: %d rows with a plan" % (args.plans, int((nseg > 0).sum())))
        return
    sol = torch.zeros(ctypes.sizeof(pp.pp_solution) // 8, dtype=torch.float64, device="cuda")
    with pp.Problem.from_instance(inst) as p:
        if args.mode is not None:
            p.force_generic(args.mode)
        for _ in range(args.solves):
            p.solve_exact_dev(sol.data_ptr())
        torch.cuda.synchronize()
        prof = p.last_solve_profile()
        rec = pp.pp_solution.from_buffer_copy(sol.cpu().numpy().tobytes())
        print("k=%d L=%d beta=%.6f m=%d sweep=%.3f ms total=%.3f ms fast=%d pair_levels=%d" %
              (k, inst.L, rec.beta_ms, rec.m, prof.ms_sweep, prof.ms_total, prof.fast_path, prof.pair_levels))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-baseline leg")
    ap.add_argument("--step-only", action="store_true",
                    help="run the warm-up and the timed steps and exit (for a profiler's launch list)")
    ap.add_argument("--only", choices=["sweep", "unequal", "batch", "greedy", "random", "partition", "kpath"],
                    help="profiler helper: run one part a few times and exit (see run_only)")
    ap.add_argument("--k", type=int, default=16, help="--only sweep/unequal/random: nodes kept of the Large instance")
    ap.add_argument("--solves", type=int, default=2, help="--only: repetitions")
    ap.add_argument("--mode", type=int, default=None, help="--only sweep: pp_problem_force_generic mode")
    ap.add_argument("--batch", type=int, default=N_BATCH, help="--only batch/greedy/partition/kpath: instances, chains or queries")
    ap.add_argument("--plans", type=int, default=N_PLANS, help="--only random: plans")
    args = ap.parse_args()
    if args.only:
        run_only(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
