"""GPU parity: the CUDA library (through its C-ABI) against the CPU oracle, bit for bit.

beta is an fp64 quotient selected by min/max on both sides, plans are integers: every
comparison here is exact equality (tolerance 0)."""
from __future__ import annotations

import numpy as np
import pytest

import oracle
import paper_2210_12219_b200 as pp
from paper_2210_12219_b200 import build
from paper_2210_12219_b200 import workloads as W
from tests.helpers import make_instance, parse_golden

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    pp.lib()


def gpu_solve(inst, generic=None):
    with pp.Problem.from_instance(inst) as p:
        if generic is not None:
            p.force_generic(1 if generic else 0)
        return p.solve_exact()


def assert_same(inst, got, want):
    assert got.status == want.status, inst.name
    assert got.beta_ms == want.beta_ms or (np.isinf(got.beta_ms) and np.isinf(want.beta_ms)), inst.name
    assert got.plan() == want.plan(), inst.name
    k = inst.k
    assert (got.cuts[max(got.m - 1, 0):] == -1).all() and (got.placement[got.m:] == -1).all()
    assert len(got.cuts) == k - 1 and len(got.placement) == k


def test_hand_worked_fixtures():
    _, cases = parse_golden()
    for inst, plans, optimum in cases:
        want_beta, m, cuts, nodes = optimum
        got = gpu_solve(inst)
        assert got.beta_ms == want_beta and got.plan() == (m, tuple(cuts), tuple(nodes))
        assert got.status == (pp.PP_INFEASIBLE if m == 0 else pp.PP_OK)
        with pp.Problem.from_instance(inst) as p:
            B = len(plans)
            nseg = np.array([q[0] for q in plans], dtype=np.uint8)
            ends = np.full((B, inst.k), -1, dtype=np.int32)
            nd = np.full((B, inst.k), -1, dtype=np.int32)
            for b, (ns, cu, no, _, _) in enumerate(plans):
                ends[b, :min(len(cu), inst.k)] = cu[:inst.k]
                nd[b, :min(len(no), inst.k)] = no[:inst.k]
            beta, status = p.eval_plans(nseg, ends, nd)
            for b, (_, _, _, wb, wf) in enumerate(plans):
                assert status[b] == wf and beta[b] == wb


def test_tiny_config_matches_bruteforce_and_dp():
    inst = W.config_tiny()
    got = gpu_solve(inst)
    assert_same(inst, got, oracle.bruteforce(inst))
    assert_same(inst, got, oracle.dp_naive(inst))


@pytest.mark.parametrize("generic", [True, False])
def test_random_small_instances(generic):
    n_inf = 0
    seed = 0
    for L, k, n in ((1, 1, 2), (1, 4, 2), (2, 2, 4), (5, 3, 20), (7, 4, 30), (12, 6, 30), (9, 5, 30),
                    (3, 6, 10), (17, 5, 20), (33, 4, 10), (16, 7, 10), (40, 3, 6)):
        for i in range(n):
            kind = i % 4
            inst = W.random_small(20000 + seed, L, k, tight=(kind == 1), ties=(kind == 2),
                                  dead_links=0.3 if kind == 3 else 0.0)
            seed += 1
            want = oracle.dp_naive(inst)
            assert_same(inst, gpu_solve(inst, generic), want)
            n_inf += want.status == oracle.INFEASIBLE
    assert seed >= 170 and n_inf >= 5


def _compare_rows(inst, p, rows):
    want = oracle.dp_fact(inst, 4, want_table=True).table
    for S, v in rows:
        got = p.debug_read_state_row(S, v)
        assert np.array_equal(got, want[S, v]), (inst.name, S, v)


@pytest.mark.parametrize("generic", [True, False])
def test_state_table_element_by_element(generic):
    # every state of small instances, sampled rows of configs 2 and 3 (several tiles of masks,
    # ragged rows: L = 12, 50, 100 are not multiples of the 16-element row padding)
    rng = np.random.default_rng(3)
    for inst in (W.config_tiny(), W.random_small(30000, 19, 5, tight=True),
                 W.random_small(30001, 8, 6, dead_links=0.3)):
        with pp.Problem.from_instance(inst) as p:
            p.force_generic(1 if generic else 0)
            p.solve_exact()
            rows = [(S, v) for S in range(1, 1 << inst.k) for v in range(inst.k)
                    if S >> v & 1 and bin(S).count("1") <= inst.L]
            _compare_rows(inst, p, rows)
    for inst in (W.config_resnet50_shaped(), W.config_deeper_cnn()):
        with pp.Problem.from_instance(inst) as p:
            p.force_generic(1 if generic else 0)
            want = oracle.dp_fact(inst, 8)
            assert_same(inst, p.solve_exact(), want)
            rows = []
            while len(rows) < 120:
                S = int(rng.integers(1, 1 << inst.k))
                vs = [v for v in range(inst.k) if S >> v & 1]
                rows.append((S, int(rng.choice(vs))))
            rows.append(((1 << inst.k) - 1, inst.k - 1))
            _compare_rows(inst, p, rows)


def test_register_tiled_sweep_on_uniform_memory_chains():
    # chains of identical layers take the register-tiled sweep kernel; rows of every raggedness
    # (L not a multiple of 8 or 16, one lane up to all 32 lanes), every window remainder r = W % 8
    # and block count q = W // 8, windows wider than the chain, ties and dead links
    n_fast = n_pair = 0
    seed = 0
    for L, k, wmin, wmax, n in ((9, 3, 8, 9, 6), (12, 5, 8, 10, 10), (17, 6, 8, 13, 10), (31, 4, 8, 16, 12),
                                (40, 6, 8, 30, 10), (64, 5, 9, 40, 8), (100, 7, 8, 60, 6),
                                (129, 4, 8, 70, 6), (200, 6, 21, 85, 4), (239, 3, 8, 140, 6),
                                (240, 4, 15, 300, 4), (23, 2, 8, 14, 6), (50, 5, 8, 60, 6)):
        for i in range(n):
            inst = W.uniform_memory_small(80000 + seed, L, k, wmin, wmax, ties=(i % 3 == 1),
                                          dead_links=0.25 if i % 3 == 2 else 0.0)
            seed += 1
            want = oracle.dp_fact(inst, 4, want_table=(L * (1 << k) <= 16384))
            with pp.Problem.from_instance(inst) as p:
                got = p.solve_exact()
                assert p.last_solve_profile().fast_path == 1, inst.name
                n_fast += 1
                assert_same(inst, got, want)
                if want.table is not None:
                    for S in range(1, 1 << k):
                        for v in range(k):
                            if S >> v & 1 and bin(S).count("1") <= L:
                                assert np.array_equal(p.debug_read_state_row(S, v), want.table[S, v]), \
                                    (inst.name, S, v)
                # the kernel that takes two source masks per warp, forced onto every level it can run
                p.force_generic(3)
                assert_same(inst, p.solve_exact(), want)
                prof = p.last_solve_profile()
                assert prof.fast_path == 1 and prof.pair_levels == max(0, min(k, L, 14) - 2), inst.name
                n_pair += prof.pair_levels > 0
                if want.table is not None:
                    for S in range(1, 1 << k):
                        for v in range(k):
                            if S >> v & 1 and bin(S).count("1") <= L:
                                assert np.array_equal(p.debug_read_state_row(S, v), want.table[S, v]), \
                                    (inst.name, S, v, "two-mask kernel")
                p.force_generic(1)
                assert_same(inst, p.solve_exact(), want)
                assert p.last_solve_profile().fast_path == 0
    assert n_fast >= 80 and n_pair >= 70
    # a node whose window is narrower than 8 layers takes the general-window variant
    inst = W.uniform_memory_small(81000, 30, 4, 3, 7)
    with pp.Problem.from_instance(inst) as p:
        assert_same(inst, p.solve_exact(), oracle.dp_fact(inst))
        assert p.last_solve_profile().fast_path == 2


def test_register_tiled_sweep_with_general_windows():
    # arbitrary layer memories: window starts come from the staged window table; includes
    # windows of one position up to the whole chain (every level count of the sparse table),
    # empty windows, windows reaching layer 0, L from one lane to 30 lanes, and every state
    # compared on the small ones
    seed = 0
    for L, k, n in ((5, 3, 8), (9, 4, 10), (17, 5, 10), (33, 6, 10), (64, 6, 6), (100, 7, 5), (150, 5, 5),
                    (199, 4, 5), (240, 4, 4), (12, 8, 6), (50, 10, 2)):
        for i in range(n):
            kind = i % 4
            inst = W.random_small(85000 + seed, L, k, tight=(kind == 1), ties=(kind == 2),
                                  dead_links=0.3 if kind == 3 else 0.0)
            if kind == 0 and L >= 30:  # long windows: a few nodes hold most of the chain
                cap = inst.node_mem_bytes.copy()
                cap[: max(1, k // 2)] = np.uint64(int(inst.layer_mem_bytes.sum()) // 2)
                inst = make_instance(inst.layer_out_bits, inst.layer_mem_bytes, cap, inst.bw_kbps, inst.name)
            seed += 1
            want = oracle.dp_fact(inst, 4, want_table=(L * (1 << k) <= 16384))
            with pp.Problem.from_instance(inst) as p:
                got = p.solve_exact()
                assert p.last_solve_profile().fast_path == 2, inst.name
                assert_same(inst, got, want)
                if want.table is not None:
                    for S in range(1, 1 << k):
                        for v in range(k):
                            if S >> v & 1 and bin(S).count("1") <= L:
                                assert np.array_equal(p.debug_read_state_row(S, v), want.table[S, v]), \
                                    (inst.name, S, v)
    for inst in (W.config_resnet50_shaped(), W.config_deeper_cnn()):
        with pp.Problem.from_instance(inst) as p:
            assert_same(inst, p.solve_exact(), oracle.dp_fact(inst, 8))
            assert p.last_solve_profile().fast_path == 2


def test_named_configs_2_and_3():
    for inst in (W.config_resnet50_shaped(), W.config_deeper_cnn()):
        want = oracle.dp_fact(inst, 8)
        got = gpu_solve(inst)
        assert_same(inst, got, want)
        assert oracle.eval_plan(inst, *got.plan()) == (got.beta_ms, 0)


def test_geometric_workload_of_section_4():
    # the paper's evaluation graph (random positions, Shannon-capacity links, equal node memory), both
    # readings of how a pair's bandwidth follows from Eq. 12; state rows compared on the k = 14 one
    for inst in (W.config_geometric(14, 64, 0), W.config_geometric(10, 64, 1, link="pairwise"),
                 W.config_geometric(12, 128, 2), W.config_geometric(9, 512, 3)):
        want = oracle.dp_fact(inst, 8)
        assert_same(inst, gpu_solve(inst), want)
        assert_same(inst, gpu_solve(inst, generic=True), want)
    inst = W.config_geometric(14, 64, 0)
    rng = np.random.default_rng(14)
    with pp.Problem.from_instance(inst) as p:
        p.solve_exact()
        rows = []
        while len(rows) < 60:
            S = int(rng.integers(1, 1 << inst.k))
            rows.append((S, int(rng.choice([v for v in range(inst.k) if S >> v & 1]))))
        _compare_rows(inst, p, rows)


def _sub_instance(inst, nodes):
    idx = np.array(nodes)
    return make_instance(inst.layer_out_bits, inst.layer_mem_bytes, inst.node_mem_bytes[idx],
                         inst.bw_kbps[np.ix_(idx, idx)], f"{inst.name}-sub")


def test_large_config_full_size():
    # config 5 (k = 18, L = 200) in the launch configuration the benchmark times.  The oracle
    # solves the whole instance for beta* and the plan; single states are checked on sampled
    # rows: the states of a node subset are exactly the table of the instance restricted to
    # those nodes, which the oracle can afford for up to 8 nodes.
    inst = W.config_large()
    want = oracle.dp_fact(inst, oracle.max_threads())
    from tests.test_workloads_golden import read_golden
    checksum, g_beta, g_m, g_cuts, g_nodes = read_golden()["large"]
    assert inst.checksum() == checksum and want.beta_ms == g_beta and want.plan() == (g_m, g_cuts, g_nodes)
    with pp.Problem.from_instance(inst) as p:
        got = p.solve_exact()
        assert_same(inst, got, want)
        assert oracle.eval_plan(inst, *got.plan()) == (got.beta_ms, 0)
        prof = p.last_solve_profile()
        assert prof.state_bytes == 2 and prof.fast_path == 1 and prof.pair_levels >= 6
        rng = np.random.default_rng(9)
        for size in (1, 2, 3, 5, 7, 8):
            nodes = sorted(int(x) for x in rng.choice(inst.k, size=size, replace=False))
            sub = _sub_instance(inst, nodes)
            table = oracle.dp_fact(sub, 4, want_table=True).table
            S = sum(1 << n for n in nodes)
            for j, n in enumerate(nodes):
                assert np.array_equal(p.debug_read_state_row(S, n), table[(1 << size) - 1, j])
        # second solve on the same handle gives the same answer (scratch is reused)
        assert_same(inst, p.solve_exact(), want)
        # the same instance with every level on the kernel that takes one source mask per warp
        p.force_generic(2)
        assert_same(inst, p.solve_exact(), want)
        prof = p.last_solve_profile()
        assert prof.fast_path == 1 and prof.pair_levels == 0
        S = sum(1 << n for n in nodes)
        for j, n in enumerate(nodes):
            assert np.array_equal(p.debug_read_state_row(S, n), table[(1 << len(nodes)) - 1, j])


def test_maximum_sizes():
    # k at the library limit (20 nodes, every sweep instantiation up to 19 source nodes) on a
    # short uniform-memory chain, and L at the limit (1024 layers) on few nodes
    inst = W.uniform_memory_small(90000, 16, pp.PP_MAX_K, 8, 12)
    want = oracle.dp_fact(inst, oracle.max_threads())
    with pp.Problem.from_instance(inst) as p:
        got = p.solve_exact()
        assert p.last_solve_profile().fast_path == 1
        assert_same(inst, got, want)
        p.force_generic(1)
        assert_same(inst, p.solve_exact(), want)
    base = W.random_small(90001, pp.PP_MAX_L, 3)
    cap = np.full(3, int(base.layer_mem_bytes.sum()) // 2, dtype=np.uint64)
    inst = make_instance(base.layer_out_bits, base.layer_mem_bytes, cap, base.bw_kbps)
    assert_same(inst, gpu_solve(inst), oracle.dp_fact(inst, oracle.max_threads()))
    # one over either limit is refused
    with pytest.raises(pp.PPError) as ei:
        pp.Problem(pp.PP_MAX_L + 1, np.ones(pp.PP_MAX_L + 1, np.uint64), np.ones(pp.PP_MAX_L + 1, np.uint64),
                   2, np.ones(2, np.uint64), np.ones(4, np.uint32))
    assert ei.value.status == pp.PP_ERR_LIMIT


def test_32bit_rank_path():
    # enough distinct gamma values that 16-bit ranks do not fit: L * U + 1 > 65534
    L, k = 700, 11
    base = W.random_small(40000, L, k)
    cap = np.full(k, int(base.layer_mem_bytes.sum()) // 4, dtype=np.uint64)
    bw = base.bw_kbps.copy()
    bw[np.triu_indices(k, 1)] += np.arange(k * (k - 1) // 2, dtype=np.uint32) + 1  # directed links
    inst = make_instance(base.layer_out_bits, base.layer_mem_bytes, cap, bw)
    assert len({int(x) for x in inst.bw_kbps.ravel() if x}) * L + 1 > 65534
    want = oracle.dp_fact(inst, oracle.max_threads())
    with pp.Problem.from_instance(inst) as p:
        got = p.solve_exact()
        assert p.last_solve_profile().state_bytes == 4
    assert_same(inst, got, want)


def test_evaluator_against_oracle():
    for inst, B in ((W.config_tiny(), 3000), (W.config_resnet50_shaped(), 3000),
                    (W.random_small(50000, 14, 7, dead_links=0.2), 2000), (W.config_large(), 5000)):
        nseg, ends, nodes = W.random_plans(inst, B, seed=B + inst.k, invalid_fraction=0.15)
        want_beta, want_status = oracle.eval_plans(inst, nseg, ends, nodes)
        with pp.Problem.from_instance(inst) as p:
            beta, status = p.eval_plans(nseg, ends, nodes)
            assert np.array_equal(status, want_status)
            assert np.array_equal(beta, want_beta)  # inf == inf
            assert (status == 0).sum() > 10 and (status != 0).sum() > 10
            # the optimum scores as itself
            sol = p.solve_exact()
            if sol.status == pp.PP_OK:
                e = np.full((1, inst.k), -1, np.int32)
                n = np.full((1, inst.k), -1, np.int32)
                e[0, :sol.m - 1] = sol.cuts[:sol.m - 1]
                n[0, :sol.m] = sol.placement[:sol.m]
                b1, s1 = p.eval_plans(np.array([sol.m], np.uint8), e, n)
                assert s1[0] == 0 and b1[0] == sol.beta_ms
            assert p.eval_plans(np.zeros(0, np.uint8), np.zeros((0, inst.k), np.int32),
                                np.zeros((0, inst.k), np.int32))[0].shape == (0,)


def test_packed_evaluator_against_oracle():
    # compressed rows (16-bit cuts, 8-bit nodes, offsets) score like the int32 rows
    for inst, B in ((W.config_tiny(), 3000), (W.config_resnet50_shaped(), 3000), (W.config_large(), 6000),
                    (W.random_small(50001, 300, 9, dead_links=0.2), 2000)):
        nseg, ends, nodes = W.random_plans(inst, B, seed=B + 3 * inst.k, invalid_fraction=0.15)
        want_beta, want_status = oracle.eval_plans(inst, nseg, ends, nodes)
        off, e16, n8 = W.pack_plans(nseg, ends, nodes)
        with pp.Problem.from_instance(inst) as p:
            beta, status = p.eval_plans_packed(nseg, off, e16, n8)
            assert np.array_equal(status, want_status)
            assert np.array_equal(beta, want_beta)
            assert (status != 0).sum() > 10 and len(set(status.tolist())) >= 4
            assert inst.L > 200 or (status == 0).sum() > 10  # the long chain's random plans rarely fit
            # a row shorter than its nseg, and a row that reaches beyond the arrays, are refused
            bad_off = off.copy()
            victim = int(np.flatnonzero(nseg > 2)[0])
            bad_off[victim + 1:] -= 1
            b2, s2 = p.eval_plans_packed(nseg, bad_off, e16, n8)
            assert s2[victim] == pp.PP_PLAN_BAD_NSEG and np.isinf(b2[victim])
            b3, s3 = p.eval_plans_packed(nseg[:5], off[:6], e16[:int(off[5]) - 1], n8[:int(off[5]) - 1])
            last = max(b for b in range(5) if off[b + 1] > off[b])  # the last plan with entries loses one
            assert s3[last] == pp.PP_PLAN_BAD_NSEG
            assert p.eval_plans_packed(np.zeros(0, np.uint8), np.zeros(1, np.uint32), np.zeros(0, np.uint16),
                                       np.zeros(0, np.uint8))[0].shape == (0,)


def test_evaluator_beyond_one_pass_of_the_grid():
    # more plans than one pass of the evaluator's grid covers (148 * 16 blocks of 256): the later
    # passes of the grid-stride loop are compared with the oracle too (the plans repeat with period
    # 5003, the oracle scores one period)
    inst = W.config_resnet50_shaped()
    period, B = 5003, 700_001
    nseg, ends, nodes = W.random_plans(inst, period, seed=99, invalid_fraction=0.1)
    want_beta, want_status = oracle.eval_plans(inst, nseg, ends, nodes)
    idx = np.arange(B) % period
    with pp.Problem.from_instance(inst) as p:
        beta, status = p.eval_plans(nseg[idx], ends[idx], nodes[idx])
        assert np.array_equal(status, want_status[idx]) and np.array_equal(beta, want_beta[idx])
        off, e16, n8 = W.pack_plans(nseg[idx], ends[idx], nodes[idx])
        beta, status = p.eval_plans_packed(nseg[idx], off, e16, n8)
        assert np.array_equal(status, want_status[idx]) and np.array_equal(beta, want_beta[idx])


def test_minmax_rate_hook_and_phase_profile():
    # the issue-rate hook returns plausible rates (one to four warp instructions per clock per SM),
    # and the phase times are reported only when asked for
    for op in range(3):
        rate = pp.debug_minmax_rate(op, 512)
        assert 0.5 < rate < 4.5, (op, rate)
    inst = W.config_resnet50_shaped()
    with pp.Problem.from_instance(inst) as p:
        p.solve_exact()
        prof = p.last_solve_profile()
        assert prof.ms_total > 0 and prof.ms_sweep == 0 and prof.ms_rank == 0
        p.set_profiling(True)
        p.solve_exact()
        prof = p.last_solve_profile()
        assert prof.ms_sweep > 0 and prof.ms_rank > 0 and prof.ms_finalize > 0
        assert prof.sweep_launches == min(inst.k, inst.L) - 1


def _stack(insts):
    return (np.stack([i.layer_out_bits for i in insts]), np.stack([i.layer_mem_bytes for i in insts]),
            np.stack([i.node_mem_bytes for i in insts]), np.stack([i.bw_kbps for i in insts]))


def test_batched_solve_full_config():
    insts = W.config_batched()
    assert len(insts) == 4096
    got = pp.solve_exact_batch(24, 8, *_stack(insts))
    n_inf = 0
    for b, inst in enumerate(insts):
        want = oracle.dp_fact(inst)
        assert got.status[b] == want.status, b
        assert got.beta_ms[b] == want.beta_ms or (np.isinf(got.beta_ms[b]) and np.isinf(want.beta_ms))
        assert got.plan(b) == want.plan(), b
        assert (got.cuts[b, max(want.m - 1, 0):] == -1).all() and (got.placement[b, want.m:] == -1).all()
        n_inf += want.status == oracle.INFEASIBLE
    assert 0 < n_inf < 4096


def test_batched_solve_odd_shapes():
    # batches too small for the instance-per-lane kernels: one block per instance, chains shorter and
    # longer than a warp, a power of two long, more nodes than layers
    for L, k, n in ((1, 1, 3), (2, 3, 6), (5, 2, 9), (13, 5, 40), (3, 6, 12), (16, 3, 8), (30, 7, 10),
                    (32, 4, 8), (33, 4, 8), (70, 3, 6)):
        insts = [W.random_small(60000 + 100 * L + i, L, k, tight=(i % 3 == 1), ties=(i % 3 == 2),
                                dead_links=0.25 if i % 4 == 3 else 0.0) for i in range(n)]
        got = pp.solve_exact_batch(L, k, *_stack(insts))
        for b, inst in enumerate(insts):
            want = oracle.dp_naive(inst)
            assert got.status[b] == want.status
            assert got.plan(b) == want.plan()
            assert got.beta_ms[b] == want.beta_ms or np.isinf(want.beta_ms)
    # a table that cannot fit one block's shared memory is refused, not mis-solved
    with pytest.raises(pp.PPError) as ei:
        pp.solve_exact_batch(200, 12, np.ones((1, 200), np.uint64), np.ones((1, 200), np.uint64),
                             np.ones((1, 12), np.uint64), np.ones((1, 12, 12), np.uint32))
    assert ei.value.status == pp.PP_ERR_LIMIT


def test_batched_solve_instance_per_lane_shapes():
    # from 64 instances on, chains of up to 32 layers on up to 8 nodes are solved 32 instances to a
    # warp: every row width of that path (4, 8, 12, 16 words), batches that end inside a group of 32,
    # more nodes than layers, and the degenerate inputs
    for L, k, n in ((1, 4, 64), (2, 3, 64), (5, 2, 97), (7, 8, 65), (13, 5, 130), (16, 3, 96), (17, 6, 71), (24, 8, 100),
                    (25, 4, 64), (30, 7, 70), (32, 4, 89)):
        insts = [W.random_small(61000 + 100 * L + i, L, k, tight=(i % 3 == 1), ties=(i % 3 == 2),
                                dead_links=0.25 if i % 4 == 3 else 0.0) for i in range(n)]
        got = pp.solve_exact_batch(L, k, *_stack(insts))
        for b, inst in enumerate(insts):
            want = oracle.dp_naive(inst)
            assert got.status[b] == want.status, (L, k, b)
            assert got.plan(b) == want.plan(), (L, k, b)
            assert got.beta_ms[b] == want.beta_ms or np.isinf(want.beta_ms)
            assert (got.cuts[b, max(want.m - 1, 0):] == -1).all() and (got.placement[b, want.m:] == -1).all()
    # an instance beyond the limits is flagged on its own, its neighbours are solved
    insts = [W.random_small(62000 + i, 12, 4) for i in range(80)]
    bits, mem, cap, bw = _stack(insts)
    bits[17, 3] = np.uint64(1) << np.uint64(41)
    mem[20, :2] = np.uint64(1) << np.uint64(63)  # the 64-bit sum of the memory wraps
    bw[23, 1, 2] = np.uint32(1) << np.uint32(24)
    got = pp.solve_exact_batch(12, 4, bits, mem, cap, bw)
    for b in (17, 20, 23):
        assert got.status[b] == pp.PP_ERR_LIMIT and got.m[b] == 0 and np.isinf(got.beta_ms[b]), b
    for b in (16, 18, 79):
        assert got.plan(b) == oracle.dp_naive(insts[b]).plan()


def test_batched_solve_asymmetric_links_and_pieces():
    # a network whose two directions differ has up to k (k - 1) distinct bandwidths: such instances are
    # ranked by the second preparing pass, symmetric ones by the first, in one batch
    rng = np.random.Generator(np.random.PCG64(20240607))
    for L, k, n in ((11, 5, 96), (24, 8, 70), (32, 7, 65)):
        insts = [W.random_small(63000 + 100 * L + i, L, k, tight=(i % 5 == 1), dead_links=0.2 if i % 4 == 3 else 0.0)
                 for i in range(n)]
        bits, mem, cap, bw = _stack(insts)
        for i in range(0, n, 2):  # every other instance: independent draws per direction, some links dead
            m = rng.integers(1000, 12000, size=(k, k)).astype(np.uint32)
            m[rng.random((k, k)) < 0.1] = 0
            np.fill_diagonal(m, 0)
            bw[i] = m
            insts[i] = W.Instance(L, k, bits[i], mem[i], cap[i], bw[i], "asymmetric")
        got = pp.solve_exact_batch(L, k, bits, mem, cap, bw)
        for b, inst in enumerate(insts):
            want = oracle.dp_naive(inst)
            assert got.status[b] == want.status, (L, k, b)
            assert got.plan(b) == want.plan(), (L, k, b)
            assert got.beta_ms[b] == want.beta_ms or np.isinf(want.beta_ms)
    # more instances than share the scratch tables at a time: worked off in pieces on the same stream
    L, k, n = 5, 3, 4096 + 45
    insts = [W.random_small(64000 + i, L, k, tight=(i % 3 == 1), ties=(i % 7 == 2)) for i in range(n)]
    got = pp.solve_exact_batch(L, k, *_stack(insts))
    for b in list(range(0, n, 17)) + list(range(4090, n)):
        want = oracle.dp_naive(insts[b])
        assert got.status[b] == want.status and got.plan(b) == want.plan(), b
        assert got.beta_ms[b] == want.beta_ms or np.isinf(want.beta_ms)


def test_workspace_and_stream_from_torch():
    import torch
    inst = W.config_resnet50_shaped()
    want = oracle.dp_fact(inst, 4)
    stream = torch.cuda.Stream()
    with pp.Problem.from_instance(inst) as p:
        ws = torch.empty(p.workspace_bytes(), dtype=torch.uint8, device="cuda")
        p.set_workspace(ws)
        p.set_stream(stream.cuda_stream)
        sol = torch.zeros(24, dtype=torch.float64, device="cuda")  # 192 bytes >= sizeof(pp_solution)
        p.solve_exact_dev(sol.data_ptr())
        stream.synchronize()
        raw = sol.cpu().numpy().tobytes()
        rec = pp.pp_solution.from_buffer_copy(raw[:176])
        assert rec.beta_ms == want.beta_ms and rec.status == want.status and rec.m == want.m
        assert tuple(rec.cuts[:want.m - 1]) == want.plan()[1]
        assert tuple(rec.placement[:want.m]) == want.plan()[2]
        small = torch.empty(16, dtype=torch.uint8, device="cuda")
        with pytest.raises(pp.PPError):
            p.set_workspace(small)
