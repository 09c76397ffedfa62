"""The seeded generators are reproducible, and the oracle reproduces its stored optima
(tests/golden/config_optima.txt, written by tests/golden/make_golden.py from the oracle only)."""
from __future__ import annotations

import os

import numpy as np
import pytest

import oracle
from paper_2210_12219_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "config_optima.txt")


def read_golden():
    out = {}
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        head, cuts, nodes = [p.strip() for p in line.split("|")]
        name, checksum, beta, m = head.split()
        out[name] = (int(checksum), float("inf") if beta == "inf" else float.fromhex(beta), int(m),
                     tuple(int(x) for x in cuts.split()), tuple(int(x) for x in nodes.split()))
    return out


def named_instances():
    cases = {i.name: i for i in (W.config_tiny(), W.config_resnet50_shaped(), W.config_deeper_cnn(),
                                 W.config_large())}
    cases.update({i.name: i for i in W.config_batched(8)})
    cases.update({i.name: i for i in (W.config_geometric(14, 64, 0), W.config_geometric(10, 64, 1, link="pairwise"))})
    return cases


def test_generators_are_reproducible():
    gold = read_golden()
    for name, inst in named_instances().items():
        assert inst.checksum() == gold[name][0], name
    a, b = W.config_large(), W.config_large()
    assert np.array_equal(a.bw_kbps, b.bw_kbps) and np.array_equal(a.bw_kbps, a.bw_kbps.T)
    assert (np.diag(a.bw_kbps) == 0).all()


def test_geometric_workload_follows_section_4():
    # Eq. 12 with a = 283230 gives 5.5 Mbps at 80 m from the router (the paper's calibration)
    assert abs(W.shannon_mbps(80.0, 0.0) - 5.5) < 1e-5 and abs(W.shannon_mbps(0.0, -80.0) - 5.499995) < 1e-5
    assert abs(W.shannon_mbps(48.0, 64.0) - W.shannon_mbps(80.0, 0.0)) < 1e-12  # only the distance counts
    for seed in range(20):
        bw, pos = W.geometric_bandwidths(12, seed)
        assert ((np.abs(pos) > 1.0) & (np.abs(pos) < 150.0)).all()  # no device within 1 m of an axis, none beyond 150 m
        assert np.array_equal(bw, bw.T) and (np.diag(bw) == 0).all() and (bw[~np.eye(12, dtype=bool)] > 0).all()
        rate = np.array([W.shannon_mbps(x, y) for x, y in pos])
        far = int(np.argmin(rate))
        assert (bw[far][np.arange(12) != far] == int(round(1000 * rate[far]))).all()  # the slower end decides
        pw, _ = W.geometric_bandwidths(12, seed, link="pairwise")
        d2 = ((pos[3] - pos[7]) ** 2).sum()
        assert pw[3, 7] == int(round(1000 * np.log2(1 + 283230.0 / max(d2, 1.0))))
    g = W.config_geometric(14, 128, 3)
    assert g.k == 14 and len(set(g.node_mem_bytes.tolist())) == 1 and int(g.node_mem_bytes[0]) == 128_000_000
    assert np.array_equal(g.layer_out_bits, W.config_resnet50_shaped().layer_out_bits)
    signs = np.sign(np.concatenate([W.geometric_bandwidths(50, s)[1].ravel() for s in range(4)]))
    assert 0.35 < (signs < 0).mean() < 0.65  # both half-ranges are used


def test_config_shapes_follow_the_recipe():
    t, r, c, l = W.config_tiny(), W.config_resnet50_shaped(), W.config_deeper_cnn(), W.config_large()
    assert (t.L, t.k) == (12, 6) and (r.L, r.k) == (50, 10) and (c.L, c.k) == (100, 14) and (l.L, l.k) == (200, 18)
    assert int(r.layer_mem_bytes.sum()) == 102_400_000 and int(c.layer_mem_bytes.sum()) == 240_000_000
    assert int(l.layer_mem_bytes.sum()) == 1_200_000_000 and len(set(l.layer_mem_bytes.tolist())) == 1
    assert int(r.node_mem_bytes.max()) * 2 < int(r.layer_mem_bytes.sum())  # at least three segments
    assert abs(float(r.layer_out_bits.mean()) / 10.2e6 - 1) < 0.5
    assert 0.9 * 8_388_608 <= int(l.layer_out_bits.min()) and int(l.layer_out_bits.max()) <= 1.1 * 8_388_608 + 1
    assert ((c.bw_kbps == 500).sum() > 0)
    u = W.uniform_memory_small(1, 40, 5, 8, 20)
    assert len(set(u.layer_mem_bytes.tolist())) == 1


def test_oracle_reproduces_stored_optima():
    gold = read_golden()
    for name, inst in named_instances().items():
        if name == "large":
            continue  # ten seconds of CPU: covered by the GPU-side test of the full-size config
        _, beta, m, cuts, nodes = gold[name]
        sol = oracle.dp_fact(inst, 2)
        assert sol.beta_ms == beta and sol.plan() == (m, cuts, nodes), name


def test_random_plans_generator():
    inst = W.config_tiny()
    nseg, ends, nodes = W.random_plans(inst, 500, seed=3, invalid_fraction=0.2)
    assert nseg.dtype == np.uint8 and ends.shape == (500, inst.k) and nodes.shape == (500, inst.k)
    _, status = oracle.eval_plans(inst, nseg, ends, nodes)
    assert (status == 0).any() and (status != 0).any()
