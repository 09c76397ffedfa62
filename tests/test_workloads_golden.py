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
    return cases


def test_generators_are_reproducible():
    gold = read_golden()
    for name, inst in named_instances().items():
        assert inst.checksum() == gold[name][0], name
    a, b = W.config_large(), W.config_large()
    assert np.array_equal(a.bw_kbps, b.bw_kbps) and np.array_equal(a.bw_kbps, a.bw_kbps.T)
    assert (np.diag(a.bw_kbps) == 0).all()


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
