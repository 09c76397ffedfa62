"""GPU parity of the partition stage (pp_partition_minsum_batch) against oracle/partition.py:
integers only, so every comparison is exact equality."""
from __future__ import annotations

import numpy as np
import pytest

import paper_2210_12219_b200 as pp
from oracle import partition as OP
from paper_2210_12219_b200 import build
from paper_2210_12219_b200 import workloads as W
from tests.test_oracle_partition import golden_cases

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    pp.lib()


def _check(weights, mem, kappa, cap_seg, every=1):
    got = pp.partition_minsum_batch(weights, mem, kappa, cap_seg)
    B = weights.shape[0]
    for b in sorted(set(range(0, B, every)) | set(range(max(B - 40, 0), B))):
        want = OP.minsum_partition(weights[b].tolist(), mem[b].tolist(), int(kappa[b]))
        if want.status == OP.INFEASIBLE:
            assert got.status[b] == pp.PP_INFEASIBLE and got.m[b] == 0 and got.cost[b] == 0
            assert (got.cuts[b] == -1).all()
            continue
        assert got.m[b] == want.m and int(got.cost[b]) == want.cost, b
        if want.m - 1 > cap_seg:
            assert got.status[b] == pp.PP_ERR_LIMIT
            continue
        assert got.status[b] == pp.PP_OK
        assert tuple(got.cuts[b, :want.m - 1].tolist()) == want.cuts, b
        assert tuple(int(x) for x in got.sizes[b, :want.m - 1]) == want.sizes
        assert (got.cuts[b, want.m - 1:] == -1).all() and (got.sizes[b, want.m - 1:] == 0).all()
    return got


def test_hand_worked_partitions_on_gpu():
    for w, mem, kappa, cost, m, cuts in golden_cases():
        got = pp.partition_minsum_batch(np.array([w], np.uint64), np.array([mem], np.uint64),
                                        np.array([kappa], np.uint64), 8)
        if m == 0:
            assert got.status[0] == pp.PP_INFEASIBLE
        else:
            assert (int(got.cost[0]), int(got.m[0]), tuple(got.cuts[0, :m - 1].tolist())) == (cost, m, cuts)


# 60 chains: one warp per chain; 8200 chains of up to 64 points: one lane per chain, the last group of
# 32 not full, every 41st chain and the last 40 compared
@pytest.mark.parametrize("B", [60, 8200])
@pytest.mark.parametrize("L", [1, 2, 7, 31, 32, 33, 64, 100, 257])
def test_random_chains(L, B):
    if B > 60 and L > 64:
        pytest.skip("chains this long take the warp-per-chain kernel at any batch size")
    rng = np.random.default_rng(100 + L + B)
    every = 1 if B == 60 else 41
    mem = rng.integers(1, 40, size=(B, L)).astype(np.uint64)
    kappa = rng.integers(30, 160, size=B).astype(np.uint64)
    kappa[::7] = 20  # some chains hold a point that fits nowhere
    weights = rng.integers(0, 10**7, size=(B, L)).astype(np.uint64)
    weights[1::3] = rng.integers(0, 4, size=weights[1::3].shape)  # tie-heavy: class numbers
    got = _check(weights, mem, kappa, L, every)
    assert (got.status == pp.PP_OK).sum() > 10
    # rows shorter than the plan: refused per chain, cost and m still reported
    if L >= 31:
        _check(weights, mem, kappa, 2, every)


def test_model_shaped_chains_and_limits():
    # the named configurations' chains (weights = output bits), one capacity for all nodes as in the
    # paper: the smallest node of the instance; the longest chain the library takes; limit checks
    for inst in (W.config_resnet50_shaped(), W.config_deeper_cnn(), W.config_large()):
        w = inst.layer_out_bits[None, :]
        mem = inst.layer_mem_bytes[None, :]
        for kappa in (int(inst.node_mem_bytes.min()), int(inst.node_mem_bytes.max())):
            _check(w, mem, np.array([kappa], np.uint64), inst.L)
    rng = np.random.default_rng(7)
    L = pp.PP_MAX_L
    mem = rng.integers(1, 100, size=(3, L)).astype(np.uint64)
    weights = rng.integers(1, 2**39, size=(3, L)).astype(np.uint64)
    _check(weights, mem, np.array([500, 5000, 10**6], np.uint64), L)
    # a weight at the limit, a memory sum that wraps: PP_ERR_LIMIT for that chain only
    weights2 = weights[:, :40].copy()
    mem2 = mem[:, :40].copy()
    weights2[0, 5] = 1 << 40
    mem2[1, 3] = mem2[1, 4] = np.uint64(2**63)
    got = pp.partition_minsum_batch(weights2, mem2, np.array([500, 500, 500], np.uint64), 40)
    assert got.status[0] == pp.PP_ERR_LIMIT and got.status[1] == pp.PP_ERR_LIMIT and got.status[2] == pp.PP_OK
    want = OP.minsum_partition(weights2[2].tolist(), mem2[2].tolist(), 500)
    assert int(got.cost[2]) == want.cost and tuple(got.cuts[2, :want.m - 1].tolist()) == want.cuts
    # empty batch and bad arguments
    assert pp.partition_minsum_batch(np.zeros((0, 5), np.uint64), np.zeros((0, 5), np.uint64),
                                     np.zeros(0, np.uint64), 5).cost.shape == (0,)
    with pytest.raises(pp.PPError):
        pp.partition_minsum_batch(np.zeros((1, pp.PP_MAX_L + 1), np.uint64), np.ones((1, pp.PP_MAX_L + 1), np.uint64),
                                  np.ones(1, np.uint64), 4)
