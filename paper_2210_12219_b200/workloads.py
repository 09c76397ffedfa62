"""Seeded synthetic partition-and-placement instances.

This module only draws numbers.  It holds none of the method's arithmetic (no
latency, no feasibility test, no search) so that the CPU oracle and the CUDA
path can both consume it without sharing any logic.

An instance is a layer chain of length L (per-layer output size in bits, per-layer
memory in bytes) and k edge nodes (memory capacity in bytes, pairwise bandwidth
in kbps).  The shapes and scales follow the paper's setting: activations that
average about 10.2 Mbit, links of a few Mbps, nodes of tens to hundreds of MB
(Section 1 and Section 4 of the paper); the chains themselves are synthetic
stand-ins for the Keras models the paper evaluates, which are not available
offline.

Random numbers come from SplitMix64 (Steele, Lea, Flood 2014), written out here,
with one independent stream per (config, instance, field); normals use the
Box-Muller transform in float64.  MB means 10**6 bytes.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

_MASK = (1 << 64) - 1
_GAMMA = 0x9E3779B97F4A7C15


def _mix(z: int) -> int:
    z &= _MASK
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK
    return z ^ (z >> 31)


class SplitMix64:
    """Counter-based 64-bit generator: output i is mix(seed + (i+1) * GAMMA)."""

    def __init__(self, seed: int):
        self.state = seed & _MASK

    def next_u64(self) -> int:
        self.state = (self.state + _GAMMA) & _MASK
        return _mix(self.state)

    def u64(self, n: int) -> np.ndarray:
        return np.array([self.next_u64() for _ in range(n)], dtype=np.uint64)

    def uniform_int(self, lo: int, hi: int, n: int) -> np.ndarray:
        """n integers in [lo, hi] (modulo reduction; bias < 2**-30 at these ranges)."""
        span = hi - lo + 1
        return np.array([lo + self.next_u64() % span for _ in range(n)], dtype=np.uint64)

    def uniform01(self, n: int) -> np.ndarray:
        """n float64 in [0, 1)."""
        return np.array([(self.next_u64() >> 11) * 2.0 ** -53 for _ in range(n)], dtype=np.float64)

    def normal(self, n: int) -> np.ndarray:
        """n standard normals, Box-Muller, one pair of uniforms per sample."""
        out = np.empty(n, dtype=np.float64)
        for i in range(n):
            u1 = ((self.next_u64() >> 11) + 1) * 2.0 ** -53  # (0, 1]
            u2 = (self.next_u64() >> 11) * 2.0 ** -53
            out[i] = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
        return out


def stream(config_id: int, instance_id: int, field_id: int) -> SplitMix64:
    """Independent generator for one field of one instance of one config."""
    s = _mix(config_id + 1)
    s = _mix(s ^ ((instance_id + 1) * _GAMMA & _MASK))
    s = _mix(s ^ ((field_id + 1) * 0xD1B54A32D192ED03 & _MASK))
    return SplitMix64(s)


F_BITS, F_MEM, F_CAP, F_BW, F_AUX = 0, 1, 2, 3, 4


@dataclass
class Instance:
    """One problem instance; all arrays are C-contiguous numpy arrays."""

    L: int
    k: int
    layer_out_bits: np.ndarray  # uint64 [L]
    layer_mem_bytes: np.ndarray  # uint64 [L]
    node_mem_bytes: np.ndarray  # uint64 [k]
    bw_kbps: np.ndarray  # uint32 [k, k], [v, w] = link v -> w, diagonal 0
    name: str = ""

    def checksum(self) -> int:
        h = 0xCBF29CE484222325
        for arr in (self.layer_out_bits, self.layer_mem_bytes, self.node_mem_bytes,
                    self.bw_kbps.astype(np.uint64).ravel()):
            for x in arr.tolist():
                h = _mix(h ^ int(x))
        return h


def _symmetric(k: int, draw) -> np.ndarray:
    """k x k symmetric matrix with zero diagonal from draw(n) -> n values (upper triangle)."""
    n = k * (k - 1) // 2
    vals = draw(n)
    bw = np.zeros((k, k), dtype=np.uint32)
    idx = 0
    for v in range(k):
        for w in range(v + 1, k):
            bw[v, w] = bw[w, v] = int(vals[idx])
            idx += 1
    return bw


def _split_exact(weights: np.ndarray, total: int) -> np.ndarray:
    """Integers proportional to weights that sum to total exactly (remainder to the last)."""
    w = weights / weights.sum()
    parts = np.floor(w * total).astype(np.uint64)
    parts[-1] = np.uint64(total - int(parts[:-1].sum()))
    return parts


def uniform_instance(config_id: int, instance_id: int, L: int, k: int, name: str = "",
                     cap_stream_offset: int = 0) -> Instance:
    """The 'Tiny' distribution: everything uniform integer (configs 1 and 4)."""
    bits = stream(config_id, instance_id, F_BITS).uniform_int(100_000, 20_000_000, L)
    mem = stream(config_id, instance_id, F_MEM).uniform_int(1_000_000, 40_000_000, L)
    cap = stream(config_id, instance_id, F_CAP + 16 * cap_stream_offset).uniform_int(
        40_000_000, 160_000_000, k)
    bw = _symmetric(k, lambda n: stream(config_id, instance_id, F_BW).uniform_int(1000, 12000, n))
    return Instance(L, k, bits, mem, cap, bw, name)


def config_tiny() -> Instance:
    """Config 1: L=12, k=6, seed 0; small enough to enumerate every plan."""
    return uniform_instance(1, 0, 12, 6, "tiny")


def config_resnet50_shaped() -> Instance:
    """Config 2: L=50, k=10; log-normal activations averaging 10.2 Mbit, 25.6 M fp32
    parameters spread with a 64x geometric rise, caps that force at least 3 segments,
    log-normal bandwidths averaging 6 Mbps."""
    L, k = 50, 10
    sigma = 0.75
    mu = np.log(10.2e6) - sigma * sigma / 2
    z = stream(2, 0, F_BITS).normal(L)
    bits = np.clip(np.rint(np.exp(mu + sigma * z)), 1e5, 1.2e8).astype(np.uint64)
    u = stream(2, 0, F_MEM).uniform01(L)
    weights = 64.0 ** (np.arange(L) / L) * (0.8 + 0.4 * u)
    mem = _split_exact(weights, 102_400_000)
    cap = stream(2, 0, F_CAP).uniform_int(24_000_000, 48_000_000, k)
    sb = 0.5
    mb = np.log(6000.0) - sb * sb / 2

    def draw(n):
        zz = stream(2, 0, F_BW).normal(n)
        return np.clip(np.rint(np.exp(mb + sb * zz)), 500, 50000)

    return Instance(L, k, bits, mem, cap, _symmetric(k, draw), "resnet50_shaped")


def config_deeper_cnn() -> Instance:
    """Config 3: L=100, k=14; five stages whose activations halve stage by stage, memory
    rising with depth (240 MB total), a fifth of the links degraded to 0.5 Mbps."""
    L, k = 100, 14
    z = stream(3, 0, F_BITS).normal(L)
    stage = np.arange(L) // 20
    raw = 2.0 ** (-stage) * np.exp(0.35 * z)
    bits = np.maximum(np.rint(raw * (8.0e6 / raw.mean())), 1).astype(np.uint64)
    u = stream(3, 0, F_MEM).uniform01(L)
    mem = _split_exact((np.arange(L) + 1.0) * (0.9 + 0.2 * u), 240_000_000)
    cap = stream(3, 0, F_CAP).uniform_int(64_000_000, 256_000_000, k)
    slow = stream(3, 0, F_AUX).uniform01(k * (k - 1) // 2) < 0.2
    fast = stream(3, 0, F_BW).uniform_int(2000, 20000, k * (k - 1) // 2)
    vals = np.where(slow, 500, fast)
    return Instance(L, k, bits, mem, cap, _symmetric(k, lambda n: vals), "deeper_cnn")


def config_batched(count: int = 4096, L: int = 24, k: int = 8) -> list[Instance]:
    """Config 4: independent instances from the 'Tiny' distributions; infeasible draws stay in."""
    return [uniform_instance(4, 1000 + i, L, k, f"batched[{i}]") for i in range(count)]


def config_large() -> Instance:
    """Config 5: L=200, k=18; near-uniform 8.4 Mbit activations (+-10 %), 1.2 GB of
    parameters split evenly, heterogeneous node memory, bandwidths 1-50 Mbps."""
    L, k = 200, 18
    u = stream(5, 0, F_BITS).uniform01(L)
    bits = np.rint(8_388_608 * (0.9 + 0.2 * u)).astype(np.uint64)
    mem = np.full(L, 6_000_000, dtype=np.uint64)
    cap = stream(5, 0, F_CAP).uniform_int(128_000_000, 512_000_000, k)
    bw = _symmetric(k, lambda n: stream(5, 0, F_BW).uniform_int(1000, 50000, n))
    return Instance(L, k, bits, mem, cap, bw, "large")


def large_unequal_layers(k: int = 18) -> Instance:
    """The Large chain with layers of unequal memory (what a real model chain looks like): the same
    bits, capacities and bandwidths (the first k nodes), each layer's 6 MB scaled by U[0.5, 1.5).
    The sliding memory windows then differ from position to position."""
    base = config_large()
    u = stream(5, 1, F_MEM).uniform01(base.L)
    mem = np.rint(base.layer_mem_bytes.astype(np.float64) * (0.5 + u)).astype(np.uint64)
    return Instance(base.L, k, base.layer_out_bits, mem, base.node_mem_bytes[:k].copy(),
                    np.ascontiguousarray(base.bw_kbps[:k, :k]), "large_unequal_layers")


SHANNON_A = 283230.0  # Section 4: chosen so that a device 80 m from the router gets 5.5 Mbps


def shannon_mbps(x: float, y: float) -> float:
    """Eq. 12: rate in Mbps of a device at (x, y) metres from the router at the origin."""
    return float(np.log2(1.0 + SHANNON_A / (x * x + y * y)))


def geometric_bandwidths(k: int, seed: int, link: str = "router") -> tuple[np.ndarray, np.ndarray]:
    """The random communication graph of the paper's evaluation (Section 4): k devices at positions
    drawn uniformly from ((-150, -1) u (1, 150))^2 around a WiFi router at the origin, link rates from
    Shannon's capacity with an SNR that falls with the square of the distance (Eq. 12).
    link = "router": the rate of a device is that of its own link to the router, and a transfer
    between two devices passes through the router, so the pair gets the smaller of the two rates.
    link = "pairwise": Eq. 12 applied to the distance between the two devices (never below 1 m).
    Returns (bw_kbps uint32 [k, k] symmetric with zero diagonal, positions float64 [k, 2])."""
    u = stream(6, seed, F_AUX).uniform01(4 * k)
    mag = 1.0 + 149.0 * u[: 2 * k]
    sign = np.where(u[2 * k:] < 0.5, -1.0, 1.0)
    pos = (mag * sign).reshape(k, 2)
    bw = np.zeros((k, k), dtype=np.uint32)
    rate = [shannon_mbps(px, py) for px, py in pos]
    for v in range(k):
        for w in range(v + 1, k):
            if link == "router":
                r = min(rate[v], rate[w])
            else:
                dx, dy = pos[v, 0] - pos[w, 0], pos[v, 1] - pos[w, 1]
                r = float(np.log2(1.0 + SHANNON_A / max(dx * dx + dy * dy, 1.0)))
            bw[v, w] = bw[w, v] = max(1, int(round(1000.0 * r)))
    return bw, pos


def config_geometric(k: int = 14, cap_mb: int = 64, seed: int = 0, link: str = "router") -> Instance:
    """The paper's evaluation setting on a synthetic chain: the ResNet50-shaped chain (config 2) on k
    devices of equal memory (64, 128, 256 or 512 MB in the paper) joined by the random geometric
    graph of Section 4."""
    base = config_resnet50_shaped()
    bw, _ = geometric_bandwidths(k, seed, link)
    cap = np.full(k, cap_mb * 1_000_000, dtype=np.uint64)
    return Instance(base.L, k, base.layer_out_bits, base.layer_mem_bytes, cap, bw,
                    "geometric_k%d_%dMB%s" % (k, cap_mb, "" if link == "router" else "_pairwise"))


def random_small(seed: int, L: int, k: int, *, tight: bool = False, dead_links: float = 0.0,
                 ties: bool = False) -> Instance:
    """Small random instance for parity sweeps.  tight=True shrinks capacities so that some
    draws have no plan; dead_links sets that fraction of links to 0 kbps; ties=True draws
    from tiny value sets so that many plans share the same bottleneck."""
    if ties:
        bits = stream(9, seed, F_BITS).uniform_int(1, 4, L) * np.uint64(6000)
        bwv = lambda n: stream(9, seed, F_BW).uniform_int(1, 3, n) * np.uint64(1000)
    else:
        bits = stream(9, seed, F_BITS).uniform_int(100_000, 20_000_000, L)
        bwv = lambda n: stream(9, seed, F_BW).uniform_int(1000, 12000, n)
    mem = stream(9, seed, F_MEM).uniform_int(1_000_000, 40_000_000, L)
    lo, hi = (15_000_000, 60_000_000) if tight else (40_000_000, 160_000_000)
    cap = stream(9, seed, F_CAP).uniform_int(lo, hi, k)
    bw = _symmetric(k, bwv)
    if dead_links > 0:
        dead = stream(9, seed, F_AUX).uniform01(k * k).reshape(k, k) < dead_links
        dead = np.triu(dead, 1)
        dead = dead | dead.T
        bw[dead] = 0
    return Instance(L, k, bits, mem, cap, bw, f"small[{seed}]")


def uniform_memory_small(seed: int, L: int, k: int, wmin: int = 8, wmax: int | None = None, *,
                         ties: bool = False, dead_links: float = 0.0) -> Instance:
    """Small instance whose layers all need the same memory (a stack of identical blocks), so
    that node w holds any run of at most W_w consecutive layers; W_w is drawn from [wmin, wmax]."""
    base = random_small(seed, L, k, ties=ties, dead_links=dead_links)
    wmax = wmax if wmax is not None else L + 4
    unit = 1_000_000
    widths = stream(10, seed, F_CAP).uniform_int(wmin, max(wmin, wmax), k)
    slack = stream(10, seed, F_AUX).uniform_int(0, unit - 1, k)
    cap = widths * np.uint64(unit) + slack
    mem = np.full(L, unit, dtype=np.uint64)
    return Instance(L, k, base.layer_out_bits, mem, cap, base.bw_kbps, f"uniform[{seed}]")


def random_plans(inst: Instance, count: int, seed: int, invalid_fraction: float = 0.1):
    """Candidate plans for the batched evaluator: random segment counts, random strictly
    increasing segment ends, random distinct nodes; a fraction is corrupted on purpose
    (repeated node, unsorted ends, out-of-range values, zero segments).

    Returns (nseg uint8 [B], ends int32 [B, k], nodes int32 [B, k]); unused slots are -1.
    """
    L, k = inst.L, inst.k
    rng = np.random.Generator(np.random.PCG64(seed))
    mmax = min(k, L)
    nseg = rng.integers(1, mmax + 1, size=count).astype(np.uint8)
    ends = np.full((count, k), -1, dtype=np.int32)
    nodes = np.full((count, k), -1, dtype=np.int32)
    for b in range(count):
        m = int(nseg[b])
        cuts = np.sort(rng.choice(L - 1, size=m - 1, replace=False)) if m > 1 else np.empty(0, int)
        ends[b, : m - 1] = cuts
        ends[b, m - 1] = L - 1
        nodes[b, :m] = rng.permutation(k)[:m]
    bad = np.flatnonzero(rng.random(count) < invalid_fraction)
    for b in bad:
        m = int(nseg[b])
        kind = int(rng.integers(0, 5))
        if kind == 0:
            nseg[b] = 0
        elif kind == 1:
            nseg[b] = min(255, mmax + 1 + int(rng.integers(0, 3)))
        elif kind == 2 and m >= 2:
            nodes[b, m - 1] = nodes[b, 0]
        elif kind == 3 and m >= 3:
            ends[b, 0], ends[b, 1] = ends[b, 1], ends[b, 0]
        else:
            nodes[b, 0] = k + int(rng.integers(0, 3))
    return nseg, ends, nodes


def pack_plans(nseg: np.ndarray, ends: np.ndarray, nodes: np.ndarray):
    """Compressed rows for the packed evaluator entry point: plan b keeps its first nseg[b] entries
    (none when nseg is outside [1, k]).  Values that 16 / 8 bits cannot hold are mapped to the
    largest code, which is out of range as well.  Returns (plan_off uint32 [B + 1], ends uint16
    [total], nodes uint8 [total])."""
    B, k = ends.shape
    keep = np.where((nseg >= 1) & (nseg <= k), nseg, 0).astype(np.int64)
    plan_off = np.zeros(B + 1, dtype=np.uint32)
    plan_off[1:] = np.cumsum(keep)
    sel = np.arange(k)[None, :] < keep[:, None]
    e = ends[sel].astype(np.int64)
    n = nodes[sel].astype(np.int64)
    e = np.where((e < 0) | (e > 0xFFFF), 0xFFFF, e).astype(np.uint16)
    n = np.where((n < 0) | (n > 0xFF), 0xFF, n).astype(np.uint8)
    return plan_off, e, n
