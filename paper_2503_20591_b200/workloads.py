"""Seeded synthetic inputs for batched replica placement.

This module only draws random host states and resource requests. It holds
none of the placement rule's arithmetic (no feasibility test, no key, no
selection), so both the CUDA path's tests and the CPU checker's tests can be
fed from it without sharing any of the method.

The paper evaluates on a private production trace replayed on 30 servers of
8 GPUs each (Section 5.1) and describes a production fleet of about 3,000
8-GPU servers (Section 2.4); it gives no distribution for the GPU count of a
request. The five workloads below are synthetic stand-ins whose host counts
(32 .. 4,096) bracket those cluster sizes.

Array conventions (all int32, C-contiguous):

    gpus_total, gpus_subscribed, gpus_committed   [N, H]   G, S, C of Section 3.4.1
    vram_gb, millicpus, mem_mb                    [N, H]   capacity a request is compared with
    limit_num, limit_den                          [N]      SR limit as a rational, in the paper's
                                                           units (S / (G * R))
    requests                                      [N, B, 4] columns (GPUs, VRAM GB, millicpus,
                                                           memory MB) -- the resource request of
                                                           Section 3.2.1
"""
from __future__ import annotations

import hashlib
from dataclasses import dataclass, field
from fractions import Fraction

import numpy as np

REPLICAS_R = 3  # Section 3.4.1: R = 3 replicas per distributed kernel

GPUS_PER_HOST = 8
VRAM_GB_PER_GPU = 80
MILLICPUS_PER_HOST = 128_000
MEM_MB_PER_HOST = 1_048_576

SWEEP_RAW_LIMITS = ("1", "5/4", "3/2", "7/4", "2", "5/2", "3", "4")

GPU_ASK_VALUES = (1, 2, 4, 8)
GPU_ASK_PROBS_DEFAULT = (0.5, 0.25, 0.15, 0.1)
GPU_ASK_PROBS_SKEWED = (0.2, 0.2, 0.3, 0.3)


@dataclass
class Workload:
    name: str
    n_snapshots: int
    n_hosts: int
    batch: int
    replicas_R: int
    gpus_total: np.ndarray
    gpus_subscribed: np.ndarray
    gpus_committed: np.ndarray
    vram_gb: np.ndarray
    millicpus: np.ndarray
    mem_mb: np.ndarray
    limit_num: np.ndarray
    limit_den: np.ndarray
    requests: np.ndarray
    raw_limits: list = field(default_factory=list)

    HOST_FIELDS = ("gpus_total", "gpus_subscribed", "gpus_committed",
                   "vram_gb", "millicpus", "mem_mb")

    @property
    def pairs(self) -> int:
        return self.n_snapshots * self.n_hosts * self.batch

    @property
    def decisions(self) -> int:
        return self.n_snapshots * self.batch

    def sha256(self) -> str:
        h = hashlib.sha256()
        for k in self.HOST_FIELDS + ("limit_num", "limit_den", "requests"):
            a = np.ascontiguousarray(getattr(self, k))
            h.update(k.encode())
            h.update(str(a.shape).encode())
            h.update(a.tobytes())
        return h.hexdigest()


def raw_limit_to_paper_units(raw: str | Fraction, replicas_R: int = REPLICAS_R) -> Fraction:
    """A 'raw' limit is subscribed GPUs per physical GPU (S / G). The paper's SR
    also divides by R, so the same watermark in the paper's units is raw / R."""
    return Fraction(raw) / replicas_R


def _host_state_default(rng: np.random.Generator, h: int):
    """G = 8; S ~ U{0..16}; C ~ U{0..min(8, S)}."""
    G = np.full(h, GPUS_PER_HOST, dtype=np.int64)
    S = rng.integers(0, 17, size=h)
    C = rng.integers(0, np.minimum(GPUS_PER_HOST, S) + 1)
    return G, S, C


def _capacities(rng: np.random.Generator, G, C):
    """VRAM of the GPUs that are not bound right now; CPU and memory left after
    a uniformly drawn amount already in use."""
    h = G.shape[0]
    vram = VRAM_GB_PER_GPU * (G - C)
    cpu = MILLICPUS_PER_HOST - rng.integers(0, MILLICPUS_PER_HOST + 1, size=h)
    mem = MEM_MB_PER_HOST - rng.integers(0, MEM_MB_PER_HOST + 1, size=h)
    return vram, cpu, mem


def _requests(rng: np.random.Generator, b: int, probs) -> np.ndarray:
    g = rng.choice(np.asarray(GPU_ASK_VALUES), size=b, p=np.asarray(probs))
    v = 16 * g
    c = rng.integers(1000, 16001, size=b)
    m = rng.integers(1024, 65537, size=b)
    return np.stack([g, v, c, m], axis=1).astype(np.int32)


def _pack(name, hosts_list, req_list, raw_limits, replicas_R=REPLICAS_R) -> Workload:
    n = len(hosts_list)
    cols = list(zip(*hosts_list))  # 6 tuples of N arrays
    arrs = [np.ascontiguousarray(np.stack(c).astype(np.int32)) for c in cols]
    lims = [raw_limit_to_paper_units(r, replicas_R) for r in raw_limits]
    return Workload(
        name=name, n_snapshots=n, n_hosts=arrs[0].shape[1], batch=req_list[0].shape[0],
        replicas_R=replicas_R,
        gpus_total=arrs[0], gpus_subscribed=arrs[1], gpus_committed=arrs[2],
        vram_gb=arrs[3], millicpus=arrs[4], mem_mb=arrs[5],
        limit_num=np.array([l.numerator for l in lims], dtype=np.int32),
        limit_den=np.array([l.denominator for l in lims], dtype=np.int32),
        requests=np.ascontiguousarray(np.stack(req_list).astype(np.int32)),
        raw_limits=[str(r) for r in raw_limits],
    )


def _default_snapshot(rng, h):
    G, S, C = _host_state_default(rng, h)
    vram, cpu, mem = _capacities(rng, G, C)
    return G, S, C, vram, cpu, mem


def uniform_cluster(n_hosts: int, batch: int, seed: int, name: str = "uniform",
                    raw_limit: str = "2") -> Workload:
    """Workloads 0 and 1: every host has 8 GPUs and the default state distribution."""
    rng = np.random.Generator(np.random.PCG64(seed))
    hosts = _default_snapshot(rng, n_hosts)
    req = _requests(rng, batch, GPU_ASK_PROBS_DEFAULT)
    return _pack(name, [hosts], [req], [raw_limit])


def oversubscribed_cluster(n_hosts: int, batch: int, seed: int,
                           name: str = "oversubscribed") -> Workload:
    """Workload 2: about 40 % of hosts at or above the raw limit 2.0 (S in 16..32, no
    request fits there); the others crowd just below it (S = 15 - X, X geometric with
    p = 0.45), so only a handful of hosts can still take an 8-GPU ask. Independently,
    committed GPUs are near the total on half of the hosts. CPU and memory are scarce
    as well (free millicpus ~ U{0..20000}, free MB ~ U{0..80000}), so which of those few
    hosts fit differs from request to request and fewer than three are found for some."""
    rng = np.random.Generator(np.random.PCG64(seed))
    G = np.full(n_hosts, GPUS_PER_HOST, dtype=np.int64)
    over = rng.random(n_hosts) < 0.4
    below = 15 - np.minimum(15, rng.geometric(0.45, size=n_hosts) - 1)
    S = np.where(over, rng.integers(16, 33, size=n_hosts), below)
    busy = rng.random(n_hosts) < 0.5
    c_busy = rng.integers(np.minimum(6, S), np.minimum(GPUS_PER_HOST, S) + 1)
    c_calm = rng.integers(0, np.minimum(GPUS_PER_HOST, S) + 1)
    C = np.where(busy, c_busy, c_calm)
    vram = VRAM_GB_PER_GPU * (G - C)
    cpu = rng.integers(0, 20_001, size=n_hosts)
    mem = rng.integers(0, 80_001, size=n_hosts)
    req = _requests(rng, batch, GPU_ASK_PROBS_SKEWED)
    return _pack(name, [(G, S, C, vram, cpu, mem)], [req], ["2"])


def tie_heavy_cluster(n_hosts: int, batch: int, seed: int, name: str = "tie_heavy",
                      n_templates: int = 8, copy_fraction: float = 0.75) -> Workload:
    """Workload 3: 75 % of hosts (random positions) are exact copies of one of 8
    template states, so placement keys tie and the host id decides."""
    rng = np.random.Generator(np.random.PCG64(seed))
    tmpl = np.stack(_default_snapshot(rng, n_templates))          # [6, n_templates]
    fresh = np.stack(_default_snapshot(rng, n_hosts))             # [6, n_hosts]
    is_copy = rng.random(n_hosts) < copy_fraction
    which = rng.integers(0, n_templates, size=n_hosts)
    state = np.where(is_copy[None, :], tmpl[:, which], fresh)
    req = _requests(rng, batch, GPU_ASK_PROBS_DEFAULT)
    return _pack(name, [tuple(state)], [req], ["2"])


def what_if_sweep(n_snapshots: int, n_hosts: int, batch: int, name: str = "what_if_sweep",
                  host_seed0: int = 1000, request_seed0: int = 2000) -> Workload:
    """Workload 4: independent snapshots, each paired with one of 8 raw limits and
    its own request batch."""
    hosts, reqs, lims = [], [], []
    for i in range(n_snapshots):
        hrng = np.random.Generator(np.random.PCG64(host_seed0 + i))
        rrng = np.random.Generator(np.random.PCG64(request_seed0 + i))
        hosts.append(_default_snapshot(hrng, n_hosts))
        reqs.append(_requests(rrng, batch, GPU_ASK_PROBS_DEFAULT))
        lims.append(SWEEP_RAW_LIMITS[i % len(SWEEP_RAW_LIMITS)])
    return _pack(name, hosts, reqs, lims)


def mixed_gpu_cluster(n_hosts: int, batch: int, seed: int, name: str = "mixed_gpus",
                      raw_limit: str = "3") -> Workload:
    """Not one of the five benchmark workloads: hosts with 1..8 GPUs (Section 3.4.1
    allows G from 1 to 8), so that the subscription-ratio order depends on the
    request's GPU count. Used by tests to exercise the general key."""
    rng = np.random.Generator(np.random.PCG64(seed))
    G = rng.integers(1, GPUS_PER_HOST + 1, size=n_hosts)
    S = rng.integers(0, 3 * G + 1)
    C = rng.integers(0, np.minimum(G, S) + 1)
    vram, cpu, mem = _capacities(rng, G, C)
    g = rng.integers(0, 9, size=batch)
    v = 16 * g
    c = rng.integers(1000, 16001, size=batch)
    m = rng.integers(1024, 65537, size=batch)
    req = np.stack([g, v, c, m], axis=1).astype(np.int32)
    return _pack(name, [(G, S, C, vram, cpu, mem)], [req], [raw_limit])


# The five benchmark workloads, by index. Sizes: (N, H, B).
CONFIG_SHAPES = {
    0: (1, 32, 1_024),
    1: (1, 256, 16_384),
    2: (1, 1_024, 262_144),
    3: (1, 4_096, 1_048_576),
    4: (256, 1_024, 4_096),
}


def make_config(index: int, batch: int | None = None, n_snapshots: int | None = None,
                seed: int | None = None) -> Workload:
    """Build benchmark workload `index` (0..4). `batch` / `n_snapshots` shrink it
    (same distributions, same seeds) for quick checks; `seed` overrides the
    workload's own seed (used to draw several distinct batches of one shape)."""
    n, h, b = CONFIG_SHAPES[index]
    b = b if batch is None else batch
    n = n if n_snapshots is None else n_snapshots
    s = index if seed is None else seed
    if index == 0:
        return uniform_cluster(h, b, s, "cfg0_tiny")
    if index == 1:
        return uniform_cluster(h, b, s, "cfg1_medium")
    if index == 2:
        return oversubscribed_cluster(h, b, s, "cfg2_oversubscribed")
    if index == 3:
        return tie_heavy_cluster(h, b, s, "cfg3_tie_heavy")
    if index == 4:
        off = 0 if seed is None else seed
        return what_if_sweep(n, h, b, "cfg4_what_if_sweep", 1000 + off, 2000 + off)
    raise ValueError(f"no such workload: {index}")


def extra_request_batches(index: int, count: int, batch: int | None = None,
                          n_snapshots: int | None = None, seed0: int = 10_000) -> list:
    """`count` further request batches [N, B, 4] for benchmark workload `index`, drawn from that
    workload's request distribution with seeds of their own (seed0 + 100 * index + k). Used to
    rotate inputs so that successive timed steps do not find their requests in the L2 cache."""
    n, _, b = CONFIG_SHAPES[index]
    b = b if batch is None else batch
    n = n if n_snapshots is None else n_snapshots
    probs = GPU_ASK_PROBS_SKEWED if index == 2 else GPU_ASK_PROBS_DEFAULT
    out = []
    for k in range(count):
        rng = np.random.Generator(np.random.PCG64(seed0 + 100 * index + k))
        out.append(np.ascontiguousarray(
            np.stack([_requests(rng, b, probs) for _ in range(n)]).astype(np.int32)))
    return out
