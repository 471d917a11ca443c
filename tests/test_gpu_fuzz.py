"""Randomised GPU parity: many small clusters and batches with odd shapes, value ranges, limits,
flags and launch shapes, each compared bit for bit with the CPU checker."""
from __future__ import annotations

import dataclasses
import os

import numpy as np
import pytest

import oracle
from paper_2503_20591_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def nb():
    import torch
    from paper_2503_20591_b200 import binding, build as lib_build
    lib_build.build()
    assert torch.cuda.is_available()
    binding.load_library()
    return binding


def random_workload(rng) -> W.Workload:
    n = int(rng.choice([1, 1, 1, 2, 5]))
    h = int(rng.choice([1, 2, 7, 31, 32, 33, 64, 100, 255, 700, 1500]))
    b = int(rng.choice([1, 3, 31, 64, 257, 1000]))
    gmax = int(rng.choice([1, 4, 8, 8, 16, 100]))
    # mixed GPU counts only up to 16 per host: the exact integer ratio key needs the lcm of the
    # distinct counts, which the library refuses (NBOS_ERR_RANGE) once it passes 2^40
    uniform = rng.random() < 0.5 or gmax > 16
    G = np.full((n, h), gmax) if uniform else rng.integers(0, gmax + 1, size=(n, h))
    S = rng.integers(0, 3 * np.maximum(G, 1) + 1)
    C = rng.integers(0, np.minimum(G, S) + 1)
    scale = int(rng.choice([1, 100, 10_000, 1_000_000, 2_000_000_000]))
    caps = [rng.integers(0, scale + 1, size=(n, h)) for _ in range(3)]
    lims = [(int(rng.integers(0, 9)), int(rng.integers(1, 13))) for _ in range(n)]
    g = rng.integers(0, gmax + 2, size=(n, b))
    req = np.stack([g] + [rng.integers(0, scale + scale // 8 + 2, size=(n, b)) for _ in range(3)], axis=-1)
    req[rng.random((n, b)) < 0.02] *= -1
    return W.Workload(
        name="fuzz", n_snapshots=n, n_hosts=h, batch=b, replicas_R=int(rng.choice([1, 3, 3, 5])),
        gpus_total=G.astype(np.int32), gpus_subscribed=S.astype(np.int32), gpus_committed=C.astype(np.int32),
        vram_gb=caps[0].astype(np.int32), millicpus=caps[1].astype(np.int32), mem_mb=caps[2].astype(np.int32),
        limit_num=np.array([l[0] for l in lims], dtype=np.int32),
        limit_den=np.array([l[1] for l in lims], dtype=np.int32),
        requests=np.ascontiguousarray(req.astype(np.int32)))


# NBOS_FUZZ_CASES widens the campaign (e.g. 20000 for a long run; the default keeps the suite short)
@pytest.mark.parametrize("seed", range(int(os.environ.get("NBOS_FUZZ_CASES", "150"))))
def test_random_cases(nb, seed):
    rng = np.random.default_rng(10_000 + seed)
    w = random_workload(rng)
    key_order = int(rng.integers(0, 2))
    flags = int(rng.integers(0, 2))
    lib_flags = int(rng.choice([0, 0, nb.NBOS_FORCE_KEY64, nb.NBOS_ROOM_FOR_COMMITS]))
    shape = dict(lanes_per_request=int(rng.choice([0, 1, 2, 4, 8, 16, 32])),
                 requests_per_lane=int(rng.choice([0, 1, 2, 4, 8])),
                 host_split=int(rng.choice([0, 0, 1, 2, 3])),
                 tile_hosts=int(rng.choice([0, 32, 64, 256])),
                 pair_mode=int(rng.choice([0, 0, 0, 1, 2, 3, 4, 5])),
                 first_fit=int(rng.choice([0, 0, 1])))
    got = nb.place_workload(w, key_order=key_order, flags=flags | lib_flags, config=nb.launch_config(**shape))
    ref = oracle.place_workload(w, key_order=key_order, flags=flags)
    what = f"seed {seed}: N={w.n_snapshots} H={w.n_hosts} B={w.batch} {shape} order={key_order} flags={flags | lib_flags}"
    np.testing.assert_array_equal(got[0], ref[0], err_msg=what)
    np.testing.assert_array_equal(got[1], ref[1], err_msg=what)
    # the sequential entry point on the same inputs (its own reference)
    if w.n_hosts <= 8192:
        import torch
        snap = nb.snapshot_from_workload(w, key_order=key_order, flags=flags | nb.NBOS_ROOM_FOR_COMMITS)
        out = torch.empty((w.n_snapshots, w.batch, 3), dtype=torch.int32, device="cuda")
        found = torch.empty((w.n_snapshots, w.batch), dtype=torch.int32, device="cuda")
        sub = torch.empty((w.n_snapshots, w.n_hosts), dtype=torch.int32, device="cuda")
        nb.nbos_place_batch_sequential(snap, torch.from_numpy(w.requests).cuda(), out, found, sub)
        assert nb.nbos_snapshot_status(snap) == nb.NBOS_OK
        nb.nbos_snapshot_destroy(snap)
        for n in range(w.n_snapshots):
            r = oracle.place_sequential(w.gpus_total[n], w.gpus_subscribed[n], w.gpus_committed[n],
                                        w.vram_gb[n], w.millicpus[n], w.mem_mb[n], int(w.limit_num[n]),
                                        int(w.limit_den[n]), w.requests[n], replicas_R=w.replicas_R,
                                        key_order=key_order, flags=flags)
            np.testing.assert_array_equal(out[n].cpu().numpy(), r[0], err_msg=what + " (sequential hosts)")
            np.testing.assert_array_equal(sub[n].cpu().numpy(), r[2], err_msg=what + " (sequential S)")
