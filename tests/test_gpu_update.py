"""GPU tests for nbos_snapshot_update: a snapshot refreshed from new cluster state (no read-back,
no synchronisation) must place exactly as a snapshot created from that state would; state that
does not fit the stored layout is reported through the status word."""
from __future__ import annotations

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


def dev_state(w):
    import torch
    return [torch.from_numpy(getattr(w, k)).cuda().reshape(-1) for k in w.HOST_FIELDS]


def limits(w):
    import torch
    return torch.from_numpy(w.limit_num), torch.from_numpy(w.limit_den)


def place(nb, snap, w, config=None):
    import torch
    req = torch.from_numpy(w.requests).cuda()
    out = torch.full((w.n_snapshots, w.batch, 3), -7, dtype=torch.int32, device="cuda")
    found = torch.full((w.n_snapshots, w.batch), -7, dtype=torch.int32, device="cuda")
    nb.nbos_place_batch(snap, req, out, found, config=config)
    return out, found


def check(nb, snap, w, key_order=0, flags=0, config=None):
    out, found = place(nb, snap, w, config)
    assert nb.nbos_snapshot_status(snap) == nb.NBOS_OK
    ref = oracle.place_workload(w, key_order=key_order, flags=flags & 1, threads=8)
    np.testing.assert_array_equal(out.cpu().numpy(), ref[0])
    np.testing.assert_array_equal(found.cpu().numpy(), ref[1])


@pytest.mark.parametrize("key_order", [0, 1])
@pytest.mark.parametrize("flags", [0, 1, 2], ids=["plain", "idle", "key64"])
def test_updates_place_like_fresh_snapshots(nb, key_order, flags):
    first = W.make_config(1, batch=2000)
    snap = nb.snapshot_from_workload(first, key_order=key_order, flags=flags)
    check(nb, snap, first, key_order, flags)
    for seed in (11, 12, 13):
        w = W.make_config(1, batch=2000, seed=seed)            # same shape and value ranges, new state
        nb.nbos_snapshot_update(snap, *limits(w), *dev_state(w))
        check(nb, snap, w, key_order, flags)
        check(nb, snap, w, key_order, flags, nb.launch_config(lanes_per_request=32, host_split=2, tile_hosts=64))
    nb.nbos_snapshot_destroy(snap)


def test_queued_updates_without_synchronisation(nb):
    import torch
    states = [W.make_config(2, batch=3000, seed=s) for s in (2, 21, 22, 23)]
    snap = nb.snapshot_from_workload(states[0])
    results = []
    for w in states[1:]:                                        # update, place, update, place ... no sync
        nb.nbos_snapshot_update(snap, *limits(w), *dev_state(w))
        results.append(place(nb, snap, w))
    torch.cuda.synchronize()
    assert nb.nbos_snapshot_status(snap) == nb.NBOS_OK
    for w, (out, found) in zip(states[1:], results):
        ref = oracle.place_workload(w, threads=8)
        np.testing.assert_array_equal(out.cpu().numpy(), ref[0])
        np.testing.assert_array_equal(found.cpu().numpy(), ref[1])
    nb.nbos_snapshot_destroy(snap)


def test_many_snapshots_new_limits_and_host_arrays(nb):
    import torch
    a = W.what_if_sweep(150, 96, 200)
    snap = nb.snapshot_from_workload(a)
    b = W.what_if_sweep(150, 96, 200, host_seed0=5000, request_seed0=6000)
    b.limit_num[:], b.limit_den[:] = a.limit_num[::-1].copy(), a.limit_den[::-1].copy()
    nb.nbos_snapshot_update(snap, *limits(b), *dev_state(b))
    check(nb, snap, b)
    c = W.what_if_sweep(150, 96, 200, host_seed0=7000, request_seed0=8000)
    host_arrays = [torch.from_numpy(getattr(c, k)).reshape(-1) for k in c.HOST_FIELDS]
    nb.nbos_snapshot_update_host(snap, *limits(c), *host_arrays)
    check(nb, snap, c)
    nb.nbos_snapshot_destroy(snap)
    # the cluster-wide dynamic limit is recomputed from the new state
    snap = nb.snapshot_from_workload(a, flags=nb.NBOS_LIMIT_CLUSTER_SR)
    nb.nbos_snapshot_update(snap, None, None, *dev_state(b))
    out, found = place(nb, snap, b)
    assert nb.nbos_snapshot_status(snap) == nb.NBOS_OK
    fresh = nb.place_workload(b, flags=nb.NBOS_LIMIT_CLUSTER_SR)
    np.testing.assert_array_equal(out.cpu().numpy(), fresh[0])
    nb.nbos_snapshot_destroy(snap)


def test_mixed_gpu_counts(nb):
    a = W.mixed_gpu_cluster(600, 1500, seed=51)
    snap = nb.snapshot_from_workload(a)
    rng = np.random.default_rng(1)
    b = W.mixed_gpu_cluster(600, 1500, seed=51)
    perm = rng.permutation(600)                                  # same hosts in another order
    for k in b.HOST_FIELDS:
        getattr(b, k)[0] = getattr(a, k)[0][perm]
    nb.nbos_snapshot_update(snap, *limits(b), *dev_state(b))
    check(nb, snap, b)
    nb.nbos_snapshot_destroy(snap)


def test_state_that_does_not_fit_is_reported(nb):
    base = W.make_config(1, batch=500)
    snap = nb.snapshot_from_workload(base)

    def update_with(mod):
        w = W.make_config(1, batch=500)
        mod(w)
        nb.nbos_snapshot_update(snap, *limits(w), *dev_state(w))
        return nb.nbos_snapshot_status(snap)

    assert update_with(lambda w: w.mem_mb.__setitem__((0, 3), 1 << 30)) == nb.NBOS_ERR_STALE_LAYOUT
    assert update_with(lambda w: w.gpus_total.__setitem__((0, 3), 16)) == nb.NBOS_ERR_STALE_LAYOUT
    assert update_with(lambda w: w.gpus_subscribed.__setitem__((0, 3), -2)) == nb.NBOS_ERR_RANGE
    assert update_with(lambda w: w.gpus_committed.__setitem__((0, 3), 9)) == nb.NBOS_ERR_RANGE

    def heavy_subscription(w):
        w.limit_num[0], w.limit_den[0] = 50, 1                   # room for 1,200 subscribed GPUs per host
        w.gpus_subscribed[0, 3] = 100                            # S + g = 108 needs a wider ratio field
    assert update_with(heavy_subscription) == nb.NBOS_ERR_STALE_LAYOUT
    # a good update clears the status and the snapshot works again
    assert update_with(lambda w: None) == nb.NBOS_OK
    check(nb, snap, base)
    # shape or flags that differ are refused at call time
    other = W.make_config(0)
    with pytest.raises((nb.NbosError, ValueError)):
        nb.nbos_snapshot_update(snap, *limits(other), *dev_state(other))
    nb.nbos_snapshot_destroy(snap)
