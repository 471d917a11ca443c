"""GPU parity for sequential placement with commits against the CPU checker, bit-exact: chosen
hosts, found counts and the subscribed GPUs of every host after the last request."""
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


def gpu_sequential(nb, w, key_order=0, flags=0):
    import torch
    snap = nb.snapshot_from_workload(w, key_order=key_order, flags=flags | nb.NBOS_ROOM_FOR_COMMITS)
    try:
        req = torch.from_numpy(w.requests).cuda()
        out = torch.full((w.n_snapshots, w.batch, 3), -7, dtype=torch.int32, device="cuda")
        found = torch.full((w.n_snapshots, w.batch), -7, dtype=torch.int32, device="cuda")
        sub = torch.full((w.n_snapshots, w.n_hosts), -7, dtype=torch.int32, device="cuda")
        nb.nbos_place_batch_sequential(snap, req, out, found, sub)
        assert nb.nbos_snapshot_status(snap) == nb.NBOS_OK
        return out.cpu().numpy(), found.cpu().numpy(), sub.cpu().numpy()
    finally:
        nb.nbos_snapshot_destroy(snap)


def cpu_sequential(w, key_order=0, flags=0):
    res = [oracle.place_sequential(w.gpus_total[n], w.gpus_subscribed[n], w.gpus_committed[n],
                                   w.vram_gb[n], w.millicpus[n], w.mem_mb[n], int(w.limit_num[n]),
                                   int(w.limit_den[n]), w.requests[n], replicas_R=w.replicas_R,
                                   key_order=key_order, flags=flags & 1)
           for n in range(w.n_snapshots)]
    return tuple(np.stack([r[i] for r in res]) for i in range(3))


def check(nb, w, key_order=0, flags=0, what=""):
    got = gpu_sequential(nb, w, key_order, flags)
    ref = cpu_sequential(w, key_order, flags)
    for name, a, b in zip(("hosts", "found", "subscribed"), got, ref):
        np.testing.assert_array_equal(a, b, err_msg=f"{what or w.name}: {name}")
    return ref


@pytest.mark.parametrize("key_order", [0, 1])
def test_benchmark_shapes(nb, key_order):
    ref = check(nb, W.make_config(0), key_order)
    assert (ref[1] == 3).any()
    check(nb, W.make_config(1, batch=6000), key_order)
    ref = check(nb, W.make_config(2, batch=3000), key_order)
    assert (ref[1] < 3).any()
    check(nb, W.make_config(3, batch=1500), key_order)            # 4,096 hosts: 4 per thread
    check(nb, W.make_config(4, batch=300, n_snapshots=40), key_order)


@pytest.mark.parametrize("flags", [0, 1, 2, 3], ids=["key32", "idle", "key64", "idle+key64"])
def test_mixed_hosts_flags_and_key_widths(nb, flags):
    for w in (W.mixed_gpu_cluster(700, 4000, seed=41), W.mixed_gpu_cluster(33, 500, seed=42),
              W.uniform_cluster(1, 20, seed=43), W.uniform_cluster(2, 20, seed=44)):
        check(nb, w, key_order=flags & 1, flags=flags)


def test_cluster_fills_up(nb):
    """A loose limit and many requests: the cluster takes kernels until nothing fits any more."""
    w = W.uniform_cluster(96, 3000, seed=9, raw_limit="4")
    ref = check(nb, w)
    assert (ref[1][0, :50] == 3).all() and (ref[1][0, -50:] < 3).all()
    cap = 32                                                    # raw limit 4 on 8 GPUs
    assert ref[2].max() <= cap
    # the largest table one block takes
    check(nb, W.uniform_cluster(8192, 300, seed=10), what="8192 hosts")
    w = W.uniform_cluster(5000, 200, seed=11)
    w.requests[0, 3] = [-1, 0, 0, 0]
    w.requests[0, 4] = [0, 0, 0, 0]
    check(nb, w, what="5000 hosts, odd requests")


@pytest.mark.parametrize("flags", [0, 2, 3], ids=["key32", "key64", "idle+key64"])
def test_tables_spread_over_a_block_cluster(nb, flags):
    """More than 8,192 hosts: 2, 4 or 8 blocks of a cluster share the table, ragged last block,
    winners in different blocks and in the same block, several snapshots, odd requests."""
    for hosts, batch, seed in ((8193, 120, 51), (20000, 150, 52), (40000, 60, 53), (65536, 40, 54)):
        w = W.uniform_cluster(hosts, batch, seed=seed)
        w.requests[0, 5] = [-1, 0, 0, 0]
        w.requests[0, 6] = [0, 0, 0, 0]
        check(nb, w, key_order=flags & 1, flags=flags, what=f"{hosts} hosts, flags {flags}")
    w = W.mixed_gpu_cluster(12000, 200, seed=55)
    check(nb, w, key_order=flags & 1, flags=flags, what="12000 mixed hosts")


def test_cluster_form_fills_up_and_batches_snapshots(nb):
    """Tight state on a large table: the best hosts sit in one block's run until they fill up and
    the choice moves to the next; three snapshots run as three clusters."""
    w = W.uniform_cluster(10000, 2500, seed=56, raw_limit="4")
    ref = check(nb, w, what="10000 hosts, loose limit")
    assert (ref[1] == 3).any()
    check(nb, W.what_if_sweep(3, 9000, 100), what="three snapshots of 9000 hosts")


def test_argument_errors(nb):
    import torch
    w = W.make_config(0)
    req = torch.from_numpy(w.requests).cuda()
    out = torch.empty((1, w.batch, 3), dtype=torch.int32, device="cuda")
    snap = nb.snapshot_from_workload(w)                          # without NBOS_ROOM_FOR_COMMITS
    with pytest.raises(nb.NbosError) as e:
        nb.nbos_place_batch_sequential(snap, req, out)
    assert e.value.status == nb.NBOS_ERR_INVALID_ARG
    nb.nbos_snapshot_destroy(snap)
    big = W.uniform_cluster(65537, 8, seed=1)
    snap = nb.snapshot_from_workload(big, flags=nb.NBOS_ROOM_FOR_COMMITS)
    with pytest.raises(nb.NbosError) as e:
        nb.nbos_place_batch_sequential(snap, torch.from_numpy(big.requests).cuda(),
                                       torch.empty((1, 8, 3), dtype=torch.int32, device="cuda"))
    assert e.value.status == nb.NBOS_ERR_RANGE
    nb.nbos_snapshot_destroy(snap)
    # the frozen-batch entry point still works on a snapshot with room for commits, same answers
    snap = nb.snapshot_from_workload(w, flags=nb.NBOS_ROOM_FOR_COMMITS)
    found = torch.empty((1, w.batch), dtype=torch.int32, device="cuda")
    nb.nbos_place_batch(snap, req, out, found)
    ref = oracle.place_workload(w)
    np.testing.assert_array_equal(out.cpu().numpy(), ref[0])
    nb.nbos_snapshot_destroy(snap)
