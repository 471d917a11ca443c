"""The allocation-free placement entry point against the ordinary one.

Some users of this library cannot allocate device memory at call time: their GPU's free memory
already belongs to another pool (a training or serving job on the same device), or they sit in a
control loop where an allocation's device-wide synchronisation costs too much. For them
nbos_place_batch_noalloc keeps the per-slice candidates in a fixed array inside the library.
It must return exactly the bytes nbos_place_batch returns (index work: bit-exact) -- which are
also the CPU checker's -- call after call, although every call reuses that array with the previous
call's contents still in it; and it must really leave the device's memory alone.

This file is collected last on purpose: a run that stops at the first failure has then already
been through every other test.
"""
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


def _run(nb, snap, w, requests, entry, **kw):
    import torch
    req = torch.from_numpy(np.ascontiguousarray(requests)).cuda()
    n, b = w.n_snapshots, requests.shape[1]
    out = torch.full((n, b, 3), -7, dtype=torch.int32, device="cuda")
    found = torch.full((n, b), -7, dtype=torch.int32, device="cuda")
    entry(snap, req, out, found, **kw)
    assert nb.nbos_snapshot_status(snap) == nb.NBOS_OK
    return out.cpu().numpy(), found.cpu().numpy()


@pytest.mark.parametrize("host_split", [0, 2, 5, 64])
def test_two_calls_in_a_row_match_the_allocating_entry_point(nb, host_split):
    for w in (W.make_config(2, batch=3000), W.mixed_gpu_cluster(777, 1500, seed=21),
              W.what_if_sweep(6, 200, 301)):
        snap = nb.snapshot_from_workload(w)
        try:
            first = w.requests
            # second call: a shorter, different batch, so stale candidates of the first call stay
            # in the array behind and beside the ones the second call writes
            second = np.ascontiguousarray(w.requests[:, ::-1][:, : max(1, w.batch // 3)])
            for requests in (first, second):
                ref = _run(nb, snap, w, requests, nb.nbos_place_batch,
                           config=nb.launch_config(lanes_per_request=32, host_split=3, tile_hosts=64))
                got = _run(nb, snap, w, requests, nb.nbos_place_batch_noalloc, host_split=host_split)
                np.testing.assert_array_equal(got[0], ref[0])
                np.testing.assert_array_equal(got[1], ref[1])
                plain = _run(nb, snap, w, requests, nb.nbos_place_batch)
                np.testing.assert_array_equal(got[0], plain[0])
                # and the checker's, computed on the CPU from the paper's rule
                sub = dataclasses.replace(w, requests=np.ascontiguousarray(requests), batch=requests.shape[1])
                want = oracle.place_workload(sub, threads=min(16, os.cpu_count() or 1))
                np.testing.assert_array_equal(got[0], want[0])
                np.testing.assert_array_equal(got[1], want[1])
        finally:
            nb.nbos_snapshot_destroy(snap)


def test_no_device_memory_is_taken_or_returned(nb):
    """Across calls of the allocation-free entry point neither the driver's count of free device
    memory nor what PyTorch's allocator holds may move: a caller whose memory is spoken for must be
    able to rely on that. (The first call per device resolves the array's address; it is made
    before the measurement, as the header asks start-up code to do.)"""
    import torch
    w = W.make_config(2, batch=2000)
    snap = nb.snapshot_from_workload(w)
    try:
        req = torch.from_numpy(w.requests).cuda()
        out = torch.empty((1, w.batch, 3), dtype=torch.int32, device="cuda")
        found = torch.empty((1, w.batch), dtype=torch.int32, device="cuda")
        nb.nbos_place_batch_noalloc(snap, req, out, found, host_split=4)     # start-up call
        torch.cuda.synchronize()
        free0, _ = torch.cuda.mem_get_info()
        reserved0, allocated0 = torch.cuda.memory_reserved(), torch.cuda.memory_allocated()
        for split in (4, 1, 7, 4):
            nb.nbos_place_batch_noalloc(snap, req, out, found, host_split=split)
        torch.cuda.synchronize()
        free1, _ = torch.cuda.mem_get_info()
        assert free1 == free0
        assert (torch.cuda.memory_reserved(), torch.cuda.memory_allocated()) == (reserved0, allocated0)
        want = oracle.place_workload(w, threads=min(16, os.cpu_count() or 1))
        np.testing.assert_array_equal(out.cpu().numpy(), want[0])
        np.testing.assert_array_equal(found.cpu().numpy(), want[1])
    finally:
        nb.nbos_snapshot_destroy(snap)


def test_wide_keys_use_the_same_array(nb):
    w = W.mixed_gpu_cluster(500, 900, seed=4)
    snap = nb.snapshot_from_workload(w, flags=nb.NBOS_FORCE_KEY64)
    try:
        for _ in range(2):
            ref = _run(nb, snap, w, w.requests, nb.nbos_place_batch)
            got = _run(nb, snap, w, w.requests, nb.nbos_place_batch_noalloc, host_split=4)
            np.testing.assert_array_equal(got[0], ref[0])
            np.testing.assert_array_equal(got[1], ref[1])
    finally:
        nb.nbos_snapshot_destroy(snap)


def test_batches_beyond_the_built_in_array_are_refused(nb):
    import torch
    w = W.make_config(1, batch=16)
    snap = nb.snapshot_from_workload(w)
    try:
        # 8 slices x 3 keys x 4 bytes = 96 bytes per request; 8 MiB holds 87,381 requests
        b = 100_000
        req = torch.zeros((1, b, 4), dtype=torch.int32, device="cuda")
        out = torch.full((1, b, 3), -7, dtype=torch.int32, device="cuda")
        with pytest.raises(nb.NbosError) as e:
            nb.nbos_place_batch_noalloc(snap, req, out, None, host_split=8)
        assert e.value.status == nb.NBOS_ERR_NO_MEMORY
        assert "built-in buffer" in str(e.value)
        assert (out == -7).all()                      # nothing was launched
        with pytest.raises(nb.NbosError) as e:
            nb.nbos_place_batch_noalloc(snap, req, out, None, host_split=65)
        assert e.value.status == nb.NBOS_ERR_INVALID_ARG
        # the same batch is fine without slicing, and with few enough slices
        ref = torch.empty_like(out)
        nb.nbos_place_batch(snap, req, ref, None)
        nb.nbos_place_batch_noalloc(snap, req, out, None, host_split=1)
        assert torch.equal(out, ref)
        out.fill_(-7)
        nb.nbos_place_batch_noalloc(snap, req, out, None, host_split=4)
        assert torch.equal(out, ref)
    finally:
        nb.nbos_snapshot_destroy(snap)
