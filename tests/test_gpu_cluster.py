"""GPU parity for the cluster-wide reductions (Sections 3.4.1 third factor, 3.4.2, 3.2.1):
sums, auto-scaler sign, dynamic cluster-wide SR limit in placement, scale-out deficit."""
from __future__ import annotations

import dataclasses

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


@pytest.mark.parametrize("maker", [lambda: W.make_config(0), lambda: W.make_config(4, batch=8),
                                   lambda: W.mixed_gpu_cluster(70001, 4, seed=1),
                                   lambda: W.what_if_sweep(7, 333, 5)])
@pytest.mark.parametrize("f", [(21, 20), (1, 1), (3, 1), (0, 1)])
def test_sums_and_autoscaler_sign(nb, maker, f):
    import torch
    w = maker()
    dev = [torch.from_numpy(getattr(w, k)).cuda().reshape(-1) for k in w.HOST_FIELDS[:3]]
    out = torch.full((w.n_snapshots, 4), -77, dtype=torch.int64, device="cuda")
    nb.nbos_cluster_sums(*dev, w.n_snapshots, w.n_hosts, out, f_num=f[0], f_den=f[1])
    got = out.cpu().numpy()
    for n in range(w.n_snapshots):
        sums = oracle.cluster_sums(w.gpus_total[n], w.gpus_subscribed[n], w.gpus_committed[n])
        assert tuple(got[n, :3]) == sums
        assert got[n, 3] == oracle.autoscale(sums[0], sums[2], *f)


@pytest.mark.parametrize("key_order", [0, 1])
@pytest.mark.parametrize("flags", [0, 1])
def test_placement_under_the_dynamic_cluster_limit(nb, key_order, flags):
    for w in (W.make_config(1, batch=3000), W.make_config(2, batch=3000),
              W.what_if_sweep(12, 200, 150), W.mixed_gpu_cluster(400, 2000, seed=12)):
        got = nb.place_workload(w, key_order=key_order, flags=flags | nb.NBOS_LIMIT_CLUSTER_SR)
        # the checker gets the limit from its own sums, snapshot by snapshot
        nums, dens = [], []
        for n in range(w.n_snapshots):
            num, den = oracle.cluster_limit(w.gpus_total[n], w.gpus_subscribed[n], w.gpus_committed[n],
                                            replicas_R=w.replicas_R)
            nums.append(num)
            dens.append(max(den, 1))
        ww = dataclasses.replace(w, limit_num=np.array(nums, dtype=np.int64),
                                 limit_den=np.array(dens, dtype=np.int64))
        ref = oracle.place_workload(ww, key_order=key_order, flags=flags)
        np.testing.assert_array_equal(got[0], ref[0])
        np.testing.assert_array_equal(got[1], ref[1])
    # nothing subscribed anywhere: limit 0, only g = 0 fits
    w = W.make_config(0)
    w.gpus_subscribed[:] = 0
    w.gpus_committed[:] = 0
    w.requests[0, :10, 0] = 0
    w.requests[0, :10, 1] = 0
    got = nb.place_workload(w, flags=nb.NBOS_LIMIT_CLUSTER_SR)
    assert (got[1][0, :10] == 3).all() and (got[1][0, 10:] == 0).all()


def test_scale_out_deficit(nb):
    import torch
    w = W.make_config(2, batch=50_001)
    hosts, found = nb.place_workload(w)
    d_found = torch.from_numpy(found).cuda()
    out = torch.full((1, 2), -5, dtype=torch.int64, device="cuda")
    nb.nbos_scale_out_deficit(d_found, 1, out)
    assert tuple(out.cpu().numpy()[0]) == oracle.scale_out_deficit(found[0])
    assert out[0, 0].item() > 0
    # many snapshots, ragged batch
    rng = np.random.default_rng(4)
    f = rng.integers(0, 4, size=(300, 1237)).astype(np.int32)
    out = torch.empty((300, 2), dtype=torch.int64, device="cuda")
    nb.nbos_scale_out_deficit(torch.from_numpy(f).cuda(), 300, out)
    got = out.cpu().numpy()
    for n in (0, 1, 150, 299):
        assert tuple(got[n]) == oracle.scale_out_deficit(f[n])
    assert got[:, 0].sum() == int((3 - f).sum())
    # empty batch
    out = torch.full((2, 2), 9, dtype=torch.int64, device="cuda")
    nb.nbos_scale_out_deficit(torch.empty((2, 0), dtype=torch.int32, device="cuda"), 2, out)
    assert (out == 0).all()
