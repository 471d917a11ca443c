"""GPU parity for executor selection (Section 3.2.2) and the execute -> migrate flow
(Section 3.2.3), against the CPU checker, bit-exact."""
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


def draw_kernels(rng, w, m):
    """m kernels with three distinct replica hosts each and a cell that asks for idle resources."""
    h = w.n_hosts
    rep = np.stack([rng.choice(h, size=3, replace=False) for _ in range(m)]).astype(np.int32)
    g = rng.integers(0, 9, size=m)
    req = np.stack([g, 16 * g, rng.integers(1000, 16001, size=m), rng.integers(1024, 65537, size=m)],
                   axis=1).astype(np.int32)
    return req, rep


def gpu_select(nb, w, req, rep):
    import torch
    dev = [torch.from_numpy(getattr(w, k)[0]).cuda() for k in w.HOST_FIELDS]
    ex = torch.full((req.shape[0],), -9, dtype=torch.int32, device="cuda")
    mask = torch.full((req.shape[0],), -9, dtype=torch.int32, device="cuda")
    nb.nbos_select_executors(*dev, torch.from_numpy(req).cuda(), torch.from_numpy(rep).cuda(), ex, mask,
                             replicas_R=w.replicas_R)
    torch.cuda.synchronize()
    return ex.cpu().numpy(), mask.cpu().numpy()


def cpu_select(w, req, rep):
    return oracle.select_executors(*[getattr(w, k)[0] for k in w.HOST_FIELDS], req, rep,
                                   replicas_R=w.replicas_R)


@pytest.mark.parametrize("maker", [lambda: W.make_config(1), lambda: W.make_config(2),
                                   lambda: W.mixed_gpu_cluster(500, 16, seed=5),
                                   lambda: W.uniform_cluster(3, 16, seed=6)])
@pytest.mark.parametrize("m", [1, 1000, 300_001, 1_300_003])
def test_executor_selection_matches_the_checker(nb, maker, m):
    w = maker()
    rng = np.random.default_rng(m)
    req, rep = draw_kernels(rng, w, m)
    rep[rng.random(m) < 0.03, rng.integers(0, 3)] = -1          # missing replicas
    req[rng.random(m) < 0.01, 0] = -1                           # nonsense asks
    if m > 10:
        rep[5] = [0, 0, 0]                                       # degenerate: same host three times
        rep[6] = [w.n_hosts, -5, 1 << 30]                        # out-of-range ids are "no replica"
    got = gpu_select(nb, w, req, rep)
    ref = cpu_select(w, req, rep)
    np.testing.assert_array_equal(got[0], ref[0])
    np.testing.assert_array_equal(got[1], ref[1])
    if m >= 1000:
        assert (ref[0] >= 0).any()


def select_both(nb, state, req, rep):
    import torch
    dev = [torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).cuda() for a in state]
    ex = torch.full((req.shape[0],), -9, dtype=torch.int32, device="cuda")
    mask = torch.full((req.shape[0],), -9, dtype=torch.int32, device="cuda")
    nb.nbos_select_executors(*dev, torch.from_numpy(req).cuda(), torch.from_numpy(rep).cuda(), ex, mask)
    torch.cuda.synchronize()
    ref = oracle.select_executors(*[np.ascontiguousarray(a, dtype=np.int32) for a in state], req, rep)
    np.testing.assert_array_equal(mask.cpu().numpy(), ref[1])
    np.testing.assert_array_equal(ex.cpu().numpy(), ref[0])
    return ref


def crowded_state(rng, hosts, g_max=8):
    """Few distinct values per component, so that replicas tie on idle GPUs and on S / G (also with
    different G: 2/4 against 4/8), some hosts without GPUs or with a negative component."""
    G = rng.integers(1, g_max + 1, size=hosts)
    C = rng.integers(0, G + 1)
    S = G * rng.integers(0, 4, size=hosts) // rng.integers(1, 3, size=hosts)
    AV = 16 * (G - C)
    AC = rng.choice([0, 4000, 16000, 64000], size=hosts)
    AM = rng.choice([0, 2048, 65536, 1 << 20], size=hosts)
    dead = rng.random(hosts) < 0.05
    G = np.where(dead, 0, G)
    AC = np.where(rng.random(hosts) < 0.02, -1, AC)
    C = np.where(rng.random(hosts) < 0.02, G + 1, C)          # more committed than there are: idle < 0
    return [G, S, C, AV, AC, AM]


def edge_asks(rng, m, hosts):
    g = rng.integers(0, 9, size=m)
    req = np.stack([g, 16 * g, rng.choice([0, 1000, 4000, 4001, 16000], size=m),
                    rng.choice([0, 1024, 2048, 2049, 65536, 1 << 20], size=m)], axis=1).astype(np.int32)
    # asks at and beyond what the packed fields hold, and negative ones
    odd = [[14, 0, 0, 0], [15, 0, 0, 0], [16, 0, 0, 0], [1 << 30, 0, 0, 0], [0, 2047, 0, 0], [0, 2048, 0, 0],
           [0, 1 << 20, 0, 0], [0, 0, (1 << 19) - 1, 0], [0, 0, 1 << 19, 0], [0, 0, 1 << 30, 0],
           [0, 0, 0, (1 << 26) - 1], [0, 0, 0, 1 << 26], [0, 0, 0, (1 << 31) - 1], [-1, 0, 0, 0], [0, -1, 0, 0],
           [0, 0, -1, 0], [0, 0, 0, -1], [0, 0, 0, 0], [-(1 << 31), 0, 0, 0]]
    req[: len(odd)] = np.array(odd, dtype=np.int64).astype(np.int32)
    rep = rng.integers(0, hosts, size=(m, 3)).astype(np.int32)
    rep[rng.random(m) < 0.05, rng.integers(0, 3)] = -1
    rep[rng.random(m) < 0.02, rng.integers(0, 3)] = hosts
    return req, rep


@pytest.mark.parametrize("hosts,m", [(7, 3000), (300, 40_000), (300, 1_000_003), (4096, 2_500_000), (4096, 10_000_002),
                                     (4300, 11_000_000), (5000, 700_000), (7000, 400_000), (40_000, 300_000), (1 << 20, 600_000)])
def test_ties_dead_hosts_and_edge_asks(nb, hosts, m):
    """Packed 8-byte host records, tables in shared memory (many kernels per host: inputs through
    the ring of bulk copies, whole tiles and a partial last one) and in global memory (few kernels,
    or more hosts than shared memory holds)."""
    rng = np.random.default_rng(hosts)
    state = crowded_state(rng, hosts)
    req, rep = edge_asks(rng, m, hosts)
    ref = select_both(nb, state, req, rep)
    assert (ref[0] >= 0).any() and (ref[0] < 0).any()
    several = np.array([bin(x).count("1") for x in ref[1][:5000]]) >= 2
    assert several.any()


def test_host_ids_not_16_byte_aligned(nb):
    """A large batch whose host-id array starts 12 bytes into an allocation: no bulk copies, plain loads."""
    import torch
    rng = np.random.default_rng(77)
    hosts, m = 1000, 800_000
    state = crowded_state(rng, hosts)
    req, rep = edge_asks(rng, m + 1, hosts)
    dev = [torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).cuda() for a in state]
    rep_dev = torch.from_numpy(rep).cuda()[1:]
    assert rep_dev.data_ptr() % 16 == 12
    ex = torch.full((m,), -9, dtype=torch.int32, device="cuda")
    mask = torch.full((m,), -9, dtype=torch.int32, device="cuda")
    nb.nbos_select_executors(*dev, torch.from_numpy(req[1:]).cuda(), rep_dev, ex, mask)
    torch.cuda.synchronize()
    ref = oracle.select_executors(*[np.ascontiguousarray(a, dtype=np.int32) for a in state], req[1:], rep[1:])
    np.testing.assert_array_equal(mask.cpu().numpy(), ref[1])
    np.testing.assert_array_equal(ex.cpu().numpy(), ref[0])


@pytest.mark.parametrize("what", ["gpus", "memory", "cpu", "vram", "subscribed", "idle", "last_host_only"])
def test_cluster_states_the_packed_form_cannot_hold(nb, what):
    """One host (or all) beyond a packed field's range: the general form decides, same answers."""
    rng = np.random.default_rng(len(what))
    hosts, m = 3000, 700_000
    state = crowded_state(rng, hosts)
    G, S, C, AV, AC, AM = state
    if what == "gpus":
        G[:] = np.where(G > 0, 2 * G, 0); C[:] = np.minimum(C, G)
    elif what == "memory":
        AM[17] = (1 << 26); G[17], C[17] = 8, 0
    elif what == "cpu":
        AC[2999] = 1 << 19; G[2999], C[2999] = 8, 0
    elif what == "vram":
        AV[1000] = 1 << 11; G[1000], C[1000] = 8, 0
    elif what == "subscribed":
        S[5] = 1 << 22; G[5], C[5] = 8, 0
    elif what == "idle":
        G[44], C[44] = 15, 0                                 # 15 idle GPUs: one more than the field holds
    elif what == "last_host_only":
        G[hosts - 1], C[hosts - 1], AM[hosts - 1] = 8, 0, (1 << 31) - 1
    req, rep = edge_asks(rng, m, hosts)
    rep[100:200, 0] = [17, 2999, 1000, 5, 44, hosts - 1, 0, 1, 2, 3] * 10
    req[100:200] = [0, 0, 0, 0]
    select_both(nb, state, req, rep)


def test_execute_then_migrate_flow(nb):
    """Kernels whose three replicas must all yield get a migration target: the best host of the
    idle-resources placement (first column). That target is never one of the yielding hosts."""
    import torch
    w = W.make_config(2)                     # heavily loaded cluster: many failed elections
    rng = np.random.default_rng(3)
    m = 50_000
    req, rep = draw_kernels(rng, w, m)
    ex, mask = gpu_select(nb, w, req, rep)
    ref_ex, ref_mask = cpu_select(w, req, rep)
    np.testing.assert_array_equal(ex, ref_ex)
    failed = np.nonzero(ex < 0)[0]
    assert failed.size > 100 and failed.size < m
    # migration targets for the failed elections
    snap = nb.snapshot_from_workload(w, flags=nb.NBOS_REQUIRE_IDLE_GPUS)
    mig_req = np.ascontiguousarray(req[failed])[None]
    out = torch.empty((1, failed.size, 3), dtype=torch.int32, device="cuda")
    found = torch.empty((1, failed.size), dtype=torch.int32, device="cuda")
    nb.nbos_place_batch(snap, torch.from_numpy(mig_req).cuda(), out, found)
    assert nb.nbos_snapshot_status(snap) == nb.NBOS_OK
    nb.nbos_snapshot_destroy(snap)
    target = out.cpu().numpy()[0, :, 0]
    ref_hosts, _ = oracle.place(*[getattr(w, k)[0] for k in w.HOST_FIELDS], int(w.limit_num[0]),
                                int(w.limit_den[0]), mig_req[0], replicas_R=w.replicas_R,
                                flags=oracle.REQUIRE_IDLE_GPUS)
    np.testing.assert_array_equal(target, ref_hosts[:, 0])
    has_target = target >= 0
    assert has_target.any()
    # a host that made its replica yield cannot be the target (it lacks the idle resources)
    assert not (target[has_target, None] == rep[failed][has_target]).any()


def test_argument_errors(nb):
    import torch
    w = W.make_config(0)
    dev = [torch.from_numpy(getattr(w, k)[0]).cuda() for k in w.HOST_FIELDS]
    req = torch.zeros((4, 4), dtype=torch.int32, device="cuda")
    rep = torch.zeros((4, 3), dtype=torch.int32, device="cuda")
    out = torch.zeros((4,), dtype=torch.int32, device="cuda")
    with pytest.raises(ValueError):
        nb.nbos_select_executors(*dev, req, rep[:3], out, out)
    with pytest.raises(nb.NbosError) as e:
        nb.nbos_select_executors(*dev, req, rep, out, out, replicas_R=0)
    assert e.value.status == nb.NBOS_ERR_INVALID_ARG
    nb.nbos_select_executors(*dev, req[:0], rep[:0], out[:0], out[:0])   # empty batch is a no-op
