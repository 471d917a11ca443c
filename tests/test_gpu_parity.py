"""GPU parity: the CUDA library, called through its C ABI, against the CPU checker, element by
element, on identical seeded inputs. Integer and index work: the bar is bit-exact."""
from __future__ import annotations

import dataclasses
import os

import numpy as np
import pytest

import oracle
from paper_2503_20591_b200 import workloads as W

pytestmark = pytest.mark.gpu

CPU_THREADS = max(1, min(32, (os.cpu_count() or 1)))


@pytest.fixture(scope="module")
def nb():
    import torch
    from paper_2503_20591_b200 import binding, build as lib_build
    lib_build.build()
    assert torch.cuda.is_available()
    binding.load_library()
    return binding


def both(nb, w, key_order=0, flags=0, config=None, lib_flags=0):
    got = nb.place_workload(w, key_order=key_order, flags=flags | lib_flags, config=config)
    ref = oracle.place_workload(w, key_order=key_order, flags=flags, threads=CPU_THREADS)
    return got, ref


def assert_same(got, ref, what=""):
    bad = np.nonzero((got[0] != ref[0]).any(axis=-1))
    assert bad[0].size == 0, (f"{what}: {bad[0].size} requests differ, first at "
                              f"{[int(b[0]) for b in bad]}: got {got[0][tuple(b[0] for b in bad)]}"
                              f" expected {ref[0][tuple(b[0] for b in bad)]}")
    np.testing.assert_array_equal(got[1], ref[1], err_msg=what)


# ---- the benchmark workloads ------------------------------------------------------------------
@pytest.mark.parametrize("index", [0, 1])
@pytest.mark.parametrize("key_order", [0, 1])
def test_small_configs_full(nb, index, key_order):
    w = W.make_config(index)
    got, ref = both(nb, w, key_order=key_order)
    assert_same(got, ref, w.name)


def test_config2_full(nb):
    w = W.make_config(2)
    got, ref = both(nb, w)
    assert_same(got, ref, w.name)
    assert (ref[1] < 3).any() and (ref[1] == 3).any()  # sentinel path and full path both hit
    check_properties(w, got[0], got[1])


def test_config4_full(nb):
    w = W.make_config(4)
    got, ref = both(nb, w)
    assert_same(got, ref, w.name)


def test_config3_full(nb):
    """Full-size launch (4,096 hosts x 1,048,576 requests, the shape the benchmark times), every
    request compared with the checker (which runs on all host cores here), plus the properties
    that hold at any size, checked without the checker."""
    w = W.make_config(3)
    hosts, found = nb.place_workload(w)
    ref = oracle.place_workload(w, threads=CPU_THREADS)
    assert_same((hosts, found), ref, "cfg3")
    check_properties(w, hosts, found)


def check_properties(w, hosts, found):
    """Invariants of a placement, from the inputs alone: ids in range, -1 only at the tail, three
    distinct hosts, every chosen host feasible, and no feasible host left out that ranks before
    the worst chosen one (or at all, when fewer than three were found)."""
    assert hosts.min() >= -1 and hosts.max() < w.n_hosts
    filled = hosts >= 0
    np.testing.assert_array_equal(found, filled.sum(axis=-1))
    assert (filled[..., :-1] >= filled[..., 1:]).all()          # -1 only at the tail
    rng = np.random.default_rng(5)
    for n in range(w.n_snapshots):
        h, req = hosts[n], w.requests[n].astype(np.int64)
        full = found[n] == 3
        assert ((h[full, 0] != h[full, 1]) & (h[full, 1] != h[full, 2]) & (h[full, 0] != h[full, 2])).all()
        G, S, C = (getattr(w, k)[n].astype(np.int64) for k in ("gpus_total", "gpus_subscribed", "gpus_committed"))
        num, den = int(w.limit_num[n]), int(w.limit_den[n])

        def fits(r, hk):
            return ((r[:, 0] <= G[hk]) & (r[:, 1] <= w.vram_gb[n][hk]) & (r[:, 2] <= w.millicpus[n][hk]) &
                    (r[:, 3] <= w.mem_mb[n][hk]) & ((S[hk] + r[:, 0]) * den <= num * G[hk] * w.replicas_R) &
                    (G[hk] >= 1) & (r.min(axis=1) >= 0))
        for k in range(3):
            sel = h[:, k] >= 0
            assert fits(req[sel], h[sel, k]).all()
        # a sample of requests against every host: nothing feasible ranks before the worst chosen
        ids = rng.choice(w.batch, size=min(512, w.batch), replace=False)
        for i in ids:
            r = req[i:i + 1]
            feas = fits(np.repeat(r, w.n_hosts, axis=0), np.arange(w.n_hosts))
            assert int(feas.sum()) >= int(found[n, i]) and (found[n, i] == 3 or int(feas.sum()) == found[n, i])
            if found[n, i] == 0:
                continue
            worst = h[i, found[n, i] - 1]
            # order: idle GPUs descending, (S + g) / G ascending (exact, cross-multiplied), id ascending
            idle = G - C
            g = int(r[0, 0])
            cand = np.nonzero(feas)[0]
            better = (idle[cand] > idle[worst]) | ((idle[cand] == idle[worst]) & (
                ((S[cand] + g) * G[worst] < (S[worst] + g) * G[cand]) |
                (((S[cand] + g) * G[worst] == (S[worst] + g) * G[cand]) & (cand < worst))))
            assert set(cand[better].tolist()) == set(h[i, :found[n, i] - 1].tolist())


# ---- every launch shape gives the same bytes --------------------------------------------------
SHAPES = [
    dict(lanes_per_request=1), dict(lanes_per_request=2), dict(lanes_per_request=4),
    dict(lanes_per_request=8), dict(lanes_per_request=16), dict(lanes_per_request=32),
    dict(lanes_per_request=1, requests_per_lane=1), dict(lanes_per_request=1, requests_per_lane=2),
    dict(lanes_per_request=4, requests_per_lane=4), dict(lanes_per_request=32, requests_per_lane=8),
    dict(lanes_per_request=1, tile_hosts=32), dict(lanes_per_request=8, tile_hosts=64),
    dict(lanes_per_request=32, tile_hosts=96, grid_blocks=3),
    dict(lanes_per_request=32, host_split=2, tile_hosts=64),
    dict(lanes_per_request=1, host_split=5, tile_hosts=32),
    dict(lanes_per_request=16, host_split=3, tile_hosts=128, grid_blocks=7),
    dict(lanes_per_request=1, grid_blocks=1),
]


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "-".join(f"{k[:5]}{v}" for k, v in s.items()))
def test_launch_shapes(nb, shape):
    cfg = nb.launch_config(**shape)
    for w in (W.make_config(2, batch=5000), W.mixed_gpu_cluster(777, 3001, seed=5)):
        got, ref = both(nb, w, config=cfg)
        assert_same(got, ref, f"{w.name} {shape}")


@pytest.mark.parametrize("lib_flags", [0, 2], ids=["key32", "key64"])
@pytest.mark.parametrize("key_order", [0, 1])
@pytest.mark.parametrize("flags", [0, 1], ids=["subscribe", "idle_now"])
def test_key_widths_orders_flags(nb, lib_flags, key_order, flags):
    for w in (W.mixed_gpu_cluster(1000, 4096, seed=11), W.make_config(2, batch=4096),
              W.make_config(4, batch=100, n_snapshots=24)):
        for shape in (dict(), dict(lanes_per_request=32, host_split=2, tile_hosts=128)):
            got, ref = both(nb, w, key_order=key_order, flags=flags, lib_flags=lib_flags,
                            config=nb.launch_config(**shape) if shape else None)
            assert_same(got, ref, f"{w.name} order={key_order} flags={flags} lib={lib_flags}")


@pytest.mark.parametrize("pair_mode", [0, 1, 2, 3, 4, 5])
@pytest.mark.parametrize("lanes", [0, 1, 4, 32])
def test_pair_evaluation_modes(nb, pair_mode, lanes):
    """Plain compares, packed test with the key computed or compared per pair, the key-order forms
    that retire requests, and the automatic choice (ranked form where available) give the same
    bytes."""
    cfg = nb.launch_config(lanes_per_request=lanes, pair_mode=pair_mode)
    for w in (W.make_config(2, batch=6000), W.mixed_gpu_cluster(900, 2500, seed=31),
              W.make_config(4, batch=80, n_snapshots=40), W.make_config(3, batch=3000)):
        for key_order in (0, 1):
            got, ref = both(nb, w, key_order=key_order, config=cfg)
            assert_same(got, ref, f"{w.name} pair_mode={pair_mode} lanes={lanes} order={key_order}")


def test_packed_test_layouts_and_fallback(nb):
    """The packed capacity test is used when the four capacities fit two 32-bit words: with one
    guard mask, with one mask per word, or not at all (plain compares). Same results each way."""
    w = W.make_config(1, batch=3000)
    s = nb.snapshot_from_workload(w)
    info = s.info()
    assert (info.packed_test, info.static_key, info.presorted) == (1, 1, 1)
    nb.nbos_snapshot_destroy(s)
    # memory capacity of exactly 2^20 MB needs 21 bits: 21 + 10 (VRAM) + 2 > 32 -> one mask per word
    w2 = W.make_config(1, batch=3000)
    w2.mem_mb[0, 7] = 1 << 20
    s = nb.snapshot_from_workload(w2)
    assert s.info().packed_test == 2
    nb.nbos_snapshot_destroy(s)
    got, ref = both(nb, w2)
    assert_same(got, ref, "two guard masks")
    # capacities far beyond 32 bits in total: plain compares
    w3 = W.make_config(1, batch=3000)
    w3.mem_mb[0, 9] = (1 << 31) - 1
    w3.millicpus[0, 11] = 1 << 30
    w3.requests[0, :100, 3] = (1 << 31) - 1
    w3.requests[0, 100:200, 2] = (1 << 30) - 5
    s = nb.snapshot_from_workload(w3)
    assert s.info().packed_test == 0
    nb.nbos_snapshot_destroy(s)
    got, ref = both(nb, w3)
    assert_same(got, ref, "plain compares")
    # mixed GPU counts: the key slope differs between hosts -> not static
    w4 = W.mixed_gpu_cluster(300, 2000, seed=8)
    s = nb.snapshot_from_workload(w4)
    assert s.info().static_key == 0
    nb.nbos_snapshot_destroy(s)
    # asks just above and at the largest capacity of each dimension
    w5 = W.make_config(1, batch=64)
    for k, arr in enumerate((w5.gpus_total, w5.vram_gb, w5.millicpus, w5.mem_mb)):
        top = int(arr.max())
        w5.requests[0, 2 * k] = [1, 16, 1000, 1024]
        w5.requests[0, 2 * k + 1] = [1, 16, 1000, 1024]
        w5.requests[0, 2 * k, k] = top
        w5.requests[0, 2 * k + 1, k] = top + 1
    got, ref = both(nb, w5)
    assert_same(got, ref, "asks at the capacity maxima")


def test_ranked_form_coarse_fields(nb):
    """Ranked form: capacities wider than their field lose low bits in the per-pair test, and a
    pair that passes it is re-tested exactly. Workloads built so that asks and capacities often
    fall into the same coarse bucket (the coarse test passes, the exact one may not), in every
    resource, with every launch shape; same bytes as the checker."""
    rng = np.random.default_rng(77)
    shapes = (dict(), dict(lanes_per_request=1), dict(lanes_per_request=4, requests_per_lane=2),
              dict(lanes_per_request=32, tile_hosts=64), dict(lanes_per_request=2, host_split=3, tile_hosts=64),
              dict(pair_mode=5), dict(pair_mode=5, lanes_per_request=8, tile_hosts=96))
    # (a) cfg3-like cluster: millicpus / memory capacities and asks crowd around the same values
    w = W.make_config(3, batch=4000)
    h = w.n_hosts
    w.millicpus[0, :] = 100_000 + rng.integers(0, 64, size=h)
    w.mem_mb[0, :] = 1_000_000 + rng.integers(0, 4096, size=h)
    w.requests[0, :, 2] = 100_000 + rng.integers(0, 64, size=w.batch)
    w.requests[0, :, 3] = 1_000_000 + rng.integers(0, 4096, size=w.batch)
    w.requests[0, :64, 3] = 1_000_000 + 4094      # only a handful of hosts have that much
    s = nb.snapshot_from_workload(w)
    info = s.info()
    nb.nbos_snapshot_destroy(s)
    assert info.ranked == 1 and info.static_key == 1 and info.presorted == 1
    assert info.ranked_dropped_bits[0] == 0          # the GPU component is always exact
    assert max(info.ranked_dropped_bits[1:]) > 0     # something is coarse at this size
    for shape in shapes:
        got, ref = both(nb, w, config=nb.launch_config(**shape) if shape else None)
        assert_same(got, ref, f"crowded capacities {shape}")
    assert (ref[1] == 3).any() and (ref[1] < 3).any()
    # (b) capacities near 2^31: most bits dropped
    w2 = W.make_config(1, batch=3000)
    w2.mem_mb[0, :] = (1 << 31) - 1 - rng.integers(0, 1 << 16, size=w2.n_hosts)
    w2.millicpus[0, :] = (1 << 30) + rng.integers(0, 1 << 12, size=w2.n_hosts)
    w2.requests[0, :, 3] = (1 << 31) - 1 - rng.integers(0, 1 << 16, size=w2.batch)
    w2.requests[0, :, 2] = (1 << 30) + rng.integers(0, 1 << 12, size=w2.batch)
    s = nb.snapshot_from_workload(w2)
    info = s.info()
    nb.nbos_snapshot_destroy(s)
    assert info.ranked == 1 and info.packed_test == 0 and min(info.ranked_dropped_bits[2:]) >= 8
    for shape in shapes:
        for key_order in (0, 1):
            got, ref = both(nb, w2, key_order=key_order, config=nb.launch_config(**shape) if shape else None)
            assert_same(got, ref, f"wide capacities {shape} order={key_order}")
    # (c) VRAM crowded too, idle reading, several snapshots with different limits
    w3 = W.make_config(4, batch=300, n_snapshots=12)
    w3.vram_gb[:, :] = 600 + rng.integers(0, 40, size=w3.vram_gb.shape)
    w3.requests[:, :, 1] = 600 + rng.integers(0, 40, size=w3.requests.shape[:2])
    for flags in (0, 1):
        got, ref = both(nb, w3, flags=flags)
        assert_same(got, ref, f"crowded VRAM flags={flags}")
    # (d) mixed GPU counts: hosts rank differently for different asks, but the same inside one GPU
    # count; the ranked form then works group by group (the groups are the host slices)
    s = nb.snapshot_from_workload(W.mixed_gpu_cluster(300, 100, seed=8))
    info = s.info()
    assert (info.ranked, info.grouped, info.static_key) == (1, 1, 0)
    nb.nbos_snapshot_destroy(s)


def test_tables_grouped_by_gpu_count(nb):
    """Hosts with different GPU counts (Section 3.4.1: 1 to 8 per server) rank differently for
    different asks. With at most 8 distinct counts per snapshot the table is stored count by
    count, each group in key order, and the kernel retires a request per group; with more counts
    it falls back to computing the key for every pair. Same bytes as the checker either way."""
    shapes = (dict(), dict(lanes_per_request=1), dict(lanes_per_request=4, requests_per_lane=2),
              dict(lanes_per_request=32), dict(lanes_per_request=8, tile_hosts=32),
              dict(lanes_per_request=2, host_split=3, tile_hosts=64))
    # many hosts; tiny groups that several hosts of one chunk straddle; one ask dimension scarce
    w_big = W.mixed_gpu_cluster(3000, 5000, seed=41)
    w_tiny = W.mixed_gpu_cluster(40, 3000, seed=42)
    w_scarce = W.mixed_gpu_cluster(1500, 4000, seed=43)
    w_scarce.millicpus[0, :] = np.minimum(w_scarce.millicpus[0, :], 4000)   # most asks exceed it
    w_two_masks = W.mixed_gpu_cluster(900, 3000, seed=44)
    w_two_masks.mem_mb[0, 5] = 1 << 20
    for w, packed in ((w_big, 1), (w_tiny, 1), (w_scarce, 1), (w_two_masks, 2)):
        s = nb.snapshot_from_workload(w)
        info = s.info()
        assert (info.static_key, info.grouped, info.packed_test) == (0, 1, packed), w.name
        nb.nbos_snapshot_destroy(s)
        for key_order in (0, 1):
            for flags in (0, 1):
                for shape in shapes:
                    got, ref = both(nb, w, key_order=key_order, flags=flags,
                                    config=nb.launch_config(**shape) if shape else None)
                    assert_same(got, ref, f"grouped {w.name} order={key_order} flags={flags} {shape}")
    # several snapshots with different sets of GPU counts in one launch
    parts = [W.mixed_gpu_cluster(500, 700, seed=50 + i) for i in range(3)]
    parts[1].gpus_total[0, :] = np.where(parts[1].gpus_total[0, :] > 4, 8, 2)
    parts[1].gpus_committed[0, :] = np.minimum(parts[1].gpus_committed[0, :], parts[1].gpus_total[0, :])
    multi = dataclasses.replace(
        parts[0], name="mixed_multi", n_snapshots=3,
        **{k: np.concatenate([getattr(q, k) for q in parts], axis=0)
           for k in W.Workload.HOST_FIELDS + ("limit_num", "limit_den", "requests")})
    got, ref = both(nb, multi)
    assert_same(got, ref, "grouped, three snapshots")
    # more than 8 distinct GPU counts: not grouped
    w_many = W.mixed_gpu_cluster(800, 3000, seed=45)
    rng = np.random.Generator(np.random.PCG64(45))
    w_many.gpus_total[0, :] = rng.integers(1, 13, size=800)
    w_many.gpus_committed[0, :] = np.minimum(w_many.gpus_committed[0, :], w_many.gpus_total[0, :])
    s = nb.snapshot_from_workload(w_many)
    assert (s.info().static_key, s.info().grouped) == (0, 0)
    nb.nbos_snapshot_destroy(s)
    got, ref = both(nb, w_many)
    assert_same(got, ref, "12 distinct GPU counts")


def test_first_fit_variant(nb):
    """Stopping at the third feasible host (table in key order, same key slope everywhere) gives
    the same bytes as the full evaluation; where the conditions do not hold the flag is ignored."""
    cfg = nb.launch_config(first_fit=1)
    for w in (W.make_config(0), W.make_config(1), W.make_config(2, batch=40_000),
              W.make_config(3, batch=20_000), W.make_config(4, batch=300, n_snapshots=64),
              W.uniform_cluster(9000, 500, seed=5), W.uniform_cluster(33, 7, seed=6),
              W.mixed_gpu_cluster(700, 3000, seed=7),          # not static: flag ignored
              W.uniform_cluster(70000, 40, seed=8)):           # not presorted: flag ignored
        for key_order in (0, 1):
            for lib_flags in (0, 2):
                got, ref = both(nb, w, key_order=key_order, config=cfg, lib_flags=lib_flags)
                assert_same(got, ref, f"first fit {w.name} order={key_order} lib={lib_flags}")
    w = W.make_config(2, batch=10_000)
    got, ref = both(nb, w, flags=1, config=cfg)
    assert_same(got, ref, "first fit, idle reading")
    w = W.make_config(1, batch=2000)
    w.mem_mb[0, 9] = (1 << 31) - 1                              # no packed table: plain compares
    w.requests[0, :50, 0] = -3
    got, ref = both(nb, w, config=cfg)
    assert_same(got, ref, "first fit, plain table")


def test_large_tables(nb):
    """Up to 65,536 hosts the table is stored in key order; beyond that it stays in host order.
    Results are the same either way."""
    w = W.uniform_cluster(9000, 600, seed=77)
    s = nb.snapshot_from_workload(w)
    assert s.info().presorted == 1
    nb.nbos_snapshot_destroy(s)
    for shape in (dict(), dict(lanes_per_request=1), dict(lanes_per_request=32, host_split=3)):
        got, ref = both(nb, w, config=nb.launch_config(**shape) if shape else None)
        assert_same(got, ref, f"9000 hosts {shape}")
    w = W.mixed_gpu_cluster(8200, 300, seed=78)
    got, ref = both(nb, w, key_order=1)
    assert_same(got, ref, "8200 mixed hosts")
    w = W.uniform_cluster(70000, 48, seed=79)
    s = nb.snapshot_from_workload(w)
    assert s.info().presorted == 0
    nb.nbos_snapshot_destroy(s)
    for shape in (dict(), dict(lanes_per_request=1)):
        got, ref = both(nb, w, config=nb.launch_config(**shape) if shape else None)
        assert_same(got, ref, f"70000 hosts {shape}")


def test_maximum_table_sizes(nb):
    """The largest table stored in key order (65,536 hosts: the position count is quadratic) and
    the largest table the library takes (2^20 hosts, host order, 64-bit keys)."""
    w = W.uniform_cluster(65_536, 96, seed=81)
    s = nb.snapshot_from_workload(w)
    assert s.info().presorted == 1
    nb.nbos_snapshot_destroy(s)
    got, ref = both(nb, w)
    assert_same(got, ref, "65,536 hosts")
    w = W.mixed_gpu_cluster(65_536, 40, seed=82)
    got, ref = both(nb, w)
    assert_same(got, ref, "65,536 mixed hosts")
    w = W.uniform_cluster(nb.NBOS_MAX_HOSTS, 24, seed=83)
    got, ref = both(nb, w)
    assert_same(got, ref, "2^20 hosts")
    assert (ref[1] == 3).all()
    w = W.mixed_gpu_cluster(nb.NBOS_MAX_HOSTS, 12, seed=84)
    got, ref = both(nb, w, key_order=1)
    assert_same(got, ref, "2^20 mixed hosts, SR first")


def test_key_width_is_chosen_from_the_data(nb):
    w = W.make_config(1)
    s = nb.snapshot_from_workload(w)
    info = s.info()
    assert (info.key_bits, info.bits_id, info.hosts_padded) == (32, 8, 256)
    assert info.bits_idle == 4 and info.bits_sr == 5
    nb.nbos_snapshot_destroy(s)
    s = nb.snapshot_from_workload(w, flags=nb.NBOS_FORCE_KEY64)
    assert s.info().key_bits == 64
    nb.nbos_snapshot_destroy(s)
    # a huge subscription count on a host that can still take requests needs more than 31 bits
    big = W.make_config(0)
    big.gpus_subscribed[0, 3] = 1 << 27
    big.limit_num[0], big.limit_den[0] = 1 << 26, 1
    s = nb.snapshot_from_workload(big)
    assert s.info().key_bits == 64
    nb.nbos_snapshot_destroy(s)
    got, ref = both(nb, big)
    assert_same(got, ref, "wide key")


# ---- edge cases -------------------------------------------------------------------------------
@pytest.mark.parametrize("n_hosts", [1, 2, 3, 31, 33, 100, 1025])
@pytest.mark.parametrize("batch", [1, 7, 300])
def test_ragged_sizes(nb, n_hosts, batch):
    w = W.uniform_cluster(n_hosts, batch, seed=n_hosts * 1000 + batch)
    got, ref = both(nb, w)
    assert_same(got, ref, f"H={n_hosts} B={batch}")
    w = W.mixed_gpu_cluster(n_hosts, batch, seed=n_hosts + batch)
    got, ref = both(nb, w, key_order=1)
    assert_same(got, ref, f"mixed H={n_hosts} B={batch}")


def test_multi_snapshot_ragged(nb):
    w = W.what_if_sweep(13, 70, 333)
    for shape in (dict(), dict(lanes_per_request=1, grid_blocks=5),
                  dict(lanes_per_request=8, host_split=2, tile_hosts=32)):
        got, ref = both(nb, w, config=nb.launch_config(**shape) if shape else None)
        assert_same(got, ref, f"sweep {shape}")


def test_negative_and_zero_requests(nb):
    w = W.make_config(1, batch=64)
    w.requests[0, 0] = [-1, 16, 1000, 1024]
    w.requests[0, 1] = [1, -16, 1000, 1024]
    w.requests[0, 2] = [1, 16, -1000, 1024]
    w.requests[0, 3] = [1, 16, 1000, -1024]
    w.requests[0, 4] = [0, 0, 0, 0]
    w.requests[0, 5] = [np.iinfo(np.int32).max] * 4
    w.requests[0, 6] = [np.iinfo(np.int32).min] * 4
    got, ref = both(nb, w)
    assert_same(got, ref, "odd requests")
    assert (got[0][0, :4] == -1).all() and (got[1][0, :4] == 0).all()
    assert got[1][0, 4] == 3


def test_hosts_without_gpus_and_saturated_hosts(nb):
    w = W.make_config(1, batch=256)
    w.gpus_total[0, ::3] = 0
    w.gpus_committed[0, ::3] = 0
    w.gpus_subscribed[0, 1::3] = 1000
    w.requests[0, :32, 0] = 0
    w.requests[0, :32, 1] = 0
    got, ref = both(nb, w)
    assert_same(got, ref, "no-GPU hosts")


def test_nothing_feasible_anywhere(nb):
    w = W.make_config(0)
    w.limit_num[0] = 0
    got, ref = both(nb, w)
    assert_same(got, ref, "limit 0")
    assert (got[0] == -1).all() and (got[1] == 0).all()


def test_empty_batch_and_optional_found(nb):
    import torch
    w = W.make_config(0)
    s = nb.snapshot_from_workload(w)
    empty = torch.empty((1, 0, 4), dtype=torch.int32, device="cuda")
    out = torch.empty((1, 0, 3), dtype=torch.int32, device="cuda")
    nb.nbos_place_batch(s, empty, out)
    req = torch.from_numpy(w.requests).cuda()
    out = torch.full((1, w.batch, 3), -7, dtype=torch.int32, device="cuda")
    nb.nbos_place_batch(s, req, out, None)
    assert nb.nbos_snapshot_status(s) == nb.NBOS_OK
    ref = oracle.place_workload(w)
    np.testing.assert_array_equal(out.cpu().numpy(), ref[0])
    nb.nbos_snapshot_destroy(s)


def test_host_buffer_entry_points(nb):
    import torch
    w = W.make_config(4, batch=257, n_snapshots=5)
    arrays = [torch.from_numpy(getattr(w, k)).reshape(-1) for k in w.HOST_FIELDS]
    s = nb.nbos_snapshot_create_host(w.n_snapshots, w.n_hosts, torch.from_numpy(w.limit_num),
                                     torch.from_numpy(w.limit_den), *arrays)
    ref = oracle.place_workload(w)
    for pinned in (False, True):
        req = torch.from_numpy(w.requests.copy())
        out = torch.empty((w.n_snapshots, w.batch, 3), dtype=torch.int32)
        found = torch.empty((w.n_snapshots, w.batch), dtype=torch.int32)
        if pinned:
            req, out, found = req.pin_memory(), out.pin_memory(), found.pin_memory()
        nb.nbos_place_batch_host(s, req, out, found)
        np.testing.assert_array_equal(out.numpy(), ref[0])
        np.testing.assert_array_equal(found.numpy(), ref[1])
    nb.nbos_snapshot_destroy(s)


def test_asynchronous_host_calls_in_a_row(nb):
    """Six calls queued without waiting, batches of different sizes (the two staging sets grow and
    are reused; the large ones go through in two chunks), a snapshot refresh between two of them,
    pinned and pageable buffers; every call's results are checked after one wait at the end."""
    import torch
    stream = torch.cuda.Stream()
    w = W.make_config(2, batch=2_200_000)
    ref = oracle.place_workload(w, threads=CPU_THREADS)
    lim = (torch.from_numpy(w.limit_num), torch.from_numpy(w.limit_den))
    arrays = [torch.from_numpy(getattr(w, k)).reshape(-1).pin_memory() for k in w.HOST_FIELDS]
    s = nb.nbos_snapshot_create_host(w.n_snapshots, w.n_hosts, *lim, *arrays, stream=stream)
    sizes = [2_199_000, 5, 1_100_000, 2_200_000, 64, 2_100_001]
    calls = []
    for i, b in enumerate(sizes):
        lo = 0 if b == w.batch else 7 * i
        req = torch.from_numpy(np.ascontiguousarray(w.requests[:, lo: lo + b])).clone()
        out = torch.full((1, b, 3), -9, dtype=torch.int32)
        found = torch.full((1, b), -9, dtype=torch.int32)
        if i != 4:
            req, out, found = req.pin_memory(), out.pin_memory(), found.pin_memory()
        if i == 3:
            nb.nbos_snapshot_update_host(s, *lim, *arrays, stream=stream)
        nb.nbos_place_batch_host_async(s, req, out, found if i % 2 == 0 else None, stream=stream)
        calls.append((i, lo, b, req, out, found))
    nb.nbos_place_batch_host_wait(s)
    assert nb.nbos_snapshot_status(s) == nb.NBOS_OK
    for i, lo, b, req, out, found in calls:
        np.testing.assert_array_equal(out.numpy()[0], ref[0][0, lo: lo + b], err_msg=f"call {i}")
        if i % 2 == 0:
            np.testing.assert_array_equal(found.numpy()[0], ref[1][0, lo: lo + b], err_msg=f"call {i}")
    # the blocking form takes its turn among them
    req = torch.from_numpy(np.ascontiguousarray(w.requests[:, :1000])).pin_memory()
    out = torch.empty((1, 1000, 3), dtype=torch.int32).pin_memory()
    nb.nbos_place_batch_host(s, req, out, stream=stream)
    np.testing.assert_array_equal(out.numpy()[0], ref[0][0, :1000])
    nb.nbos_snapshot_destroy(s)


@pytest.mark.parametrize("seed", range(8))
def test_random_sequences_of_host_calls(nb, seed):
    """Refreshes from three different states, asynchronous and blocking placements of random sizes
    and waits, in random order on one stream; every placement is checked against the state that
    was current when it was queued."""
    import torch
    rng = np.random.default_rng(seed)
    hosts, pool = int(rng.choice([33, 700, 1024])), int(rng.choice([5000, 120_000]))
    states = [W.uniform_cluster(hosts, pool, seed=seed * 7 + k) for k in range(3)]
    w0 = states[0]
    stream = torch.cuda.Stream() if seed % 2 else torch.cuda.current_stream()

    def pin(a):
        return torch.from_numpy(np.ascontiguousarray(a)).pin_memory()

    lim = (torch.from_numpy(w0.limit_num), torch.from_numpy(w0.limit_den))
    arrs = [[pin(getattr(s, k).reshape(-1)) for k in s.HOST_FIELDS] for s in states]
    snap = nb.nbos_snapshot_create_host(1, hosts, *lim, *arrs[0], stream=stream)
    cur, pending = 0, []

    def check_all():
        for si, lo, b, req, out, found in pending:
            s = states[si]
            ref = oracle.place(*[getattr(s, k)[0] for k in s.HOST_FIELDS], int(s.limit_num[0]), int(s.limit_den[0]),
                               w0.requests[0, lo:lo + b], replicas_R=s.replicas_R)
            np.testing.assert_array_equal(out.numpy()[0], ref[0], err_msg=f"state {si}, requests {lo}..{lo + b}")
            np.testing.assert_array_equal(found.numpy()[0], ref[1])
        pending.clear()

    for _ in range(int(rng.integers(6, 14))):
        op = rng.choice(["update", "async", "async", "async", "block", "wait"])
        if op == "update":
            cur = int(rng.integers(0, 3))
            nb.nbos_snapshot_update_host(snap, *lim, *arrs[cur], stream=stream)
        elif op == "wait":
            nb.nbos_place_batch_host_wait(snap)
            check_all()
        else:
            b = int(rng.choice([1, 31, 1000, 4097]))
            lo = int(rng.integers(0, pool - b + 1))
            req = pin(w0.requests[:, lo:lo + b]) if rng.random() < 0.8 else torch.from_numpy(np.ascontiguousarray(w0.requests[:, lo:lo + b]))
            out, found = torch.full((1, b, 3), -9, dtype=torch.int32), torch.full((1, b), -9, dtype=torch.int32)
            if rng.random() < 0.8:
                out, found = out.pin_memory(), found.pin_memory()
            if op == "async":
                nb.nbos_place_batch_host_async(snap, req, out, found, stream=stream)
                pending.append((cur, lo, b, req, out, found))
            else:
                nb.nbos_place_batch_host(snap, req, out, found, stream=stream)
                pending.append((cur, lo, b, req, out, found))
                check_all()
    nb.nbos_place_batch_host_wait(snap)
    check_all()
    assert nb.nbos_snapshot_status(snap) == nb.NBOS_OK
    torch.cuda.synchronize()
    nb.nbos_snapshot_destroy(snap)


def test_create_rejects_bad_values(nb):
    import torch
    w = W.make_config(0)

    def create(mod):
        ww = W.make_config(0)
        mod(ww)
        return nb.snapshot_from_workload(ww)

    for mod, code in ((lambda x: x.gpus_subscribed.__setitem__((0, 5), -1), nb.NBOS_ERR_RANGE),
                      (lambda x: x.gpus_committed.__setitem__((0, 5), 9), nb.NBOS_ERR_RANGE),
                      (lambda x: x.gpus_total.__setitem__((0, 5), 5000), nb.NBOS_ERR_RANGE),
                      (lambda x: x.mem_mb.__setitem__((0, 31), -5), nb.NBOS_ERR_RANGE),
                      (lambda x: x.limit_den.__setitem__(0, 0), nb.NBOS_ERR_INVALID_ARG),
                      (lambda x: x.limit_num.__setitem__(0, -1), nb.NBOS_ERR_INVALID_ARG)):
        with pytest.raises(nb.NbosError) as e:
            create(mod)
        assert e.value.status == code
    # the context is fine afterwards
    got, ref = both(nb, w)
    assert_same(got, ref)
    # workspace too small / misaligned
    dev = [torch.from_numpy(getattr(w, k)).cuda().reshape(-1) for k in w.HOST_FIELDS]
    with pytest.raises(nb.NbosError) as e:
        nb.nbos_snapshot_create(1, 32, torch.from_numpy(w.limit_num), torch.from_numpy(w.limit_den),
                                *dev, workspace=torch.empty(512, dtype=torch.uint8, device="cuda"))
    assert e.value.status == nb.NBOS_ERR_NO_MEMORY


def test_streams_and_repeated_calls(nb):
    import torch
    w = W.make_config(2, batch=20000)
    ref = oracle.place_workload(w, threads=CPU_THREADS)
    s = nb.snapshot_from_workload(w)
    req = torch.from_numpy(w.requests).cuda()
    streams = [torch.cuda.Stream() for _ in range(3)]
    outs = [torch.empty((1, w.batch, 3), dtype=torch.int32, device="cuda") for _ in streams]
    torch.cuda.synchronize()
    for rep in range(3):
        for st, out in zip(streams, outs):
            nb.nbos_place_batch(s, req, out, None, stream=st)
    torch.cuda.synchronize()
    assert nb.nbos_snapshot_status(s) == nb.NBOS_OK
    for out in outs:
        np.testing.assert_array_equal(out.cpu().numpy(), ref[0])
    nb.nbos_snapshot_destroy(s)


def test_bounded_wait_gives_up_and_context_survives(nb):
    """A wait that nothing will ever satisfy must end by itself, be reported, and leave the
    device usable (no trap, no hang). The self-test runs the placement kernel's own wait function:
    one warp's wait runs out, the other leaves through the block's abort flag."""
    gave_up, ms = nb.nbos_probe_wait_timeout(20_000_000)   # 20 ms
    assert gave_up == 3                                     # both warps came back empty-handed
    assert 15.0 < ms < 2000.0
    w = W.make_config(0)
    got, ref = both(nb, w)
    assert_same(got, ref)


def test_a_wait_that_ran_out_is_reported_by_the_snapshot_and_survives_an_update(nb):
    """The status word a placement kernel raises when it gives up on a wait reaches the caller as
    NBOS_ERR_DEVICE_TIMEOUT, and a later refresh of the snapshot does not wipe it."""
    import torch
    w = W.make_config(1, batch=256)
    dev = [torch.from_numpy(getattr(w, k)).cuda().reshape(-1) for k in w.HOST_FIELDS]
    lim = (torch.from_numpy(w.limit_num), torch.from_numpy(w.limit_den))
    s = nb.nbos_snapshot_create(w.n_snapshots, w.n_hosts, *lim, *dev)
    try:
        assert nb.nbos_snapshot_status(s) == nb.NBOS_OK
        ms = nb.nbos_probe_wait_timeout_on_snapshot(s, 5_000_000)    # 5 ms
        assert 3.0 < ms < 2000.0
        assert nb.nbos_snapshot_status(s) == nb.NBOS_ERR_DEVICE_TIMEOUT
        nb.nbos_snapshot_update(s, *lim, *dev)
        assert nb.nbos_snapshot_status(s) == nb.NBOS_ERR_DEVICE_TIMEOUT
        # the device itself is fine: a placement on a fresh snapshot is exact
        got, ref = both(nb, w)
        assert_same(got, ref)
    finally:
        nb.nbos_snapshot_destroy(s)
    # what an update reports is cleared by the next good update
    s = nb.nbos_snapshot_create(w.n_snapshots, w.n_hosts, *lim, *dev)
    try:
        bad = [d.clone() for d in dev]
        bad[1][3] = -5                                               # a negative subscribed count
        nb.nbos_snapshot_update(s, *lim, *bad)
        assert nb.nbos_snapshot_status(s) == nb.NBOS_ERR_RANGE
        nb.nbos_snapshot_update(s, *lim, *dev)
        assert nb.nbos_snapshot_status(s) == nb.NBOS_OK
    finally:
        nb.nbos_snapshot_destroy(s)
