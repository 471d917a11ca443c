"""Pins for the CPU checker's cluster-wide quantities (Sections 3.4.1 third factor, 3.4.2,
3.2.1): worked examples, library sums, and the dynamic limit's effect on placement."""
from fractions import Fraction

import numpy as np

import oracle
from paper_2503_20591_b200 import workloads as W

AMPLE = (640, 128000, 1048576)


def test_sums_match_numpy():
    for w in (W.make_config(1), W.make_config(2), W.mixed_gpu_cluster(333, 4, seed=2)):
        G, S, C = w.gpus_total[0], w.gpus_subscribed[0], w.gpus_committed[0]
        assert oracle.cluster_sums(G, S, C) == (int(G.sum()), int(S.sum()), int(C.sum()))
        num, den = oracle.cluster_limit(G, S, C, replicas_R=3)
        assert Fraction(num, den) == Fraction(int(S.sum()), int(G.sum()) * 3)


def test_dynamic_limit_worked_example():
    """Two 8-GPU servers with S = 16 and S = 8: sum S = 24, sum G = 16, R = 3 -> limit 24/48 = 1/2.
    Server 0 sits at 16/24 = 2/3 > 1/2: rejected for every ask. Server 1 at 8/24: it may grow to
    (8+g)/24 <= 1/2, i.e. g <= 4."""
    G, S, C = np.array([8, 8]), np.array([16, 8]), np.array([0, 0])
    num, den = oracle.cluster_limit(G, S, C)
    assert (num, den) == (24, 48)
    ample = [np.full(2, x) for x in AMPLE]
    req = np.array([[g, 16 * g, 1000, 1024] for g in (0, 1, 4, 5)], dtype=np.int32)
    hosts, found = oracle.place(G, S, C, *ample, num, den, req)
    assert hosts.tolist() == [[1, -1, -1], [1, -1, -1], [1, -1, -1], [-1, -1, -1]]
    assert found.tolist() == [1, 1, 1, 0]
    # an empty cluster (nothing subscribed) has limit 0: only g = 0 fits
    num, den = oracle.cluster_limit(G, np.array([0, 0]), C)
    assert num == 0
    _, found = oracle.place(G, np.array([0, 0]), C, *ample, num, den, req)
    assert found.tolist() == [2, 0, 0, 0]


def test_servers_above_the_cluster_average_are_rejected():
    """With the dynamic limit a server whose SR is above the cluster-wide SR takes nothing with
    g >= 1, whatever else it has; at least one server is at or below the average."""
    w = W.make_config(1, batch=200)
    G, S, C = (x[0].astype(np.int64) for x in (w.gpus_total, w.gpus_subscribed, w.gpus_committed))
    num, den = oracle.cluster_limit(G, S, C)
    hosts, found = oracle.place(G, S, C, w.vram_gb[0], w.millicpus[0], w.mem_mb[0], num, den,
                                w.requests[0])
    avg = Fraction(num, den)
    chosen = hosts[hosts >= 0]
    reqg = np.repeat(w.requests[0][:, 0], 3).reshape(-1, 3)[hosts >= 0]
    for h, g in zip(chosen, reqg):
        assert Fraction(int(S[h] + g), int(G[h]) * 3) <= avg
    assert (found > 0).any()


def test_autoscaler_rule():
    """f = 1.05 = 21/20 (Section 3.4.2). 100 GPUs in use -> expected capacity 105."""
    assert oracle.autoscale(104, 100) == 1      # 104 < 105: scale out
    assert oracle.autoscale(105, 100) == 0
    assert oracle.autoscale(106, 100) == -1     # more provisioned than expected: may release
    assert oracle.autoscale(0, 0) == 0
    assert oracle.autoscale(240, 0) == -1       # idle cluster
    assert oracle.autoscale(240, 240) == 1      # everything in use: 252 expected
    assert oracle.autoscale(21, 20) == 0 and oracle.autoscale(20, 20) == 1
    assert oracle.autoscale(100, 100, 1, 1) == 0
    for G in range(0, 60):
        for C in range(0, 60):
            want = (Fraction(21, 20) * C > G) - (Fraction(21, 20) * C < G)
            assert oracle.autoscale(G, C) == want


def test_scale_out_deficit():
    assert oracle.scale_out_deficit(np.array([3, 3, 3])) == (0, 0)
    assert oracle.scale_out_deficit(np.array([0, 1, 2, 3])) == (6, 3)
    assert oracle.scale_out_deficit(np.zeros(0, dtype=np.int32)) == (0, 0)
    w = W.make_config(2, batch=4000)
    _, found = oracle.place_workload(w)
    d, n = oracle.scale_out_deficit(found[0])
    assert d == int((3 - found[0]).sum()) and n == int((found[0] < 3).sum()) and n > 0
