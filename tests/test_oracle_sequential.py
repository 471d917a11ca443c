"""Pins for the CPU checker's sequential placement (each placed kernel subscribes its GPUs before
the next one is placed): a hand-worked run, a closed form, a pure-Python re-implementation on
exact fractions, and relations to the frozen-snapshot batch."""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2503_20591_b200 import workloads as W

AMPLE = (640, 128000, 1048576)


def test_hand_worked_run():
    """Four 8-GPU hosts, nothing committed, S = (0, 0, 2, 4), limit 2/3 -> at most 16 subscribed.
    Every request asks for 4 GPUs. Equal idle GPUs everywhere, so the lowest S/(G R) wins, then id.
      r0: S = 0,0,2,4 -> hosts 0,1,2            -> S = 4,4,6,4
      r1: S = 4,4,6,4 -> hosts 0,1,3 (ties: id) -> S = 8,8,6,8
      r2: S = 8,8,6,8 -> hosts 2,0,1            -> S = 12,12,10,8
      r3: -> hosts 3,2,0                         -> S = 16,12,14,12
      r4: host 0 is full (16+4 > 16) and so is host 2 (14+4 > 16); hosts 1 and 3 fit (12+4 = 16)
          -> only two found: nothing is committed, output 1,3,-1.
      r5: same state as r4 -> same answer."""
    G, S, C = np.full(4, 8), np.array([0, 0, 2, 4]), np.zeros(4, dtype=int)
    ample = [np.full(4, x) for x in AMPLE]
    req = np.array([[4, 64, 1000, 1024]] * 6, dtype=np.int32)
    hosts, found, s_final = oracle.place_sequential(G, S, C, *ample, 2, 3, req)
    assert hosts.tolist() == [[0, 1, 2], [0, 1, 3], [2, 0, 1], [3, 2, 0], [1, 3, -1], [1, 3, -1]]
    assert found.tolist() == [3, 3, 3, 3, 2, 2]
    assert s_final.tolist() == [16, 12, 14, 12]


def test_closed_form_round_robin():
    """H identical empty hosts (H divisible by 3), every request asks for 1 GPU, limit L: request t
    takes hosts 3t, 3t+1, 3t+2 (mod H) until every host holds cap = floor(L G R) subscriptions;
    after that nothing fits."""
    H, cap = 12, 5                       # limit 5/24 with G = 8, R = 3 -> cap = 5
    G, S, C = np.full(H, 8), np.zeros(H, dtype=int), np.zeros(H, dtype=int)
    ample = [np.full(H, x) for x in AMPLE]
    n_fit = H * cap // 3
    req = np.array([[1, 16, 1000, 1024]] * (n_fit + 4), dtype=np.int32)
    hosts, found, s_final = oracle.place_sequential(G, S, C, *ample, 5, 24, req)
    for t in range(n_fit):
        assert hosts[t].tolist() == [(3 * t + k) % H for k in range(3)], t
    assert (found[:n_fit] == 3).all() and (found[n_fit:] == 0).all()
    assert (hosts[n_fit:] == -1).all()
    assert (s_final == cap).all()


def python_sequential(G, S, C, AV, AC, AM, num, den, requests, R=3, key_order=0, flags=0):
    S = [int(x) for x in S]
    out, found = [], []
    for g, v, c, m in np.asarray(requests, dtype=np.int64):
        cand = []
        for h in range(len(G)):
            if min(g, v, c, m) < 0 or G[h] < 1 or g > G[h] or v > AV[h] or c > AC[h] or m > AM[h]:
                continue
            if Fraction(S[h] + int(g), int(G[h]) * R) > Fraction(num, den):
                continue
            if flags & 1 and g > G[h] - C[h]:
                continue
            idle, sr = int(G[h] - C[h]), Fraction(S[h] + int(g), int(G[h]) * R)
            cand.append(((-idle, sr, h) if key_order == 0 else (sr, -idle, h), h))
        best = [h for _, h in sorted(cand)[:3]]
        found.append(len(best))
        out.append(best + [-1] * (3 - len(best)))
        if len(best) == 3:
            for h in best:
                S[h] += int(g)
    return np.array(out, dtype=np.int32), np.array(found, dtype=np.int32), np.array(S, dtype=np.int32)


@pytest.mark.parametrize("seed", range(4))
@pytest.mark.parametrize("key_order", [0, 1])
def test_against_python_reimplementation(seed, key_order):
    w = (W.make_config(0, batch=300) if seed % 2 == 0 else W.mixed_gpu_cluster(40, 300, seed=seed))
    args = (w.gpus_total[0], w.gpus_subscribed[0], w.gpus_committed[0], w.vram_gb[0], w.millicpus[0],
            w.mem_mb[0], int(w.limit_num[0]), int(w.limit_den[0]), w.requests[0])
    a = oracle.place_sequential(*args, key_order=key_order, flags=seed // 2)
    b = python_sequential(*args, key_order=key_order, flags=seed // 2)
    for x, y in zip(a, b):
        np.testing.assert_array_equal(x, y)
    assert (a[1] == 3).any()


def test_relations_to_the_frozen_batch():
    w = W.make_config(1, batch=500)
    args = (w.gpus_total[0], w.gpus_subscribed[0], w.gpus_committed[0], w.vram_gb[0], w.millicpus[0],
            w.mem_mb[0], int(w.limit_num[0]), int(w.limit_den[0]))
    frozen = oracle.place(*args, w.requests[0])
    seq = oracle.place_sequential(*args, w.requests[0])
    # the first request sees the untouched snapshot
    assert seq[0][0].tolist() == frozen[0][0].tolist()
    # later ones do not all get the same three hosts any more
    assert len({tuple(r) for r in seq[0]}) > len({tuple(r) for r in frozen[0]})
    # conservation: what was subscribed is 3 x the GPUs of the kernels that were created
    created = seq[1] == 3
    assert int(seq[2].sum() - w.gpus_subscribed[0].sum()) == 3 * int(w.requests[0][created, 0].sum())
    # no host ever exceeds the limit: S <= floor(num G R / den)
    cap = (int(w.limit_num[0]) * w.gpus_total[0].astype(np.int64) * 3) // int(w.limit_den[0])
    grew = seq[2] > w.gpus_subscribed[0]
    assert (seq[2][grew] <= cap[grew]).all()
    # requests that ask for nothing change nothing: sequential == frozen
    zero = w.requests[0].copy()
    zero[:, 0] = 0
    zero[:, 1] = 0
    a = oracle.place(*args, zero)
    b = oracle.place_sequential(*args, zero)
    np.testing.assert_array_equal(a[0], b[0])
    np.testing.assert_array_equal(b[2], w.gpus_subscribed[0])
