"""Pins for the CPU checker: it is compared with things other than itself.

 - the value the paper prints (Section 3.4.1 subscription-ratio example);
 - placements worked out by hand from the rule (tests/golden/hand_worked_cases.txt);
 - an independent second implementation built on exact fractions + numpy.lexsort;
 - brute force over all ordered triples on tiny clusters;
 - a closed form (uniform GPUs, ample capacity, loose limit);
 - invariants and metamorphic relations;
 - planted mistakes: each plausible slip in the checker's source must break a pin.
"""
from __future__ import annotations

import ctypes
import itertools
import os
import re
import subprocess
from fractions import Fraction

import numpy as np
import pytest

import oracle
from oracle import placement as oracle_placement
from paper_2503_20591_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
AMPLE = (640, 128000, 1048576)


# ----------------------------------------------------------------------------------------------
# golden fixtures
# ----------------------------------------------------------------------------------------------
def load_cases(path=os.path.join(GOLDEN, "hand_worked_cases.txt")):
    cases, cur = [], None
    for line in open(path):
        line = line.split("#")[0].strip()
        if not line:
            continue
        tok = line.split()
        if tok[0] == "case":
            kv = dict(t.split("=") for t in tok[2:])
            num, den = kv["limit"].split("/")
            cur = dict(name=tok[1], R=int(kv["R"]), num=int(num), den=int(den),
                       order={"idle_first": 0, "sr_first": 1}[kv["order"]],
                       flags=int(kv["flags"]), hosts=[], reqs=[])
            cases.append(cur)
        elif tok[0] == "host":
            cur["hosts"].append([int(x) for x in tok[1:7]])
        elif tok[0] == "req":
            arrow = tok.index("->")
            req = [int(x) for x in tok[1:arrow]]
            exp = [int(x) for x in tok[arrow + 1:arrow + 4]]
            found = int(tok[arrow + 4].split("=")[1])
            cur["reqs"].append((req, exp, found))
    return cases


def run_case(case, place_fn):
    """Returns a list of (request, expected, got) mismatches."""
    hosts = np.array(case["hosts"], dtype=np.int32)
    bad = []
    for req, exp, found in case["reqs"]:
        h, f = place_fn(hosts[:, 0], hosts[:, 1], hosts[:, 2], hosts[:, 3], hosts[:, 4],
                        hosts[:, 5], case["num"], case["den"], np.array([req], dtype=np.int32),
                        replicas_R=case["R"], key_order=case["order"], flags=case["flags"])
        if list(h[0]) != exp or int(f[0]) != found:
            bad.append((req, exp + [found], list(h[0]) + [int(f[0])]))
    return bad


def test_paper_sr_example():
    """Section 3.4.1 prints SR = 16 / (8 * 3) = 0.667."""
    rows = [l.split() for l in open(os.path.join(GOLDEN, "sr_worked_example.txt"))
            if l.strip() and not l.startswith("#")]
    assert rows
    for S, G, R, printed in rows:
        sr = oracle.subscription_ratio(int(S), int(G), int(R))
        assert f"{sr:.3f}" == printed
        assert Fraction(int(S), int(G) * int(R)) == Fraction(2, 3)


@pytest.mark.parametrize("case", load_cases(), ids=lambda c: c["name"])
def test_hand_worked_cases(case):
    assert run_case(case, oracle.place) == []


# ----------------------------------------------------------------------------------------------
# independent second implementation: exact fractions + numpy.lexsort
# ----------------------------------------------------------------------------------------------
def second_opinion(G, S, C, AV, AC, AM, num, den, requests, R=3, key_order=0, flags=0):
    G, S, C, AV, AC, AM = (np.asarray(x, dtype=np.int64) for x in (G, S, C, AV, AC, AM))
    H = len(G)
    limit = Fraction(num, den)
    out = np.full((len(requests), 3), -1, dtype=np.int32)
    found = np.zeros(len(requests), dtype=np.int32)
    ids = np.arange(H)
    for r, (g, v, c, m) in enumerate(np.asarray(requests, dtype=np.int64)):
        if min(g, v, c, m) < 0:
            continue
        sr_after = [Fraction(int(S[h] + g), int(G[h]) * R) if G[h] >= 1 else None for h in range(H)]
        ok = np.array([G[h] >= 1 and g <= G[h] and v <= AV[h] and c <= AC[h] and m <= AM[h]
                       and sr_after[h] <= limit
                       and (not (flags & 1) or g <= G[h] - C[h]) for h in range(H)], dtype=bool)
        cand = ids[ok]
        if cand.size == 0:
            continue
        # rank the distinct SR values so lexsort can work on integers
        distinct = sorted({sr_after[h] for h in cand})
        sr_rank = np.array([distinct.index(sr_after[h]) for h in cand])
        neg_idle = -(G[cand] - C[cand])
        keys = (cand, sr_rank, neg_idle) if key_order == 0 else (cand, neg_idle, sr_rank)
        order = cand[np.lexsort(keys)]       # last key is the primary one
        k = min(3, order.size)
        out[r, :k] = order[:k]
        found[r] = k
    return out, found


def _small_random_cluster(rng, H, mixed):
    G = rng.integers(1, 9, size=H) if mixed else np.full(H, 8)
    S = rng.integers(0, 3 * G + 2)
    C = rng.integers(0, np.minimum(G, S) + 1)
    AV = 80 * (G - C)
    AC = rng.integers(0, 20001, size=H)
    AM = rng.integers(0, 70001, size=H)
    return G, S, C, AV, AC, AM


def _small_random_requests(rng, B):
    g = rng.integers(0, 10, size=B)
    return np.stack([g, 16 * g, rng.integers(0, 16001, size=B), rng.integers(0, 65537, size=B)],
                    axis=1).astype(np.int32)


@pytest.mark.parametrize("seed", range(6))
@pytest.mark.parametrize("key_order", [0, 1])
def test_against_fraction_lexsort(seed, key_order):
    rng = np.random.default_rng(100 + seed)
    H = int(rng.integers(1, 40))
    cl = _small_random_cluster(rng, H, mixed=(seed % 2 == 0))
    req = _small_random_requests(rng, 60)
    num, den = [(2, 3), (1, 1), (5, 12), (4, 3), (1, 3), (7, 12)][seed]
    flags = seed % 3 == 0
    a = oracle.place(*cl, num, den, req, key_order=key_order, flags=int(flags))
    b = second_opinion(*cl, num, den, req, key_order=key_order, flags=int(flags))
    np.testing.assert_array_equal(a[0], b[0])
    np.testing.assert_array_equal(a[1], b[1])
    assert (a[1] < 3).any() or H > 3      # the sparse case is exercised somewhere


def test_against_fraction_lexsort_on_generated_workloads():
    for w in (W.make_config(0, batch=48), W.make_config(2, batch=12),
              W.make_config(3, batch=4), W.mixed_gpu_cluster(64, 40, seed=7)):
        for key_order in (0, 1):
            args = (w.gpus_total[0], w.gpus_subscribed[0], w.gpus_committed[0], w.vram_gb[0],
                    w.millicpus[0], w.mem_mb[0], int(w.limit_num[0]), int(w.limit_den[0]),
                    w.requests[0])
            a = oracle.place(*args, key_order=key_order)
            b = second_opinion(*args, key_order=key_order)
            np.testing.assert_array_equal(a[0], b[0])
            np.testing.assert_array_equal(a[1], b[1])


# ----------------------------------------------------------------------------------------------
# brute force over ordered triples (tiny clusters)
# ----------------------------------------------------------------------------------------------
def _rank_tuple(G, S, C, h, g, key_order):
    idle = int(G[h] - C[h])
    sr = Fraction(int(S[h] + g), int(G[h]) * 3)
    return (-idle, sr, h) if key_order == 0 else (sr, -idle, h)


@pytest.mark.parametrize("seed", range(5))
def test_brute_force_triples(seed):
    rng = np.random.default_rng(500 + seed)
    H = int(rng.integers(3, 7))
    G, S, C, AV, AC, AM = _small_random_cluster(rng, H, mixed=True)
    req = _small_random_requests(rng, 25)
    num, den = 1, 1
    for key_order in (0, 1):
        hosts, found = oracle.place(G, S, C, AV, AC, AM, num, den, req, key_order=key_order)
        for r, (g, v, c, m) in enumerate(req):
            feas = [h for h in range(H)
                    if g <= G[h] and v <= AV[h] and c <= AC[h] and m <= AM[h]
                    and Fraction(int(S[h] + g), int(G[h]) * 3) <= Fraction(num, den)]
            k = min(3, len(feas))
            assert found[r] == k
            best = None
            for trip in itertools.permutations(feas, k):
                score = tuple(_rank_tuple(G, S, C, h, int(g), key_order) for h in trip)
                if best is None or score < best[0]:
                    best = (score, trip)
            expect = list(best[1]) + [-1] * (3 - k) if best else [-1, -1, -1]
            assert list(hosts[r]) == expect


# ----------------------------------------------------------------------------------------------
# closed form
# ----------------------------------------------------------------------------------------------
def test_closed_form_uniform_cluster():
    """Uniform G, ample capacity, loose limit: nothing is rejected, the order does not depend on
    the request, and it is (C ascending, S ascending, id) -- so every request gets the same triple."""
    rng = np.random.default_rng(9)
    H = 50
    G = np.full(H, 8)
    S = rng.integers(0, 17, size=H)
    C = rng.integers(0, 9, size=H)
    ample = [np.full(H, x) for x in AMPLE]
    req = np.array([[g, 16 * g, 1000, 1024] for g in (0, 1, 2, 4, 8)], dtype=np.int32)
    hosts, found = oracle.place(G, S, C, *ample, 100, 1, req)
    expect = sorted(range(H), key=lambda h: (C[h], S[h], h))[:3]
    assert (found == 3).all()
    for row in hosts:
        assert list(row) == expect
    # swapped order: (S ascending, C ascending, id)
    hosts, _ = oracle.place(G, S, C, *ample, 100, 1, req, key_order=oracle.KEY_SR_FIRST)
    expect = sorted(range(H), key=lambda h: (S[h], C[h], h))[:3]
    for row in hosts:
        assert list(row) == expect


# ----------------------------------------------------------------------------------------------
# invariants (predicate written here, independently) and metamorphic relations
# ----------------------------------------------------------------------------------------------
def check_invariants(w, n, hosts, found, key_order=0, flags=0, request_ids=None):
    G, S, C = (x[n].astype(np.int64) for x in (w.gpus_total, w.gpus_subscribed, w.gpus_committed))
    AV, AC, AM = (x[n].astype(np.int64) for x in (w.vram_gb, w.millicpus, w.mem_mb))
    num, den, R = int(w.limit_num[n]), int(w.limit_den[n]), w.replicas_R
    reqs = w.requests[n] if request_ids is None else w.requests[n][request_ids]
    idle = G - C
    for r, (g, v, c, m) in enumerate(reqs.astype(np.int64)):
        ok = ((G >= 1) & (g <= G) & (v <= AV) & (c <= AC) & (m <= AM)
              & ((S + g) * den <= num * G * R))
        if flags & 1:
            ok &= g <= idle
        if min(g, v, c, m) < 0:
            ok[:] = False
        k = int(found[r])
        assert k == min(3, int(ok.sum()))
        chosen = [int(x) for x in hosts[r][:k]]
        assert all(x == -1 for x in hosts[r][k:])
        assert len(set(chosen)) == k and all(0 <= x < len(G) and ok[x] for x in chosen)

        def rank(h):
            # cross-multiplied SR against a common denominator: (S+g) * prod / G is avoided;
            # use exact fractions instead
            sr = Fraction(int(S[h] + g), int(G[h]) * R)
            return (-int(idle[h]), sr, h) if key_order == 0 else (sr, -int(idle[h]), h)

        ranks = [rank(h) for h in chosen]
        assert ranks == sorted(ranks)
        if k == 3:
            worst = ranks[-1]
            for h in np.nonzero(ok)[0]:
                if int(h) not in chosen:
                    assert rank(int(h)) > worst


def test_invariants_on_generated_workloads():
    for w in (W.make_config(0, batch=64), W.make_config(2, batch=24),
              W.make_config(4, batch=6, n_snapshots=9), W.mixed_gpu_cluster(96, 64, seed=3)):
        for key_order in (0, 1):
            hosts, found = oracle.place_workload(w, key_order=key_order)
            for n in range(w.n_snapshots):
                check_invariants(w, n, hosts[n], found[n], key_order=key_order)
    w = W.make_config(2, batch=24)
    hosts, found = oracle.place_workload(w, flags=oracle.REQUIRE_IDLE_GPUS)
    check_invariants(w, 0, hosts[0], found[0], flags=1)


def test_sparse_workload_hits_the_sentinel():
    w = W.make_config(2, batch=2048)
    _, found = oracle.place_workload(w, flags=oracle.REQUIRE_IDLE_GPUS)
    assert (found < 3).any()


def test_host_permutation_only_moves_ids():
    """Permuting hosts changes results only through the id tie-break: with all-distinct
    (idle, SR) pairs the answer is the same set of hosts, mapped through the permutation."""
    rng = np.random.default_rng(11)
    H = 40
    G = np.full(H, 8)
    pairs = rng.permutation([(s, c) for s in range(0, 17) for c in range(0, 9) if c <= s])[:H]
    S, C = pairs[:, 0], pairs[:, 1]
    ample = [np.full(H, x) for x in AMPLE]
    req = _small_random_requests(rng, 30)
    req[:, 2:] = 1000
    base, bf = oracle.place(G, S, C, *ample, 2, 3, req)
    perm = rng.permutation(H)            # new position p holds old host perm[p]
    h2, f2 = oracle.place(G[perm], S[perm], C[perm], *ample, 2, 3, req)
    np.testing.assert_array_equal(bf, f2)
    mapped = np.where(h2 >= 0, perm[np.clip(h2, 0, H - 1)], -1)
    np.testing.assert_array_equal(base, mapped)


def test_raising_the_limit_never_loses_candidates():
    w = W.make_config(4, batch=32, n_snapshots=8)
    prev = None
    for raw in W.SWEEP_RAW_LIMITS:
        lim = W.raw_limit_to_paper_units(raw)
        _, found = oracle.place(w.gpus_total[0], w.gpus_subscribed[0], w.gpus_committed[0],
                                w.vram_gb[0], w.millicpus[0], w.mem_mb[0],
                                lim.numerator, lim.denominator, w.requests[0])
        if prev is not None:
            assert (found >= prev).all()
        prev = found


def test_never_feasible_host_changes_nothing():
    w = W.make_config(1, batch=64)
    args = [w.gpus_total[0], w.gpus_subscribed[0], w.gpus_committed[0], w.vram_gb[0],
            w.millicpus[0], w.mem_mb[0]]
    base = oracle.place(*args, 2, 3, w.requests[0])
    extra = [np.append(a, x) for a, x in zip(args, (8, 1000, 0, 640, 128000, 1048576))]
    more = oracle.place(*extra, 2, 3, w.requests[0])
    np.testing.assert_array_equal(base[0], more[0])
    np.testing.assert_array_equal(base[1], more[1])


def test_degenerate_inputs():
    one = [np.array([x]) for x in (8, 0, 0, 640, 128000, 1048576)]
    # negative request fields fit nowhere
    for bad in ([-1, 0, 0, 0], [1, -1, 0, 0], [1, 0, -5, 0], [1, 0, 0, -7]):
        h, f = oracle.place(*one, 2, 3, np.array([bad], dtype=np.int32))
        assert list(h[0]) == [-1, -1, -1] and f[0] == 0
    # a server without GPUs is never a candidate, not even for g = 0
    zero = [np.array([x]) for x in (0, 0, 0, 640, 128000, 1048576)]
    h, f = oracle.place(*zero, 2, 3, np.array([[0, 0, 0, 0]], dtype=np.int32))
    assert f[0] == 0
    # empty batch, empty cluster
    h, f = oracle.place(*one, 2, 3, np.zeros((0, 4), dtype=np.int32))
    assert h.shape == (0, 3) and f.shape == (0,)
    none = [np.zeros(0, dtype=np.int32)] * 6
    h, f = oracle.place(*none, 2, 3, np.array([[1, 16, 1000, 1024]], dtype=np.int32))
    assert list(h[0]) == [-1, -1, -1] and f[0] == 0
    # limit 0: only S = 0, g = 0 stays within it
    h, f = oracle.place(*one, 0, 1, np.array([[0, 0, 0, 0], [1, 0, 0, 0]], dtype=np.int32))
    assert list(f) == [1, 0]


def test_thread_pool_front_end_is_the_same_function():
    w = W.make_config(4, batch=700, n_snapshots=3)
    a = oracle.place_workload(w, threads=1)
    b = oracle.place_workload(w, threads=4)
    np.testing.assert_array_equal(a[0], b[0])
    np.testing.assert_array_equal(a[1], b[1])


# ----------------------------------------------------------------------------------------------
# planted mistakes: every slip below must be caught by the hand-worked cases
# ----------------------------------------------------------------------------------------------
MUTATIONS = [
    ("idle order reversed", "return idle_a > idle_b; /* more idle GPUs first */",
     "return idle_a < idle_b;"),
    ("SR order reversed", "if (sr != 0) return sr < 0;             /* then lower SR             */",
     "if (sr != 0) return sr > 0;"),
    ("tie-break reversed", "return a < b; /* then lower host index */", "return a > b;"),
    ("SR before placement (g dropped)", "int64_t lhs = (Sa + g) * (Gb * R);",
     "int64_t lhs = (Sa) * (Gb * R);"),
    ("cross-multiplication transposed", "int64_t lhs = (Sa + g) * (Gb * R);",
     "int64_t lhs = (Sa + g) * (Ga * R);"),
    ("limit test not strict", "> cl->limit_num * G * R) return 0;", ">= cl->limit_num * G * R) return 0;"),
    ("R dropped from the limit test", "> cl->limit_num * G * R) return 0;",
     "> cl->limit_num * G) return 0;"),
    ("g left out of the limit test", "if ((S + (int64_t)g) * cl->limit_den", "if ((S) * cl->limit_den"),
    ("GPU capacity test dropped", "if (g > G) return 0;", ""),
    ("VRAM compared with CPU", "if (v > cl->AV[h]) return 0;", "if (v > cl->AC[h]) return 0;"),
    ("CPU test dropped", "if (c > cl->AC[h]) return 0;", ""),
    ("memory test dropped", "if (m > cl->AM[h]) return 0;", ""),
    ("idle test uses S instead of C", "(int64_t)g > G - C) return 0;", "(int64_t)g > G - S) return 0;"),
    ("idle flag ignored", "if ((cl->flags & NBOS_ORACLE_REQUIRE_IDLE_GPUS) &&", "if (0 &&"),
    ("idle = committed GPUs ascending", "int64_t idle_a = (int64_t)cl->G[a] - cl->C[a];",
     "int64_t idle_a = -(int64_t)cl->C[a];"),
    ("two placed instead of three", "#define NBOS_ORACLE_REPLICAS_PLACED 3",
     "#define NBOS_ORACLE_REPLICAS_PLACED 2"),
    ("order flag ignored", "if (cl->key_order == NBOS_ORACLE_KEY_SR_FIRST) {", "if (0) {"),
]


@pytest.mark.parametrize("mutation", MUTATIONS, ids=lambda m: m[0])
def test_planted_mistake_is_caught(mutation, tmp_path):
    _, old, new = mutation
    src = open(os.path.join(os.path.dirname(oracle_placement.__file__), "nbos_oracle.c")).read()
    if mutation[0] == "idle = committed GPUs ascending":
        src = src.replace("int64_t idle_b = (int64_t)cl->G[b] - cl->C[b];",
                          "int64_t idle_b = -(int64_t)cl->C[b];")
    assert src.count(old) == 1, f"mutation anchor not found exactly once: {old!r}"
    mutated = src.replace(old, new)
    c_path, so_path = tmp_path / "m.c", tmp_path / "m.so"
    c_path.write_text(mutated)
    subprocess.run(["gcc", "-O1", "-std=c99", "-fPIC", "-shared", "-w", "-o", str(so_path),
                    str(c_path)], check=True)
    lib = ctypes.CDLL(str(so_path))
    lib.nbos_oracle_place.restype = ctypes.c_int
    lib.nbos_oracle_place.argtypes = oracle_placement._load().nbos_oracle_place.argtypes

    def place_mut(G, S, C, AV, AC, AM, num, den, requests, replicas_R=3, key_order=0, flags=0):
        cl, keep = oracle_placement._cluster(G, S, C, AV, AC, AM, num, den, replicas_R,
                                             key_order, flags)
        req = np.ascontiguousarray(requests, dtype=np.int32).reshape(-1, 4)
        hosts = np.empty((req.shape[0], 3), dtype=np.int32)
        found = np.empty(req.shape[0], dtype=np.int32)
        p = oracle_placement._i32p
        lib.nbos_oracle_place(ctypes.byref(cl), req.ctypes.data_as(p), req.shape[0],
                              hosts.ctypes.data_as(p), found.ctypes.data_as(p))
        return hosts, found

    failures = sum(len(run_case(c, place_mut)) for c in load_cases())
    assert failures > 0, f"no hand-worked case notices: {mutation[0]}"
