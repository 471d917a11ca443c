"""Pins for the CPU checker's executor selection (Section 3.2.2): hand-worked cases, an
independent implementation on exact fractions, invariants, and planted mistakes."""
from __future__ import annotations

import ctypes
import os
import subprocess
from fractions import Fraction

import numpy as np
import pytest

import oracle
from oracle import placement as oracle_placement

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "executor_cases.txt")


def load_cases():
    cases, cur = [], None
    for line in open(GOLDEN):
        line = line.split("#")[0].strip()
        if not line:
            continue
        tok = line.split()
        if tok[0] == "case":
            cur = dict(name=tok[1], R=int(tok[2].split("=")[1]), hosts=[], execs=[])
            cases.append(cur)
        elif tok[0] == "host":
            cur["hosts"].append([int(x) for x in tok[1:7]])
        elif tok[0] == "exec":
            bar, arrow = tok.index("|"), tok.index("->")
            cur["execs"].append(([int(x) for x in tok[1:bar]], [int(x) for x in tok[bar + 1:arrow]],
                                 int(tok[arrow + 1]), int(tok[arrow + 2].split("=")[1])))
    return cases


def run_case(case, fn):
    hosts = np.array(case["hosts"], dtype=np.int32)
    bad = []
    for req, rep, want_exec, want_mask in case["execs"]:
        ex, mask = fn(*[hosts[:, i] for i in range(6)], np.array([req], dtype=np.int32),
                      np.array([rep], dtype=np.int32), replicas_R=case["R"])
        if (int(ex[0]), int(mask[0])) != (want_exec, want_mask):
            bad.append((req, rep, (want_exec, want_mask), (int(ex[0]), int(mask[0]))))
    return bad


@pytest.mark.parametrize("case", load_cases(), ids=lambda c: c["name"])
def test_hand_worked_executor_cases(case):
    assert run_case(case, oracle.select_executors) == []


def second_opinion(G, S, C, AV, AC, AM, requests, replica_hosts, R=3):
    ex, masks = [], []
    for (g, v, c, m), rep in zip(np.asarray(requests, dtype=np.int64), np.asarray(replica_hosts)):
        cands, mask = [], 0
        for slot, h in enumerate(rep):
            if h < 0 or h >= len(G) or min(g, v, c, m) < 0 or G[h] < 1:
                continue
            if g <= G[h] - C[h] and v <= AV[h] and c <= AC[h] and m <= AM[h]:
                mask |= 1 << slot
                cands.append((-(int(G[h]) - int(C[h])), Fraction(int(S[h]), int(G[h]) * R), int(h), slot))
        ex.append(min(cands)[2] if cands else -1)
        masks.append(mask)
    return np.array(ex, dtype=np.int32), np.array(masks, dtype=np.int32)


@pytest.mark.parametrize("seed", range(5))
def test_against_fraction_implementation(seed):
    rng = np.random.default_rng(900 + seed)
    H, M = int(rng.integers(3, 60)), 400
    G = rng.integers(0, 9, size=H)
    S = rng.integers(0, 3 * G + 2)
    C = rng.integers(0, np.minimum(G, S) + 1)
    AV, AC, AM = 80 * (G - C), rng.integers(0, 20001, size=H), rng.integers(0, 70001, size=H)
    g = rng.integers(0, 9, size=M)
    req = np.stack([g, 16 * g, rng.integers(0, 16001, size=M), rng.integers(0, 65537, size=M)], axis=1)
    rep = np.stack([rng.permutation(H)[:3] if H >= 3 else rng.integers(0, H, 3) for _ in range(M)])
    rep[rng.random(M) < 0.05, 2] = -1
    a = oracle.select_executors(G, S, C, AV, AC, AM, req, rep)
    b = second_opinion(G, S, C, AV, AC, AM, req, rep)
    np.testing.assert_array_equal(a[0], b[0])
    np.testing.assert_array_equal(a[1], b[1])
    # invariants: the executor is one of the replicas that can run; -1 iff none can
    for k in range(M):
        runnable = [rep[k, s] for s in range(3) if a[1][k] >> s & 1]
        assert (a[0][k] == -1) == (len(runnable) == 0)
        assert a[0][k] == -1 or a[0][k] in runnable
    assert (a[0] == -1).any() and (a[0] >= 0).any()


MUTATIONS = [
    ("idle test uses total GPUs", "if ((int64_t)g > G - C) continue;          /* idle GPUs, bound at once */",
     "if ((int64_t)g > G) continue;"),
    ("idle order reversed", "before = idle_h > idle_b;", "before = idle_h < idle_b;"),
    ("SR order reversed", "before = sr != 0 ? sr < 0 : h < best;", "before = sr != 0 ? sr > 0 : h < best;"),
    ("host tie-break reversed", "before = sr != 0 ? sr < 0 : h < best;", "before = sr != 0 ? sr < 0 : h > best;"),
    ("VRAM test dropped", "if (v > cl->AV[h] || c > cl->AC[h] || m > cl->AM[h]) continue;",
     "if (c > cl->AC[h] || m > cl->AM[h]) continue;"),
    ("CPU test dropped", "if (v > cl->AV[h] || c > cl->AC[h] || m > cl->AM[h]) continue;",
     "if (v > cl->AV[h] || m > cl->AM[h]) continue;"),
    ("memory test dropped", "if (v > cl->AV[h] || c > cl->AC[h] || m > cl->AM[h]) continue;",
     "if (v > cl->AV[h] || c > cl->AC[h]) continue;"),
    ("mask bit by host instead of slot", "mask |= 1 << slot;", "mask |= 1 << (h % 3);"),
    ("first runnable wins", "if (before) best = h;", ""),
]


@pytest.mark.parametrize("mutation", MUTATIONS, ids=lambda m: m[0])
def test_planted_mistake_is_caught(mutation, tmp_path):
    _, old, new = mutation
    src = open(os.path.join(os.path.dirname(oracle_placement.__file__), "nbos_oracle.c")).read()
    assert src.count(old) == 1, f"mutation anchor not found exactly once: {old!r}"
    (tmp_path / "m.c").write_text(src.replace(old, new))
    subprocess.run(["gcc", "-O1", "-std=c99", "-fPIC", "-shared", "-w", "-o", str(tmp_path / "m.so"),
                    str(tmp_path / "m.c")], check=True)
    lib = ctypes.CDLL(str(tmp_path / "m.so"))
    lib.nbos_oracle_select_executors.restype = ctypes.c_int
    lib.nbos_oracle_select_executors.argtypes = oracle_placement._load().nbos_oracle_select_executors.argtypes

    def mutated(G, S, C, AV, AC, AM, requests, replica_hosts, replicas_R=3):
        cl, keep = oracle_placement._cluster(G, S, C, AV, AC, AM, 1, 1, replicas_R, 0, 0)
        req = np.ascontiguousarray(requests, dtype=np.int32).reshape(-1, 4)
        rep = np.ascontiguousarray(replica_hosts, dtype=np.int32).reshape(-1, 3)
        ex = np.empty(req.shape[0], dtype=np.int32)
        mask = np.empty(req.shape[0], dtype=np.int32)
        p = oracle_placement._i32p
        lib.nbos_oracle_select_executors(ctypes.byref(cl), req.ctypes.data_as(p), rep.ctypes.data_as(p),
                                         req.shape[0], ex.ctypes.data_as(p), mask.ctypes.data_as(p))
        return ex, mask

    assert sum(len(run_case(c, mutated)) for c in load_cases()) > 0, f"unnoticed: {mutation[0]}"
