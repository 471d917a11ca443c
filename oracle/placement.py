"""ctypes front end of the plain-C placement checker (nbos_oracle.c).

Test infrastructure only: slow, single-threaded per call, written for being
checked by eye against Sections 3.2.1 and 3.4.1 of the paper. `place_workload`
may run several calls at once on a thread pool (each call is still the plain
single-threaded loop over its own slice of requests); that is a convenience for
the tests' wall clock, not an optimisation of the checker.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

import numpy as np

KEY_IDLE_FIRST = 0
KEY_SR_FIRST = 1
REQUIRE_IDLE_GPUS = 1

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "nbos_oracle.c")
_LIB = os.path.join(_HERE, "libnbos_oracle.so")
_lib = None

_i32p = ctypes.POINTER(ctypes.c_int32)


class _Cluster(ctypes.Structure):
    _fields_ = [
        ("n_hosts", ctypes.c_int32),
        ("replicas_R", ctypes.c_int32),
        ("key_order", ctypes.c_int32),
        ("flags", ctypes.c_int32),
        ("limit_num", ctypes.c_int64),
        ("limit_den", ctypes.c_int64),
        ("G", _i32p), ("S", _i32p), ("C", _i32p),
        ("AV", _i32p), ("AC", _i32p), ("AM", _i32p),
    ]


def build(force: bool = False) -> str:
    """Compile nbos_oracle.c with gcc into libnbos_oracle.so next to it."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.run(["gcc", "-O2", "-std=c99", "-Wall", "-Wextra", "-fPIC", "-shared",
                        "-o", tmp, _SRC], check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.nbos_oracle_subscription_ratio.restype = ctypes.c_double
        lib.nbos_oracle_subscription_ratio.argtypes = [ctypes.c_int64] * 3
        lib.nbos_oracle_compare_sr_after.restype = ctypes.c_int
        lib.nbos_oracle_compare_sr_after.argtypes = [ctypes.c_int64] * 6
        lib.nbos_oracle_feasible.restype = ctypes.c_int
        lib.nbos_oracle_feasible.argtypes = [ctypes.POINTER(_Cluster)] + [ctypes.c_int32] * 5
        lib.nbos_oracle_ranks_before.restype = ctypes.c_int
        lib.nbos_oracle_ranks_before.argtypes = [ctypes.POINTER(_Cluster)] + [ctypes.c_int32] * 3
        lib.nbos_oracle_place.restype = ctypes.c_int
        lib.nbos_oracle_place.argtypes = [ctypes.POINTER(_Cluster), _i32p, ctypes.c_int64,
                                          _i32p, _i32p]
        lib.nbos_oracle_select_executors.restype = ctypes.c_int
        lib.nbos_oracle_select_executors.argtypes = [ctypes.POINTER(_Cluster), _i32p, _i32p,
                                                     ctypes.c_int64, _i32p, _i32p]
        lib.nbos_oracle_place_sequential.restype = ctypes.c_int
        lib.nbos_oracle_place_sequential.argtypes = [ctypes.POINTER(_Cluster), _i32p, ctypes.c_int64,
                                                     _i32p, _i32p, _i32p]
        i64p = ctypes.POINTER(ctypes.c_int64)
        lib.nbos_oracle_cluster_sums.restype = None
        lib.nbos_oracle_cluster_sums.argtypes = [ctypes.POINTER(_Cluster), i64p]
        lib.nbos_oracle_cluster_limit.restype = None
        lib.nbos_oracle_cluster_limit.argtypes = [ctypes.POINTER(_Cluster), i64p, i64p]
        lib.nbos_oracle_autoscale.restype = ctypes.c_int
        lib.nbos_oracle_autoscale.argtypes = [ctypes.c_int64] * 4
        lib.nbos_oracle_scale_out_deficit.restype = None
        lib.nbos_oracle_scale_out_deficit.argtypes = [_i32p, ctypes.c_int64, i64p, i64p]
        _lib = lib
    return _lib


def _as_i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _cluster(G, S, C, AV, AC, AM, limit_num, limit_den, replicas_R, key_order, flags):
    arrs = [_as_i32(x) for x in (G, S, C, AV, AC, AM)]
    h = arrs[0].shape[0]
    if any(a.shape != (h,) for a in arrs):
        raise ValueError("host arrays must all be 1-D of the same length")
    cl = _Cluster(h, int(replicas_R), int(key_order), int(flags), int(limit_num), int(limit_den),
                  *[a.ctypes.data_as(_i32p) for a in arrs])
    return cl, arrs  # arrs kept alive by the caller


def subscription_ratio(S: int, G: int, R: int) -> float:
    return float(_load().nbos_oracle_subscription_ratio(S, G, R))


def compare_sr_after(Sa, Ga, Sb, Gb, g, R) -> int:
    return int(_load().nbos_oracle_compare_sr_after(Sa, Ga, Sb, Gb, g, R))


def feasible(G, S, C, AV, AC, AM, limit_num, limit_den, h, request, replicas_R=3, flags=0) -> bool:
    cl, keep = _cluster(G, S, C, AV, AC, AM, limit_num, limit_den, replicas_R, 0, flags)
    g, v, c, m = (int(x) for x in request)
    return bool(_load().nbos_oracle_feasible(ctypes.byref(cl), int(h), g, v, c, m))


def ranks_before(G, S, C, a, b, g, replicas_R=3, key_order=KEY_IDLE_FIRST) -> bool:
    z = np.zeros(len(G), dtype=np.int32)
    cl, keep = _cluster(G, S, C, z, z, z, 1, 1, replicas_R, key_order, 0)
    return bool(_load().nbos_oracle_ranks_before(ctypes.byref(cl), int(a), int(b), int(g)))


def place(G, S, C, AV, AC, AM, limit_num, limit_den, requests, replicas_R=3,
          key_order=KEY_IDLE_FIRST, flags=0):
    """One snapshot, one batch. Returns (hosts [B,3] int32, found [B] int32)."""
    cl, keep = _cluster(G, S, C, AV, AC, AM, limit_num, limit_den, replicas_R, key_order, flags)
    req = _as_i32(requests).reshape(-1, 4)
    b = req.shape[0]
    hosts = np.empty((b, 3), dtype=np.int32)
    found = np.empty((b,), dtype=np.int32)
    rc = _load().nbos_oracle_place(ctypes.byref(cl), req.ctypes.data_as(_i32p), b,
                                   hosts.ctypes.data_as(_i32p), found.ctypes.data_as(_i32p))
    if rc != 0:
        raise ValueError("nbos_oracle_place rejected its arguments")
    return hosts, found


def select_executors(G, S, C, AV, AC, AM, requests, replica_hosts, replicas_R=3):
    """Section 3.2.2: which replica of each kernel runs the cell. Returns (executor [M] int32
    host index or -1, can_run [M] int32 bit mask over the three replica slots)."""
    cl, keep = _cluster(G, S, C, AV, AC, AM, 1, 1, replicas_R, 0, 0)
    req = _as_i32(requests).reshape(-1, 4)
    rep = _as_i32(replica_hosts).reshape(-1, 3)
    if rep.shape[0] != req.shape[0]:
        raise ValueError("one row of replica hosts per request")
    m = req.shape[0]
    ex = np.empty((m,), dtype=np.int32)
    mask = np.empty((m,), dtype=np.int32)
    rc = _load().nbos_oracle_select_executors(ctypes.byref(cl), req.ctypes.data_as(_i32p),
                                              rep.ctypes.data_as(_i32p), m,
                                              ex.ctypes.data_as(_i32p), mask.ctypes.data_as(_i32p))
    if rc != 0:
        raise ValueError("nbos_oracle_select_executors rejected its arguments")
    return ex, mask


def place_sequential(G, S, C, AV, AC, AM, limit_num, limit_den, requests, replicas_R=3,
                     key_order=KEY_IDLE_FIRST, flags=0):
    """One snapshot, requests placed one after the other; a request that finds three hosts adds
    its GPUs to their subscribed count before the next one is placed.
    Returns (hosts [B,3], found [B], S_final [H])."""
    cl, keep = _cluster(G, S, C, AV, AC, AM, limit_num, limit_den, replicas_R, key_order, flags)
    req = _as_i32(requests).reshape(-1, 4)
    b = req.shape[0]
    hosts = np.empty((b, 3), dtype=np.int32)
    found = np.empty((b,), dtype=np.int32)
    s_final = np.empty((cl.n_hosts,), dtype=np.int32)
    rc = _load().nbos_oracle_place_sequential(ctypes.byref(cl), req.ctypes.data_as(_i32p), b,
                                              hosts.ctypes.data_as(_i32p), found.ctypes.data_as(_i32p),
                                              s_final.ctypes.data_as(_i32p))
    if rc != 0:
        raise ValueError("nbos_oracle_place_sequential rejected its arguments")
    return hosts, found, s_final


def cluster_sums(G, S, C, replicas_R=3):
    """(sum G, sum S, sum C) of one snapshot."""
    z = np.zeros(len(G), dtype=np.int32)
    cl, keep = _cluster(G, S, C, z, z, z, 1, 1, replicas_R, 0, 0)
    out = (ctypes.c_int64 * 3)()
    _load().nbos_oracle_cluster_sums(ctypes.byref(cl), out)
    return int(out[0]), int(out[1]), int(out[2])


def cluster_limit(G, S, C, replicas_R=3):
    """Dynamic cluster-wide SR limit of Section 3.4.1 as (num, den) = (sum S, sum G * R)."""
    z = np.zeros(len(G), dtype=np.int32)
    cl, keep = _cluster(G, S, C, z, z, z, 1, 1, replicas_R, 0, 0)
    num, den = ctypes.c_int64(0), ctypes.c_int64(0)
    _load().nbos_oracle_cluster_limit(ctypes.byref(cl), ctypes.byref(num), ctypes.byref(den))
    return int(num.value), int(den.value)


def autoscale(sum_G, sum_C, f_num=21, f_den=20) -> int:
    """Section 3.4.2 with f = f_num / f_den: +1 scale out, -1 may release servers, 0 equal."""
    return int(_load().nbos_oracle_autoscale(int(sum_G), int(sum_C), int(f_num), int(f_den)))


def scale_out_deficit(found):
    """(sum of 3 - found, number of requests with found < 3) over one batch."""
    f = _as_i32(found).reshape(-1)
    d, n = ctypes.c_int64(0), ctypes.c_int64(0)
    _load().nbos_oracle_scale_out_deficit(f.ctypes.data_as(_i32p), f.shape[0], ctypes.byref(d),
                                          ctypes.byref(n))
    return int(d.value), int(n.value)


def place_workload(w, key_order=KEY_IDLE_FIRST, flags=0, threads: int = 1,
                   snapshots=None, request_slice=None):
    """Run the checker over a workload object (fields as in the input generators):
    every snapshot against its own batch. Returns (hosts [N,B,3], found [N,B]).
    `threads` > 1 splits the request list of each snapshot into slices handled by
    separate calls on a thread pool."""
    snaps = range(w.n_snapshots) if snapshots is None else list(snapshots)
    sl = slice(None) if request_slice is None else request_slice
    outs_h, outs_f = [], []

    def one(n, req):
        return place(w.gpus_total[n], w.gpus_subscribed[n], w.gpus_committed[n],
                     w.vram_gb[n], w.millicpus[n], w.mem_mb[n],
                     int(w.limit_num[n]), int(w.limit_den[n]), req,
                     replicas_R=w.replicas_R, key_order=key_order, flags=flags)

    jobs = []
    for n in snaps:
        req = w.requests[n][sl]
        parts = max(1, min(threads, (req.shape[0] + 255) // 256)) if threads > 1 else 1
        for chunk in np.array_split(np.arange(req.shape[0]), parts):
            lo, hi = (int(chunk[0]), int(chunk[-1]) + 1) if chunk.size else (0, 0)
            jobs.append((n, req[lo:hi]))
    if threads > 1:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            res = list(ex.map(lambda j: one(*j), jobs))
    else:
        res = [one(*j) for j in jobs]
    i = 0
    for n in snaps:
        hs, fs = [], []
        while i < len(jobs) and jobs[i][0] == n:
            hs.append(res[i][0]); fs.append(res[i][1]); i += 1
        outs_h.append(np.concatenate(hs)); outs_f.append(np.concatenate(fs))
    return np.stack(outs_h), np.stack(outs_f)
