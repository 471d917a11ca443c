"""ctypes front end of libnbos.so: the same entry points as include/nbos.h, by the same names.

Argument marshalling only. Tensors are torch tensors (device memory and streams are PyTorch's
job here); every step of the placement path runs inside the library's CUDA kernels. There is no
fallback: if libnbos.so is missing or cannot be loaded the first call raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libnbos.so")

NBOS_OK = 0
NBOS_ERR_INVALID_ARG = -1
NBOS_ERR_RANGE = -2
NBOS_ERR_CUDA = -3
NBOS_ERR_UNSUPPORTED_DEVICE = -4
NBOS_ERR_DEVICE_TIMEOUT = -5
NBOS_ERR_NO_MEMORY = -6
NBOS_ERR_STALE_LAYOUT = -7

NBOS_KEY_IDLE_FIRST = 0
NBOS_KEY_SR_FIRST = 1
NBOS_REQUIRE_IDLE_GPUS = 1
NBOS_FORCE_KEY64 = 2
NBOS_LIMIT_CLUSTER_SR = 4
NBOS_ROOM_FOR_COMMITS = 8

NBOS_MAX_HOSTS = 1 << 20
NBOS_MAX_REPLICAS = 1024
NBOS_SEQUENTIAL_MAX_HOSTS = 65536

NBOS_PROBE_MIX_ALU = 0
NBOS_PROBE_MIX_IMAD = 1
NBOS_PROBE_MIX_BOTH = 2

# every symbol include/nbos.h and include/nbos_probe.h declare
EXPORTED_SYMBOLS = (
    "nbos_snapshot_workspace_bytes", "nbos_snapshot_create", "nbos_snapshot_create_host",
    "nbos_snapshot_update", "nbos_snapshot_update_host",
    "nbos_snapshot_destroy", "nbos_snapshot_get_info", "nbos_place_batch", "nbos_place_batch_ex",
    "nbos_place_batch_host", "nbos_place_batch_host_async", "nbos_place_batch_host_wait",
    "nbos_place_batch_noalloc", "nbos_select_executors",
    "nbos_cluster_sums", "nbos_scale_out_deficit", "nbos_place_batch_sequential",
    "nbos_snapshot_status", "nbos_strerror", "nbos_last_error_detail",
    "nbos_probe_int32_issue", "nbos_probe_wait_timeout", "nbos_probe_wait_timeout_on_snapshot",
)

_i32p = ctypes.POINTER(ctypes.c_int32)


class nbos_snapshot_desc(ctypes.Structure):
    _fields_ = [
        ("n_snapshots", ctypes.c_int32), ("n_hosts", ctypes.c_int32),
        ("replicas_R", ctypes.c_int32), ("key_order", ctypes.c_int32),
        ("flags", ctypes.c_int32), ("reserved", ctypes.c_int32),
        ("limit_num", ctypes.c_void_p), ("limit_den", ctypes.c_void_p),
        ("gpus_total", ctypes.c_void_p), ("gpus_subscribed", ctypes.c_void_p),
        ("gpus_committed", ctypes.c_void_p), ("vram_gb", ctypes.c_void_p),
        ("millicpus", ctypes.c_void_p), ("mem_mb", ctypes.c_void_p),
    ]


class nbos_snapshot_info(ctypes.Structure):
    _fields_ = [
        ("n_snapshots", ctypes.c_int32), ("n_hosts", ctypes.c_int32),
        ("hosts_padded", ctypes.c_int32), ("key_bits", ctypes.c_int32),
        ("bits_idle", ctypes.c_int32), ("bits_sr", ctypes.c_int32), ("bits_id", ctypes.c_int32),
        ("key_order", ctypes.c_int32), ("flags", ctypes.c_int32), ("replicas_R", ctypes.c_int32),
        ("packed_test", ctypes.c_int32), ("static_key", ctypes.c_int32),
        ("presorted", ctypes.c_int32), ("grouped", ctypes.c_int32),
        ("workspace_bytes", ctypes.c_int64),
        ("ranked", ctypes.c_int32), ("ranked_dropped_bits", ctypes.c_int32 * 4),
        ("reserved", ctypes.c_int32),
    ]


class nbos_cluster_state(ctypes.Structure):
    _fields_ = [
        ("n_hosts", ctypes.c_int32), ("replicas_R", ctypes.c_int32),
        ("gpus_total", ctypes.c_void_p), ("gpus_subscribed", ctypes.c_void_p),
        ("gpus_committed", ctypes.c_void_p), ("vram_gb", ctypes.c_void_p),
        ("millicpus", ctypes.c_void_p), ("mem_mb", ctypes.c_void_p),
    ]


class nbos_launch_config(ctypes.Structure):
    _fields_ = [
        ("lanes_per_request", ctypes.c_int32), ("requests_per_lane", ctypes.c_int32),
        ("host_split", ctypes.c_int32), ("tile_hosts", ctypes.c_int32),
        ("grid_blocks", ctypes.c_int32), ("pair_mode", ctypes.c_int32),
        ("first_fit", ctypes.c_int32), ("reserved", ctypes.c_int32),
    ]


class NbosError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(what)


_lib = None


def load_library() -> ctypes.CDLL:
    """Open libnbos.so (built in-tree by paper_2503_20591_b200.build). Raises if it is absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise NbosError(NBOS_ERR_CUDA, f"{LIB_PATH} has not been built: run "
                                       "`python -m paper_2503_20591_b200.build` (needs nvcc); "
                                       "there is no CPU fallback")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i64, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_size_t
    P = ctypes.POINTER
    lib.nbos_snapshot_workspace_bytes.argtypes = [P(nbos_snapshot_desc), P(sz)]
    lib.nbos_snapshot_create.argtypes = [P(nbos_snapshot_desc), vp, sz, vp, P(vp)]
    lib.nbos_snapshot_create_host.argtypes = [P(nbos_snapshot_desc), vp, P(vp)]
    lib.nbos_snapshot_update.argtypes = [vp, P(nbos_snapshot_desc), vp]
    lib.nbos_snapshot_update_host.argtypes = [vp, P(nbos_snapshot_desc), vp]
    lib.nbos_snapshot_destroy.argtypes = [vp]
    lib.nbos_snapshot_get_info.argtypes = [vp, P(nbos_snapshot_info)]
    lib.nbos_place_batch.argtypes = [vp, vp, i64, vp, vp, vp]
    lib.nbos_place_batch_ex.argtypes = [vp, vp, i64, vp, vp, vp, P(nbos_launch_config)]
    lib.nbos_place_batch_host.argtypes = [vp, vp, i64, vp, vp, vp]
    lib.nbos_place_batch_host_async.argtypes = [vp, vp, i64, vp, vp, vp]
    lib.nbos_place_batch_host_wait.argtypes = [vp]
    lib.nbos_place_batch_noalloc.argtypes = [vp, vp, i64, vp, vp, vp, ctypes.c_int32]
    lib.nbos_select_executors.argtypes = [P(nbos_cluster_state), vp, vp, i64, vp, vp, vp]
    lib.nbos_cluster_sums.argtypes = [vp, vp, vp] + [ctypes.c_int32] * 4 + [vp, vp]
    lib.nbos_scale_out_deficit.argtypes = [vp, ctypes.c_int32, i64, vp, vp]
    lib.nbos_place_batch_sequential.argtypes = [vp, vp, i64, vp, vp, vp, vp]
    lib.nbos_snapshot_status.argtypes = [vp, vp]
    lib.nbos_strerror.argtypes = [ctypes.c_int]
    lib.nbos_strerror.restype = ctypes.c_char_p
    lib.nbos_last_error_detail.argtypes = []
    lib.nbos_last_error_detail.restype = ctypes.c_char_p
    lib.nbos_probe_int32_issue.argtypes = [ctypes.c_int] * 4 + [vp, P(ctypes.c_double),
                                                                P(ctypes.c_float)]
    lib.nbos_probe_wait_timeout.argtypes = [ctypes.c_uint64, vp, P(ctypes.c_int),
                                            P(ctypes.c_float)]
    lib.nbos_probe_wait_timeout_on_snapshot.argtypes = [vp, ctypes.c_uint64, vp, P(ctypes.c_float)]
    for name in EXPORTED_SYMBOLS:
        fn = getattr(lib, name)
        if name not in ("nbos_strerror", "nbos_last_error_detail"):
            fn.restype = ctypes.c_int
    _lib = lib
    return lib


def nbos_strerror(status: int) -> str:
    return load_library().nbos_strerror(status).decode()


def nbos_last_error_detail() -> str:
    return load_library().nbos_last_error_detail().decode()


def _check(status: int) -> None:
    if status != NBOS_OK:
        raise NbosError(status, f"{nbos_strerror(status)} ({status}): {nbos_last_error_detail()}")


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream) if hasattr(stream, "cuda_stream") else int(stream)


def _ptr(t) -> int:
    return 0 if t is None else int(t.data_ptr())


def _i32(t: torch.Tensor, what: str, device_type: str) -> torch.Tensor:
    if not isinstance(t, torch.Tensor) or t.dtype != torch.int32:
        raise TypeError(f"{what} must be an int32 torch tensor")
    if t.device.type != device_type:
        raise ValueError(f"{what} must live on {device_type}, not {t.device}")
    if not t.is_contiguous():
        raise ValueError(f"{what} must be contiguous")
    return t


@dataclass
class Snapshot:
    """Handle returned by nbos_snapshot_create*; keeps the workspace and limit arrays alive."""
    handle: int
    n_snapshots: int
    n_hosts: int
    keep: tuple = ()

    def info(self) -> nbos_snapshot_info:
        return nbos_snapshot_get_info(self)


def _make_desc(n_snapshots, n_hosts, replicas_R, key_order, flags, limit_num, limit_den, arrays,
               device_type):
    if flags & NBOS_LIMIT_CLUSTER_SR and limit_num is None:
        ln = ld = None
    else:
        ln = _i32(limit_num, "limit_num", "cpu")
        ld = _i32(limit_den, "limit_den", "cpu")
        if ln.numel() != n_snapshots or ld.numel() != n_snapshots:
            raise ValueError("limit_num / limit_den need one entry per snapshot")
    arrs = []
    for name, a in zip(("gpus_total", "gpus_subscribed", "gpus_committed", "vram_gb", "millicpus",
                        "mem_mb"), arrays):
        a = _i32(a, name, device_type)
        if a.numel() != n_snapshots * n_hosts:
            raise ValueError(f"{name} must have n_snapshots * n_hosts elements")
        arrs.append(a)
    d = nbos_snapshot_desc(n_snapshots, n_hosts, replicas_R, key_order, flags, 0,
                           _ptr(ln), _ptr(ld), *[_ptr(a) for a in arrs])
    return d, (ln, ld, *arrs)


def nbos_snapshot_workspace_bytes(n_snapshots: int, n_hosts: int, flags: int = 0) -> int:
    d = nbos_snapshot_desc(n_snapshots, n_hosts, 3, 0, flags, 0, 0, 0, 0, 0, 0, 0, 0, 0)
    out = ctypes.c_size_t(0)
    _check(load_library().nbos_snapshot_workspace_bytes(ctypes.byref(d), ctypes.byref(out)))
    return int(out.value)


def nbos_snapshot_create(n_snapshots, n_hosts, limit_num, limit_den, gpus_total, gpus_subscribed,
                         gpus_committed, vram_gb, millicpus, mem_mb, replicas_R=3,
                         key_order=NBOS_KEY_IDLE_FIRST, flags=0, workspace=None,
                         stream=None) -> Snapshot:
    """Device arrays in, snapshot handle out. `workspace` is a uint8 CUDA tensor of at least
    nbos_snapshot_workspace_bytes(...) bytes; one is allocated with torch when omitted."""
    lib = load_library()
    arrays = (gpus_total, gpus_subscribed, gpus_committed, vram_gb, millicpus, mem_mb)
    d, keep = _make_desc(n_snapshots, n_hosts, replicas_R, key_order, flags, limit_num, limit_den,
                         arrays, "cuda")
    if workspace is None:
        workspace = torch.empty(nbos_snapshot_workspace_bytes(n_snapshots, n_hosts, flags),
                                dtype=torch.uint8, device=gpus_total.device)
    out = ctypes.c_void_p(0)
    _check(lib.nbos_snapshot_create(ctypes.byref(d), _ptr(workspace), workspace.numel(),
                                    _stream_ptr(stream), ctypes.byref(out)))
    return Snapshot(int(out.value), n_snapshots, n_hosts, keep=(workspace,) + keep)


def nbos_snapshot_create_host(n_snapshots, n_hosts, limit_num, limit_den, gpus_total,
                              gpus_subscribed, gpus_committed, vram_gb, millicpus, mem_mb,
                              replicas_R=3, key_order=NBOS_KEY_IDLE_FIRST, flags=0,
                              stream=None) -> Snapshot:
    """Host (CPU tensor) arrays in; the library stages them itself."""
    lib = load_library()
    arrays = (gpus_total, gpus_subscribed, gpus_committed, vram_gb, millicpus, mem_mb)
    d, keep = _make_desc(n_snapshots, n_hosts, replicas_R, key_order, flags, limit_num, limit_den,
                         arrays, "cpu")
    out = ctypes.c_void_p(0)
    _check(lib.nbos_snapshot_create_host(ctypes.byref(d), _stream_ptr(stream), ctypes.byref(out)))
    return Snapshot(int(out.value), n_snapshots, n_hosts)


def _update(fn_name, device_type, snap, limit_num, limit_den, arrays, stream):
    info = nbos_snapshot_get_info(snap)
    d, keep = _make_desc(snap.n_snapshots, snap.n_hosts, info.replicas_R, info.key_order, info.flags,
                         limit_num, limit_den, arrays, device_type)
    _check(getattr(load_library(), fn_name)(snap.handle, ctypes.byref(d), _stream_ptr(stream)))
    if device_type == "cuda":
        snap.keep = snap.keep[:1] + keep   # the queued kernels read the new arrays: keep them alive


def nbos_snapshot_update(snap: Snapshot, limit_num, limit_den, gpus_total, gpus_subscribed,
                         gpus_committed, vram_gb, millicpus, mem_mb, stream=None) -> None:
    """Refresh the snapshot from new device arrays of the same shape; asynchronous, no read-back.
    Problems with the new state show up in nbos_snapshot_status."""
    _update("nbos_snapshot_update", "cuda", snap, limit_num, limit_den,
            (gpus_total, gpus_subscribed, gpus_committed, vram_gb, millicpus, mem_mb), stream)


def nbos_snapshot_update_host(snap: Snapshot, limit_num, limit_den, gpus_total, gpus_subscribed,
                              gpus_committed, vram_gb, millicpus, mem_mb, stream=None) -> None:
    """Same from host (CPU tensor) arrays."""
    _update("nbos_snapshot_update_host", "cpu", snap, limit_num, limit_den,
            (gpus_total, gpus_subscribed, gpus_committed, vram_gb, millicpus, mem_mb), stream)


def nbos_snapshot_destroy(snap: Snapshot) -> None:
    if snap is not None and snap.handle:
        h, snap.handle = snap.handle, 0
        _check(load_library().nbos_snapshot_destroy(h))
        snap.keep = ()


def nbos_snapshot_get_info(snap: Snapshot) -> nbos_snapshot_info:
    info = nbos_snapshot_info()
    _check(load_library().nbos_snapshot_get_info(snap.handle, ctypes.byref(info)))
    return info


def nbos_snapshot_status(snap: Snapshot, stream=None) -> int:
    """Synchronises the stream; returns NBOS_OK or NBOS_ERR_DEVICE_TIMEOUT (does not raise)."""
    return int(load_library().nbos_snapshot_status(snap.handle, _stream_ptr(stream)))


def _batch_of(snap: Snapshot, requests: torch.Tensor) -> int:
    if requests.numel() % (4 * snap.n_snapshots):
        raise ValueError("requests must hold n_snapshots * batch * 4 values")
    return requests.numel() // (4 * snap.n_snapshots)


def nbos_place_batch(snap: Snapshot, requests, out_hosts, out_found=None, stream=None,
                     config: nbos_launch_config | None = None) -> None:
    """Device tensors: requests [N,B,4], out_hosts [N,B,3], out_found [N,B] or None. Asynchronous
    on the stream. `config` forwards to nbos_place_batch_ex."""
    lib = load_library()
    _i32(requests, "requests", "cuda")
    _i32(out_hosts, "out_hosts", "cuda")
    if out_found is not None:
        _i32(out_found, "out_found", "cuda")
    b = _batch_of(snap, requests)
    if out_hosts.numel() != snap.n_snapshots * b * 3:
        raise ValueError("out_hosts must hold n_snapshots * batch * 3 values")
    if out_found is not None and out_found.numel() != snap.n_snapshots * b:
        raise ValueError("out_found must hold n_snapshots * batch values")
    if config is None:
        _check(lib.nbos_place_batch(snap.handle, _ptr(requests), b, _ptr(out_hosts),
                                    _ptr(out_found), _stream_ptr(stream)))
    else:
        _check(lib.nbos_place_batch_ex(snap.handle, _ptr(requests), b, _ptr(out_hosts),
                                       _ptr(out_found), _stream_ptr(stream), ctypes.byref(config)))


def nbos_place_batch_ex(snap, requests, out_hosts, out_found=None, stream=None, config=None):
    nbos_place_batch(snap, requests, out_hosts, out_found, stream, config)


def _place_batch_host(name, snap, requests, out_hosts, out_found, stream):
    lib = load_library()
    _i32(requests, "requests", "cpu")
    _i32(out_hosts, "out_hosts", "cpu")
    if out_found is not None:
        _i32(out_found, "out_found", "cpu")
    b = _batch_of(snap, requests)
    if out_hosts.numel() != snap.n_snapshots * b * 3:
        raise ValueError("out_hosts must hold n_snapshots * batch * 3 values")
    if out_found is not None and out_found.numel() != snap.n_snapshots * b:
        raise ValueError("out_found must hold n_snapshots * batch values")
    _check(getattr(lib, name)(snap.handle, _ptr(requests), b, _ptr(out_hosts), _ptr(out_found),
                              _stream_ptr(stream)))


def nbos_place_batch_host(snap: Snapshot, requests, out_hosts, out_found=None, stream=None) -> None:
    """CPU tensors (pinned or not). Returns when the results are in `out_hosts` / `out_found`."""
    _place_batch_host("nbos_place_batch_host", snap, requests, out_hosts, out_found, stream)


def nbos_place_batch_host_async(snap: Snapshot, requests, out_hosts, out_found=None, stream=None) -> None:
    """CPU tensors (pinned, or the copies block). Returns once the work is queued; the results
    are in `out_hosts` / `out_found` after nbos_place_batch_host_wait. The caller keeps the three
    tensors alive and unchanged until then."""
    _place_batch_host("nbos_place_batch_host_async", snap, requests, out_hosts, out_found, stream)


def nbos_place_batch_host_wait(snap: Snapshot) -> None:
    """Blocks until every host-buffer call made so far on the snapshot's device has delivered."""
    _check(load_library().nbos_place_batch_host_wait(snap.handle))


def nbos_place_batch_noalloc(snap: Snapshot, requests, out_hosts, out_found=None, stream=None,
                             host_split: int = 0) -> None:
    """Same result as nbos_place_batch, for callers that must not allocate device memory (their
    GPU memory belongs to another pool, or an allocation's synchronisation does not fit their
    latency budget): the slice candidates live in a fixed array inside the library. This wrapper
    allocates nothing either; it only passes pointers. Calls that overlap on the GPU race on the
    shared array; batches beyond the array's size raise NbosError (NBOS_ERR_NO_MEMORY)."""
    lib = load_library()
    _i32(requests, "requests", "cuda")
    _i32(out_hosts, "out_hosts", "cuda")
    if out_found is not None:
        _i32(out_found, "out_found", "cuda")
    b = _batch_of(snap, requests)
    if out_hosts.numel() != snap.n_snapshots * b * 3:
        raise ValueError("out_hosts must hold n_snapshots * batch * 3 values")
    if out_found is not None and out_found.numel() != snap.n_snapshots * b:
        raise ValueError("out_found must hold n_snapshots * batch values")
    _check(lib.nbos_place_batch_noalloc(snap.handle, _ptr(requests), b, _ptr(out_hosts),
                                        _ptr(out_found), _stream_ptr(stream), host_split))


def nbos_select_executors(gpus_total, gpus_subscribed, gpus_committed, vram_gb, millicpus, mem_mb,
                          requests, replica_hosts, out_executor, out_can_run, replicas_R=3,
                          stream=None) -> None:
    """Device tensors: six state arrays [H], requests [M,4], replica_hosts [M,3], outputs [M]."""
    lib = load_library()
    arrs = [_i32(a, n, "cuda") for n, a in zip(("gpus_total", "gpus_subscribed", "gpus_committed",
                                                "vram_gb", "millicpus", "mem_mb"),
                                               (gpus_total, gpus_subscribed, gpus_committed, vram_gb,
                                                millicpus, mem_mb))]
    h = arrs[0].numel()
    if any(a.numel() != h for a in arrs):
        raise ValueError("the six cluster-state arrays must have the same length")
    for n, t in (("requests", requests), ("replica_hosts", replica_hosts),
                 ("out_executor", out_executor), ("out_can_run", out_can_run)):
        _i32(t, n, "cuda")
    m = requests.numel() // 4
    if requests.numel() != 4 * m or replica_hosts.numel() != 3 * m or out_executor.numel() != m \
            or out_can_run.numel() != m:
        raise ValueError("requests [M,4], replica_hosts [M,3], outputs [M] must agree on M")
    st = nbos_cluster_state(h, replicas_R, *[_ptr(a) for a in arrs])
    _check(lib.nbos_select_executors(ctypes.byref(st), _ptr(requests), _ptr(replica_hosts), m,
                                     _ptr(out_executor), _ptr(out_can_run), _stream_ptr(stream)))


def nbos_cluster_sums(gpus_total, gpus_subscribed, gpus_committed, n_snapshots, n_hosts, out_sums,
                      f_num=21, f_den=20, stream=None) -> None:
    """Device tensors [N*H] int32 in; out_sums [N,4] int64 = (sum G, sum S, sum C, auto-scaler sign)."""
    for n, t in (("gpus_total", gpus_total), ("gpus_subscribed", gpus_subscribed),
                 ("gpus_committed", gpus_committed)):
        _i32(t, n, "cuda")
        if t.numel() != n_snapshots * n_hosts:
            raise ValueError(f"{n} must have n_snapshots * n_hosts elements")
    if out_sums.dtype != torch.int64 or out_sums.numel() != 4 * n_snapshots or not out_sums.is_cuda:
        raise ValueError("out_sums must be a CUDA int64 tensor of n_snapshots * 4 elements")
    _check(load_library().nbos_cluster_sums(_ptr(gpus_total), _ptr(gpus_subscribed), _ptr(gpus_committed),
                                            n_snapshots, n_hosts, f_num, f_den, _ptr(out_sums),
                                            _stream_ptr(stream)))


def nbos_scale_out_deficit(found, n_snapshots, out_deficit, stream=None) -> None:
    """found [N,B] int32 (CUDA) in; out_deficit [N,2] int64 = (sum of 3 - found, requests short)."""
    _i32(found, "found", "cuda")
    if found.numel() % n_snapshots:
        raise ValueError("found must hold n_snapshots * batch values")
    if out_deficit.dtype != torch.int64 or out_deficit.numel() != 2 * n_snapshots or not out_deficit.is_cuda:
        raise ValueError("out_deficit must be a CUDA int64 tensor of n_snapshots * 2 elements")
    _check(load_library().nbos_scale_out_deficit(_ptr(found), n_snapshots, found.numel() // n_snapshots,
                                                 _ptr(out_deficit), _stream_ptr(stream)))


def nbos_place_batch_sequential(snap: Snapshot, requests, out_hosts, out_found=None,
                                out_subscribed=None, stream=None) -> None:
    """Device tensors as for nbos_place_batch, plus out_subscribed [N,H] int32 or None. The
    snapshot must have been created with NBOS_ROOM_FOR_COMMITS."""
    lib = load_library()
    _i32(requests, "requests", "cuda")
    _i32(out_hosts, "out_hosts", "cuda")
    for n, t in (("out_found", out_found), ("out_subscribed", out_subscribed)):
        if t is not None:
            _i32(t, n, "cuda")
    b = _batch_of(snap, requests)
    if out_hosts.numel() != snap.n_snapshots * b * 3:
        raise ValueError("out_hosts must hold n_snapshots * batch * 3 values")
    if out_found is not None and out_found.numel() != snap.n_snapshots * b:
        raise ValueError("out_found must hold n_snapshots * batch values")
    if out_subscribed is not None and out_subscribed.numel() != snap.n_snapshots * snap.n_hosts:
        raise ValueError("out_subscribed must hold n_snapshots * n_hosts values")
    _check(lib.nbos_place_batch_sequential(snap.handle, _ptr(requests), b, _ptr(out_hosts),
                                           _ptr(out_found), _ptr(out_subscribed), _stream_ptr(stream)))


def nbos_probe_int32_issue(mix: int, iters: int, blocks: int, threads: int, stream=None):
    """Returns (thread-level integer instructions, milliseconds)."""
    ops, ms = ctypes.c_double(0), ctypes.c_float(0)
    _check(load_library().nbos_probe_int32_issue(mix, iters, blocks, threads, _stream_ptr(stream),
                                                 ctypes.byref(ops), ctypes.byref(ms)))
    return float(ops.value), float(ms.value)


def nbos_probe_wait_timeout(limit_ns: int, stream=None):
    """Returns (mask of the warps whose wait ran out: 3 = both, 0 = none; milliseconds)."""
    gave_up, ms = ctypes.c_int(0), ctypes.c_float(0)
    _check(load_library().nbos_probe_wait_timeout(limit_ns, _stream_ptr(stream),
                                                  ctypes.byref(gave_up), ctypes.byref(ms)))
    return int(gave_up.value), float(ms.value)


def nbos_probe_wait_timeout_on_snapshot(snap: Snapshot, limit_ns: int, stream=None) -> float:
    """Runs the bounded-wait self-test so that it reports in `snap`'s status word; returns ms."""
    ms = ctypes.c_float(0)
    _check(load_library().nbos_probe_wait_timeout_on_snapshot(snap.handle, limit_ns, _stream_ptr(stream),
                                                              ctypes.byref(ms)))
    return float(ms.value)


def launch_config(lanes_per_request=0, requests_per_lane=0, host_split=0, tile_hosts=0,
                  grid_blocks=0, pair_mode=0, first_fit=0) -> nbos_launch_config:
    c = nbos_launch_config()
    c.lanes_per_request, c.requests_per_lane = lanes_per_request, requests_per_lane
    c.host_split, c.tile_hosts, c.grid_blocks = host_split, tile_hosts, grid_blocks
    c.pair_mode = pair_mode
    c.first_fit = first_fit
    return c


# ---- convenience on top of the ABI (still marshalling only) --------------------------------
def snapshot_from_workload(w, device="cuda", key_order=NBOS_KEY_IDLE_FIRST, flags=0,
                           stream=None) -> Snapshot:
    """Copy a generated workload's host state to the device and create a snapshot from it."""
    dev = [torch.from_numpy(getattr(w, k)).to(device).reshape(-1) for k in w.HOST_FIELDS]
    own = bool(flags & NBOS_LIMIT_CLUSTER_SR)
    return nbos_snapshot_create(w.n_snapshots, w.n_hosts, None if own else torch.from_numpy(w.limit_num),
                                None if own else torch.from_numpy(w.limit_den), *dev, replicas_R=w.replicas_R,
                                key_order=key_order, flags=flags, stream=stream)


def place_workload(w, key_order=NBOS_KEY_IDLE_FIRST, flags=0, config=None, device="cuda"):
    """Whole path on the device for a generated workload; returns CPU numpy (hosts, found)."""
    snap = snapshot_from_workload(w, device, key_order, flags)
    try:
        req = torch.from_numpy(w.requests).to(device)
        out = torch.empty((w.n_snapshots, w.batch, 3), dtype=torch.int32, device=device)
        found = torch.empty((w.n_snapshots, w.batch), dtype=torch.int32, device=device)
        nbos_place_batch(snap, req, out, found, config=config)
        status = nbos_snapshot_status(snap)
        if status != NBOS_OK:
            raise NbosError(status, nbos_strerror(status))
        return out.cpu().numpy(), found.cpu().numpy()
    finally:
        nbos_snapshot_destroy(snap)
