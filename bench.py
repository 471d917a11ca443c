#!/usr/bin/env python
"""Benchmark of batched replica placement on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
    python -m torch.distributed.run --nnodes=1 --nproc-per-node N ... bench.py --gpus N ...

One step = the whole path on one batch: snapshot derivation from the cluster-state arrays, then
the placement of every request of the batch (feasibility + key for every (request, host) pair,
best three hosts per request). Default workload: 4,096 hosts x 1,048,576 requests, the largest of
the five benchmark shapes. K steps are timed as one round (device events, barrier and
synchronisation on both sides, maximum over ranks); rounds repeat until a second of device time
has been measured, and the median round is reported. Prints ONE JSON line on rank 0.

`--impl reference` times the plain CPU checker (as it stands, one thread) on a bounded sample of
the same workload; it is a slow, deliberately simple program, reported for context.
"""
from __future__ import annotations

import argparse
import json
import os
import re
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

SM_COUNT_B200 = 148
ALU_LANES_PER_SM = 64             # integer ALU pipe: 16 lanes in each of the 4 scheduler partitions
IMAD_LANES_PER_SM = 64            # multiply pipe (32-bit integer multiply-add / subtract): 16 per partition
ALGORITHMIC_OPS_PER_PAIR = 6      # 4 capacity compares + 1 multiply-add (key) + 1 compare vs 3rd best
L2_BYTES = 126 * 1024 * 1024
# ncu summary of the placement kernel on the default workload. Its "bench-counters" block holds the
# figures that only a profiler can give (DRAM bytes and warp instructions per launch) together
# with the kernel time of the profiled build; they are reported only while this run's kernel time
# is within 5 % of that, i.e. while the profile still describes the kernel being timed.
PLACE_KERNEL_PROFILE = "profiles/place_kernel_ranked_cfg3_ncu.md"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=("ours", "reference"), default="ours")
    ap.add_argument("--workload", type=int, default=3,
                    help="benchmark workload index 0..4; 5 = 4,096 servers with 1..8 GPUs (not one of the five)")
    ap.add_argument("--batch", type=int, default=None, help="shrink the batch (profiling captures)")
    ap.add_argument("--snapshots", type=int, default=None, help="shrink workload 4")
    ap.add_argument("--min-timed-ms", type=float, default=1000.0,
                    help="repeat the round of --steps steps until this much device time is measured")
    ap.add_argument("--max-rounds", type=int, default=400)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-other-workloads", action="store_true",
                    help="skip the kernel timing + full checker comparison of the other benchmark shapes")
    ap.add_argument("--cpu-sample", type=int, default=None, help="requests in the timed CPU sample")
    ap.add_argument("--fresh-snapshot", action="store_true",
                    help="create a new snapshot in every step instead of refreshing one")
    ap.add_argument("--all-workloads", action="store_true",
                    help="also time first-fit, executor selection and sequential placement")
    ap.add_argument("--scaling", choices=("weak", "strong"), default="weak",
                    help="N > 1: every rank places its own full batch (weak) or one batch is cut over the ranks (strong)")
    ap.add_argument("--lanes", type=int, default=0,
                    help="force lanes per request (profiling a shrunk batch in the full batch's shape)")
    ap.add_argument("--pair-mode", type=int, default=0, help="force the pair evaluation form of the timed launch")
    return ap.parse_args()


# ------------------------------------------------------------------------------------------------
# clocks: sampled through NVML (read-only) from a thread while the timed region runs
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    REASONS = {
        0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap",
        0x8: "hw_slowdown", 0x10: "sync_boost", 0x20: "sw_thermal_slowdown",
        0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting",
    }

    def __init__(self, torch_device_index: int):
        self.samples, self.reason_bits, self.power = [], 0, []
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self._nv = pynvml
            uuid = str(torch.cuda.get_device_properties(torch_device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            try:
                self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            except TypeError:
                self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception as e:  # NVML missing: the JSON says so
            self.error = repr(e)

    def _poll(self):
        nv, h = self._nv, self._h
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)))
                try:
                    self.reason_bits |= int(nv.nvmlDeviceGetCurrentClocksEventReasons(h))
                except Exception:
                    self.reason_bits |= int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(h))
                self.power.append(nv.nvmlDeviceGetPowerUsage(h) / 1000.0)
            except Exception:
                pass
            time.sleep(0.004)

    def start(self):
        if self._h is not None:
            self.samples, self.reason_bits, self.power = [], 0, []
            self._stop.clear()
            self._thread = threading.Thread(target=self._poll, daemon=True)
            self._thread.start()

    def stop(self):
        if self._thread is not None:
            self._stop.set()
            self._thread.join()
            self._thread = None

    def summary(self):
        if self._h is None or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [],
                    "note": "NVML unavailable: " + getattr(self, "error", "no samples")}
        reasons = [name for bit, name in self.REASONS.items()
                   if self.reason_bits & bit and name != "gpu_idle"]
        return {"sm_mhz": statistics.median(self.samples), "sm_min_mhz": min(self.samples),
                "sm_max_mhz": self.max_mhz, "reasons": reasons, "samples": len(self.samples),
                "power_w_max": max(self.power) if self.power else None,
                "power_w_median": statistics.median(self.power) if self.power else None}


# ------------------------------------------------------------------------------------------------
# reference arm: the CPU checker on a bounded sample
# ------------------------------------------------------------------------------------------------
def time_checker(w, sample: int, steps: int, warmup: int):
    """Run the checker `warmup + steps` times over the first `sample` requests of every
    snapshot; returns (decisions per step, seconds per step, last result)."""
    import oracle
    sl = slice(0, sample)
    res = None
    for _ in range(warmup):
        res = oracle.place_workload(w, request_slice=sl)
    t0 = time.perf_counter()
    for _ in range(steps):
        res = oracle.place_workload(w, request_slice=sl)
    dt = (time.perf_counter() - t0) / max(1, steps)
    return w.n_snapshots * min(sample, w.batch), dt, res


def make_workload(W, args):
    if args.workload == 5:
        return W.mixed_gpu_cluster(4096, args.batch or (1 << 20), seed=5, name="mixed_gpu_counts_4096")
    return W.make_config(args.workload, batch=args.batch, n_snapshots=args.snapshots)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    from paper_2503_20591_b200 import workloads as W
    w = make_workload(W, args)
    # size the sample so that the whole run stays near a minute at ~25 M pairs/s per core
    budget_pairs = 60.0 * 25e6 / max(1, args.steps + args.warmup)
    sample = args.cpu_sample or int(budget_pairs / (w.n_snapshots * w.n_hosts))
    sample = max(16, min(w.batch, 1 << max(4, sample.bit_length() - 1)))
    dec, dt, _ = time_checker(w, sample, args.steps, args.warmup)
    value = dec / dt
    line = {
        "impl": "reference", "metric": "placement decisions/sec", "value": value,
        "unit": "decisions/s", "pairs_per_s": value * w.n_hosts, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int32",
        "data": "synthetic",
        "config": {"workload": w.name, "n_snapshots": w.n_snapshots, "n_hosts": w.n_hosts,
                   "batch": w.batch, "sample_requests_per_step": dec},
        "cpu_baseline": {"value": value, "unit": "decisions/s", "cores": 1, "kind": "oracle",
                         "sample": f"first {sample} requests of each snapshot against all "
                                   f"{w.n_hosts} hosts, per step"},
        "e2e": {"value": value, "unit": "decisions/s", "h2d_bytes_per_step": 0,
                "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


# ------------------------------------------------------------------------------------------------
# helpers of our arm
# ------------------------------------------------------------------------------------------------
def read_profile_counters(path: str):
    """The JSON object of the ```bench-counters fenced block of an ncu summary, or None."""
    try:
        text = open(os.path.join(ROOT, path)).read()
        m = re.search(r"```bench-counters\s*(\{.*?\})\s*```", text, re.S)
        return json.loads(m.group(1)) if m else None
    except Exception:
        return None


def time_launches(torch, stream, fn, reps: int, warm: int = 3):
    """Median and all per-launch times (ms, device events) of `fn(i)` over `reps` launches."""
    for i in range(warm):
        fn(i)
    torch.cuda.synchronize()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
    for i, (a, b) in enumerate(evs):
        a.record(stream)
        fn(i)
        b.record(stream)
    torch.cuda.synchronize()
    ms = [a.elapsed_time(b) for a, b in evs]
    return statistics.median(ms), ms


def workload_character(w, hosts: np.ndarray, found: np.ndarray, sample: int = 1024):
    """What the inputs and outputs look like, so that a reader can tell how much the pair
    evaluation has to do: how many hosts each request found, how many different answers the
    batch has, how often each test of Sections 3.2.1 / 3.4.1 rejects a (request, host) pair
    (sampled requests x all hosts, every test counted on its own), and how far into the key order
    the third chosen host lies."""
    out = {"found_histogram": np.bincount(found.ravel(), minlength=4).tolist()}
    flat = hosts.reshape(-1, 3).astype(np.int64) + 1            # -1 -> 0
    codes = (flat[:, 0] * (w.n_hosts + 1) + flat[:, 1]) * (w.n_hosts + 1) + flat[:, 2]
    if w.n_snapshots > 1:
        codes = codes + np.repeat(np.arange(w.n_snapshots, dtype=np.int64), w.batch) * (w.n_hosts + 1) ** 3
    out["distinct_output_triples"] = int(np.unique(codes).size)
    rng = np.random.default_rng(1)
    rej = np.zeros(6)
    feas = 0.0
    pos3 = []
    for n in range(min(w.n_snapshots, 8)):
        ids = rng.choice(w.batch, size=min(sample, w.batch), replace=False)
        r = w.requests[n][ids].astype(np.int64)
        G, S, C = (getattr(w, k)[n].astype(np.int64) for k in ("gpus_total", "gpus_subscribed", "gpus_committed"))
        tests = [r[:, 0:1] > G[None, :],
                 (S[None, :] + r[:, 0:1]) * int(w.limit_den[n]) > int(w.limit_num[n]) * G[None, :] * w.replicas_R,
                 r[:, 1:2] > w.vram_gb[n][None, :], r[:, 2:3] > w.millicpus[n][None, :],
                 r[:, 3:4] > w.mem_mb[n][None, :]]
        anyrej = np.zeros_like(tests[0])
        for k, t in enumerate(tests):
            rej[k] += t.mean()
            anyrej |= t
        rej[5] += 1
        feas += 1.0 - anyrej.mean()
        if len(np.unique(G)) == 1:   # one GPU count: hosts rank the same for every ask
            order = np.lexsort((np.arange(w.n_hosts), S, -(G - C)))
            rank = np.empty(w.n_hosts, dtype=np.int64)
            rank[order] = np.arange(w.n_hosts)
            third = hosts[n][:, 2]
            pos3.append(np.where(third >= 0, rank[np.maximum(third, 0)], w.n_hosts - 1))
    k = rej[5]
    out["pair_rejection_rates"] = {
        "gpus_over_server_total": rej[0] / k, "subscription_ratio_limit": rej[1] / k,
        "vram": rej[2] / k, "millicpus": rej[3] / k, "memory": rej[4] / k,
        "pairs_feasible": feas / k,
        "sample": f"{min(sample, w.batch)} requests x all hosts of {int(k)} snapshot(s); every test counted on its own"}
    if pos3:
        p = np.concatenate(pos3)
        out["third_host_position_in_key_order"] = {
            "mean_fraction_of_table": float((p + 1).mean() / w.n_hosts), "median": float(np.median(p)),
            "max": int(p.max()),
            "note": "position of a request's third chosen host when all hosts are sorted by (idle GPUs desc, "
                    "subscribed asc, id); a form that stops matching a request once it has three hosts "
                    "(pair_mode 4) has that fraction of its pairs live"}
    return out


# ------------------------------------------------------------------------------------------------
# our arm
# ------------------------------------------------------------------------------------------------
def run_ours(args):
    import torch
    from paper_2503_20591_b200 import binding as nb, build as lib_build, sharding, workloads as W

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    else:
        dist = None
        torch.cuda.set_device(0)
    dev = torch.device("cuda", torch.cuda.current_device())
    if rank == 0:
        lib_build.build()
    if dist is not None:
        dist.barrier()
    nb.load_library()

    # ---- inputs: one cluster snapshot per rank, several request batches rotated so that their
    # total exceeds the L2 cache. Weak scaling: every rank places its own full batch. Strong
    # scaling: the same batches on every rank, each rank places its slice of the flattened
    # request list (single-snapshot workloads) ----
    w = make_workload(W, args)
    strong = args.scaling == "strong" and world > 1
    if strong and w.n_snapshots != 1:
        raise SystemExit("--scaling strong cuts the batch of a single-snapshot workload")
    per_batch_bytes = w.decisions * (16 + 12 + 4)
    n_rot = max(2, min(12, -(-int(1.3 * L2_BYTES) // per_batch_bytes)))
    own_first = rank == 0 or strong
    batches = [w.requests] if own_first else []
    if args.workload == 5:
        batches += [W.mixed_gpu_cluster(w.n_hosts, w.batch, seed=50 + k + (0 if strong else 100 * rank)).requests
                    for k in range(n_rot - len(batches))]
    else:
        batches += W.extra_request_batches(args.workload, n_rot - len(batches), batch=w.batch,
                                           n_snapshots=w.n_snapshots, seed0=10_000 + (0 if strong else 1000 * rank))
    lo, hi = sharding.shard_bounds(w.batch, rank, world) if strong else (0, w.batch)
    my_batch = hi - lo
    d_state = [torch.from_numpy(getattr(w, k)).to(dev).reshape(-1) for k in w.HOST_FIELDS]
    lim_num, lim_den = torch.from_numpy(w.limit_num), torch.from_numpy(w.limit_den)
    d_req = [torch.from_numpy(np.ascontiguousarray(b[:, lo:hi])).to(dev) for b in batches]
    d_out = [torch.empty((w.n_snapshots, my_batch, 3), dtype=torch.int32, device=dev) for _ in batches]
    d_found = [torch.empty((w.n_snapshots, my_batch), dtype=torch.int32, device=dev) for _ in batches]
    workspace = torch.empty(nb.nbos_snapshot_workspace_bytes(w.n_snapshots, w.n_hosts),
                            dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()
    launch_cfg = (nb.launch_config(lanes_per_request=args.lanes, pair_mode=args.pair_mode)
                  if (args.lanes or args.pair_mode) else None)

    # The snapshot object is created once; every step refreshes it from the cluster-state arrays
    # (all derivation kernels run again, nothing is read back) and places one batch. With
    # --fresh-snapshot every step creates a new snapshot instead (one host synchronisation each).
    live = None if args.fresh_snapshot else nb.nbos_snapshot_create(
        w.n_snapshots, w.n_hosts, lim_num, lim_den, *d_state, replicas_R=w.replicas_R,
        workspace=workspace, stream=stream)

    def step(i, ev=None):
        if live is None:
            snap = nb.nbos_snapshot_create(w.n_snapshots, w.n_hosts, lim_num, lim_den, *d_state,
                                           replicas_R=w.replicas_R, workspace=workspace, stream=stream)
        else:
            snap = live
            nb.nbos_snapshot_update(snap, lim_num, lim_den, *d_state, stream=stream)
        k = i % n_rot
        if ev is not None:
            ev[0].record(stream)
        nb.nbos_place_batch(snap, d_req[k], d_out[k], d_found[k], stream=stream, config=launch_cfg)
        if ev is not None:
            ev[1].record(stream)
        return snap

    def sync_all():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    def max_over_ranks(ms):
        if dist is None:
            return ms
        t = torch.tensor([ms], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    sampler = ClockSampler(dev.index)
    warmup = max(3, args.warmup)
    snaps = [step(i) for i in range(warmup)]
    sync_all()
    if live is None:
        for s in snaps:
            nb.nbos_snapshot_destroy(s)

    # ---- timed rounds of exactly --steps steps each ----
    kern_events = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                   for _ in range(args.steps)]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    round_ms, kern_ms_all = [], []
    last_snap = live
    sampler.start()
    while True:
        snaps = []
        e0.record(stream)
        for i in range(args.steps):
            snaps.append(step(i, kern_events[i]))
        e1.record(stream)
        sync_all()
        round_ms.append(max_over_ranks(e0.elapsed_time(e1)))
        if len(kern_ms_all) < 20000:
            kern_ms_all += [a.elapsed_time(b) for a, b in kern_events]
        if live is None:
            for s in snaps[:-1]:
                nb.nbos_snapshot_destroy(s)
            if last_snap is not None:
                nb.nbos_snapshot_destroy(last_snap)
        last_snap = snaps[-1]
        if sum(round_ms) >= args.min_timed_ms or len(round_ms) >= args.max_rounds:
            break
    sampler.stop()
    status = nb.nbos_snapshot_status(last_snap, stream)
    if status != nb.NBOS_OK:
        raise RuntimeError("device status: " + nb.nbos_strerror(status))
    ms_per_step = statistics.median(round_ms) / args.steps
    kern_ms = statistics.median(kern_ms_all)
    decisions_all = w.n_snapshots * my_batch if not strong else w.decisions
    if not strong:
        decisions_all *= world
    value = decisions_all / (ms_per_step * 1e-3)
    clocks = sampler.summary()
    # the output of the timed launch on the first batch (rank 0: the workload's own requests),
    # taken before anything else writes the result buffers
    got_hosts = d_out[0].cpu().numpy()
    got_found = d_found[0].cpu().numpy()
    info = nb.nbos_snapshot_get_info(last_snap)

    # ---- the same launch in the other pair-evaluation forms (own output buffers) ----
    forms = None
    if rank == 0:
        forms = {}
        alt_out, alt_found = torch.empty_like(d_out[0]), torch.empty_like(d_found[0])
        for name, pm in (("key_compared_per_pair_with_counter", 3), ("retiring_key_order", 4)):
            cfg_alt = nb.launch_config(lanes_per_request=args.lanes, pair_mode=pm)
            nb.nbos_place_batch(last_snap, d_req[0], alt_out, alt_found, stream=stream, config=cfg_alt)
            same = bool(torch.equal(alt_out, d_out[0]) and torch.equal(alt_found, d_found[0]))
            scratch_out, scratch_found = torch.empty_like(d_out[0]), torch.empty_like(d_found[0])
            med, _ = time_launches(torch, stream, lambda i: nb.nbos_place_batch(
                last_snap, d_req[i % n_rot], scratch_out, scratch_found, stream=stream, config=cfg_alt), 20)
            forms[name] = {"pair_mode": pm, "kernel_ms": med, "pairs_per_s": w.n_hosts * w.n_snapshots * my_batch / (med * 1e-3),
                           "same_output_as_timed_launch": same}

    # creation on its own, for the record (one host synchronisation inside)
    t0 = time.perf_counter()
    for _ in range(10):
        nb.nbos_snapshot_destroy(nb.nbos_snapshot_create(
            w.n_snapshots, w.n_hosts, lim_num, lim_den, *d_state, replicas_R=w.replicas_R, stream=stream))
    torch.cuda.synchronize()
    create_ms = (time.perf_counter() - t0) / 10 * 1e3
    nb.nbos_snapshot_destroy(last_snap)

    # ---- end to end: host buffers in, host buffers out, through the *_host entry points ----
    e2e = None
    if not args.no_e2e:
        h_state = [torch.from_numpy(getattr(w, k)).reshape(-1).pin_memory() for k in w.HOST_FIELDS]
        h_req = [torch.from_numpy(np.ascontiguousarray(b[:, lo:hi])).pin_memory() for b in batches[:2]]
        h_out = [torch.empty((w.n_snapshots, my_batch, 3), dtype=torch.int32).pin_memory() for _ in range(2)]
        h_found = [torch.empty((w.n_snapshots, my_batch), dtype=torch.int32).pin_memory() for _ in range(2)]

        e2e_live = None if args.fresh_snapshot else nb.nbos_snapshot_create_host(
            w.n_snapshots, w.n_hosts, lim_num, lim_den, *h_state, replicas_R=w.replicas_R, stream=stream)

        def e2e_step(i, blocking):
            if e2e_live is None:
                snap = nb.nbos_snapshot_create_host(w.n_snapshots, w.n_hosts, lim_num, lim_den,
                                                    *h_state, replicas_R=w.replicas_R, stream=stream)
            else:
                snap = e2e_live
                nb.nbos_snapshot_update_host(snap, lim_num, lim_den, *h_state, stream=stream)
            place = nb.nbos_place_batch_host if (blocking or e2e_live is None) else nb.nbos_place_batch_host_async
            place(snap, h_req[i % 2], h_out[i % 2], h_found[i % 2], stream=stream)
            if e2e_live is None:
                nb.nbos_snapshot_destroy(snap)

        e2e_steps = max(3, min(args.steps, 50))

        def e2e_time(blocking):
            for i in range(3):
                e2e_step(i, blocking)
            if not blocking and e2e_live is not None:
                nb.nbos_place_batch_host_wait(e2e_live)
            sync_all()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            rounds = []
            while True:
                a.record(stream)
                for i in range(e2e_steps):
                    e2e_step(i, blocking)
                if not blocking and e2e_live is not None:
                    nb.nbos_place_batch_host_wait(e2e_live)    # the last results are in the host buffers
                b.record(stream)
                sync_all()
                rounds.append(max_over_ranks(a.elapsed_time(b)))
                if sum(rounds) >= 0.5 * args.min_timed_ms or len(rounds) >= args.max_rounds:
                    break
            return statistics.median(rounds) / e2e_steps, len(rounds)

        blocking_ms, blocking_rounds = e2e_time(True)
        e2e_ms, e2e_rounds = e2e_time(False)
        # what the last two queued steps left in the host buffers against the device path on the same requests
        same = True
        chk = e2e_live if e2e_live is not None else nb.nbos_snapshot_create_host(
            w.n_snapshots, w.n_hosts, lim_num, lim_den, *h_state, replicas_R=w.replicas_R, stream=stream)
        for k in range(2):
            d_req_k = h_req[k].to(dev)
            d_out_k = torch.empty((w.n_snapshots, my_batch, 3), dtype=torch.int32, device=dev)
            d_found_k = torch.empty((w.n_snapshots, my_batch), dtype=torch.int32, device=dev)
            nb.nbos_place_batch(chk, d_req_k, d_out_k, d_found_k, stream=stream)
            sync_all()
            same = same and bool(torch.equal(d_out_k.cpu(), h_out[k])) and bool(torch.equal(d_found_k.cpu(), h_found[k]))
        h2d = w.n_snapshots * my_batch * 16 + 6 * 4 * w.n_snapshots * w.n_hosts + 8 * w.n_snapshots
        d2h = w.n_snapshots * my_batch * (12 + 4)
        nb.nbos_snapshot_destroy(chk)
        e2e = {"value": decisions_all / (e2e_ms * 1e-3), "unit": "decisions/s",
               "ms_per_step": e2e_ms, "steps": e2e_steps, "rounds": e2e_rounds,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "host_memory": "pinned",
               "mode": ("every step = nbos_snapshot_update_host + nbos_place_batch_host_async from and to pinned host "
                        "buffers (two request / result buffer sets in turn); steps are queued without waiting in "
                        "between, so the copies in of one step run beside the kernels and copies out of the step "
                        "before; the timed region ends after nbos_place_batch_host_wait, so all copies of all timed steps lie inside it"
                        if e2e_live is not None else "fresh snapshot per step, blocking calls"),
               "blocking_call": {"value": decisions_all / (blocking_ms * 1e-3), "ms_per_step": blocking_ms,
                                 "rounds": blocking_rounds,
                                 "note": "nbos_place_batch_host: returns with the results in the host buffers, "
                                         "one step at a time (the latency of a step)"},
               "output_identical_to_device_path": same}

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return 0

    # ---- integer issue-rate probe, same process, same clocks ----
    probe = {}
    for name, mix in (("alu", nb.NBOS_PROBE_MIX_ALU), ("imad", nb.NBOS_PROBE_MIX_IMAD),
                      ("both", nb.NBOS_PROBE_MIX_BOTH)):
        nb.nbos_probe_int32_issue(mix, 2048, SM_COUNT_B200 * 8, 256)
        ops, ms = nb.nbos_probe_int32_issue(mix, 8192, SM_COUNT_B200 * 8, 256)
        probe[name + "_gops"] = ops / ms / 1e6

    my_pairs = w.n_hosts * w.n_snapshots * my_batch
    sm_mhz = clocks.get("sm_mhz") or clocks.get("sm_max_mhz") or 1965.0
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    peak_gops = sms * (ALU_LANES_PER_SM + IMAD_LANES_PER_SM) * sm_mhz * 1e6 / 1e9
    achieved_gops = ALGORITHMIC_OPS_PER_PAIR * my_pairs / (kern_ms * 1e-3) / 1e9
    # counters that only a profiler gives: reported while the profiled build's kernel time still
    # matches this run's
    prof = read_profile_counters(PLACE_KERNEL_PROFILE) if (args.workload == 3 and args.batch is None
                                                           and not args.pair_mode and not args.lanes and not strong) else None
    prof_ok = bool(prof) and abs(kern_ms - prof["kernel_ms"]) <= 0.05 * prof["kernel_ms"]
    instr = prof["warp_instructions_per_32_pairs"] if prof_ok else None
    roofline = {
        "bound": "alu", "kernel": "place_kernel", "achieved": achieved_gops, "peak": peak_gops,
        "unit": "Gop/s (thread-level INT32 operations)", "frac": achieved_gops / peak_gops,
        "peak_source": f"integer issue rate of both integer-capable pipes (= one warp instruction per scheduler "
                       f"per clock): {sms} SMs x ({ALU_LANES_PER_SM} ALU + {IMAD_LANES_PER_SM} multiply-pipe lanes) x "
                       f"{sm_mhz:.0f} MHz sampled during the timed region; probe_both_gops is this "
                       "peak measured in the same process, probe_alu_gops / probe_imad_gops each pipe alone",
        "pair_evaluation": ("ranked form: every (request, host) pair is tested against its own request -- the four "
                            "capacities and the host's rank against the request's current third best -- by one packed 32-bit "
                            "subtraction and one logic operation (a second, finer level and the exact test only for "
                            "the few pairs that pass); no request is ever switched off"
                            if (info.ranked and not args.pair_mode) else f"pair_mode {args.pair_mode}"),
        "note": "achieved counts the 6 algorithmic operations of a pair (4 capacity compares, key multiply-add, "
                "compare with the third best). The kernel executes fewer instructions per pair than that "
                "(warp_instructions_per_32_pairs): the five compares share one packed subtraction and its "
                "guard test, and the key is the host's precomputed rank. So frac can exceed 1; issue_slot_frac is the executed-instruction view "
                "of the same launch (warp instructions issued / issue slots)",
        "ops_per_pair": ALGORITHMIC_OPS_PER_PAIR, "kernel_ms": kern_ms,
        "kernel_ms_min": min(kern_ms_all), "kernel_launches_timed": len(kern_ms_all),
        "pairs_per_s_kernel": my_pairs / (kern_ms * 1e-3),
        "issue_slot_frac": (instr * my_pairs / 32 / (kern_ms * 1e-3) / (sms * 4 * sm_mhz * 1e6)) if instr else None,
        "warp_instructions_per_32_pairs": instr,
        "traffic": prof["dram_bytes_per_launch"] if prof_ok else None,
        "source": ({"file": PLACE_KERNEL_PROFILE, "kernel_ms_profiled_build": prof["kernel_ms"],
                    "fields": ["traffic", "warp_instructions_per_32_pairs", "issue_slot_frac"],
                    "matches_this_run": prof_ok} if prof else None),
        "algorithmic_bytes": w.n_snapshots * my_batch * (16 + 12 + 4),
        "stream_gbs": w.n_snapshots * my_batch * (16 + 12 + 4) / (kern_ms * 1e-3) / 1e9,
        "probe_alu_gops": probe["alu_gops"], "probe_imad_gops": probe["imad_gops"],
        "probe_both_gops": probe["both_gops"],
        "other_forms": forms,
    }

    # ---- CPU checker: timed on one core on a bounded sample; then run over the whole batch on all
    # cores (not timed) and compared byte for byte with the output of the timed launch ----
    cpu_baseline = None
    if not args.no_cpu_baseline:
        import oracle
        sample = args.cpu_sample or max(16, min(w.batch, (1 << 30) // (w.n_snapshots * w.n_hosts)))
        dec, dt, res = time_checker(w, sample, 1, 0)
        cores = os.cpu_count() or 1
        t0 = time.perf_counter()
        if sample >= w.batch:
            ref = res
        else:
            ref = oracle.place_workload(w, threads=cores)
        full_s = time.perf_counter() - t0
        ref_hosts, ref_found = ref[0][:, lo:hi], ref[1][:, lo:hi]
        same = bool(np.array_equal(ref_hosts, got_hosts) and np.array_equal(ref_found, got_found))
        cpu_baseline = {"value": dec / dt, "unit": "decisions/s", "pairs_per_s": dec * w.n_hosts / dt,
                        "cores": 1, "host_cores_available": cores, "kind": "oracle",
                        "seconds": dt,
                        "sample": f"first {sample} requests of each snapshot against all "
                                  f"{w.n_hosts} hosts, once, one thread",
                        "gpu_output_identical": same,
                        "compared_requests": int(ref_found.size),
                        "compared_with": "the output of the timed launch on the workload's own batch; the checker "
                                         f"ran over the whole batch on {cores} threads for this ({full_s:.1f} s, not timed as a baseline)"}
    character = workload_character(w, got_hosts, got_found) if not strong else None

    # ---- the other benchmark shapes: placement kernel only, each compared in full with the checker ----
    others = None
    if not args.no_other_workloads:
        others = {}
        shapes = [W.make_config(idx) for idx in range(5) if idx != args.workload or args.batch is not None]
        # not one of the five: servers with 1..8 GPUs, so that the ranking depends on the ask
        if args.all_workloads and args.workload != 5:
            shapes.append(W.mixed_gpu_cluster(4096, 1 << 20, seed=5, name="mixed_gpu_counts_4096"))
        for ww in shapes:
            sn = nb.snapshot_from_workload(ww, device=dev)
            rq = torch.from_numpy(ww.requests).to(dev)
            oh = torch.empty((ww.n_snapshots, ww.batch, 3), dtype=torch.int32, device=dev)
            of = torch.empty((ww.n_snapshots, ww.batch), dtype=torch.int32, device=dev)
            ms, _ = time_launches(torch, stream, lambda i: nb.nbos_place_batch(sn, rq, oh, of, stream=stream), 20)
            inf = sn.info()
            entry = {"kernel_ms": ms, "decisions_per_s": ww.decisions / ms * 1e3,
                     "pairs_per_s": ww.pairs / ms * 1e3,
                     "frac": ALGORITHMIC_OPS_PER_PAIR * ww.pairs / (ms * 1e-3) / 1e9 / peak_gops,
                     "ranked": inf.ranked, "packed_test": inf.packed_test, "static_key": inf.static_key,
                     "grouped": inf.grouped,
                     "note": "same inputs every launch (L2-resident), median of 20 launches"}
            oh_np, of_np = oh.cpu().numpy(), of.cpu().numpy()
            entry.update(workload_character(ww, oh_np, of_np))
            if not args.no_cpu_baseline and ww.pairs <= (1 << 31):
                import oracle
                ref = oracle.place_workload(ww, threads=os.cpu_count() or 1)
                entry["gpu_output_identical"] = bool(np.array_equal(ref[0], oh_np) and np.array_equal(ref[1], of_np))
                entry["compared_requests"] = int(of_np.size)
            if args.all_workloads:
                # first-fit variant (stops at the third feasible host): decisions/s only
                ff = nb.launch_config(first_fit=1)
                oh2 = torch.empty_like(oh)
                ms_ff, _ = time_launches(torch, stream, lambda i: nb.nbos_place_batch(sn, rq, oh2, of, stream=stream, config=ff), 20)
                entry.update({"first_fit_kernel_ms": ms_ff,
                              "first_fit_decisions_per_s": ww.decisions / ms_ff * 1e3,
                              "first_fit_same_output": bool(torch.equal(oh, oh2))})
            others[ww.name] = entry
            nb.nbos_snapshot_destroy(sn)

    if args.all_workloads:
        # executor selection (Section 3.2.2): HBM-bound gather kernel, 36 algorithmic bytes per kernel
        w1 = W.make_config(3)
        m = 16 * 1024 * 1024
        g = torch.Generator(device="cpu").manual_seed(11)
        rep = torch.randint(0, w1.n_hosts, (m, 3), generator=g, dtype=torch.int32).to(dev)
        gq = torch.randint(0, 9, (m,), generator=g, dtype=torch.int32)
        rq = torch.stack([gq, 16 * gq, torch.randint(1000, 16001, (m,), generator=g, dtype=torch.int32),
                          torch.randint(1024, 65537, (m,), generator=g, dtype=torch.int32)], dim=1).contiguous().to(dev)
        st = [torch.from_numpy(getattr(w1, k)[0]).to(dev) for k in w1.HOST_FIELDS]
        ex = torch.empty((m,), dtype=torch.int32, device=dev)
        mk = torch.empty((m,), dtype=torch.int32, device=dev)
        ms, _ = time_launches(torch, stream, lambda i: nb.nbos_select_executors(*st, rq, rep, ex, mk, stream=stream), 20)
        peak_hbm, peak_kind = 6650.0, "fallback"
        try:
            peak_hbm, peak_kind = float(json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))["hbm_gbs"]), "measured"
        except Exception:
            pass
        gbs = m * 36 / (ms * 1e-3) / 1e9
        others["executor_selection"] = {
            "kernels": m, "hosts": w1.n_hosts, "kernel_ms": ms, "kernels_per_s": m / ms * 1e3,
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": peak_hbm, "unit": "GB/s",
                         "frac": gbs / peak_hbm, "peak_source": f"copy bandwidth, {peak_kind}",
                         "algorithmic_bytes_per_kernel": 36},
            "designated": int((ex >= 0).sum().item()), "all_yield": int((ex < 0).sum().item()),
            "note": "inputs + outputs 576 MiB, larger than L2; median of 20 calls"}

        # sequential placement with commits: serial over requests, parallel over hosts / snapshots
        for label, ww in (("sequential_cfg4_shape", W.make_config(4)),
                          ("sequential_one_snapshot_4096_hosts", W.make_config(3, batch=65_536)),
                          ("sequential_one_snapshot_32768_hosts_block_cluster", W.uniform_cluster(32_768, 4096, seed=1))):
            sn = nb.snapshot_from_workload(ww, device=dev, flags=nb.NBOS_ROOM_FOR_COMMITS)
            rq = torch.from_numpy(ww.requests).to(dev)
            oh = torch.empty((ww.n_snapshots, ww.batch, 3), dtype=torch.int32, device=dev)
            of = torch.empty((ww.n_snapshots, ww.batch), dtype=torch.int32, device=dev)
            ms, _ = time_launches(torch, stream, lambda i: nb.nbos_place_batch_sequential(sn, rq, oh, of, stream=stream), 3, warm=1)
            others[label] = {"n_snapshots": ww.n_snapshots, "n_hosts": ww.n_hosts, "batch": ww.batch,
                             "kernel_ms": ms, "decisions_per_s": ww.decisions / ms * 1e3,
                             "us_per_request_per_snapshot": ms * 1e3 / ww.batch,
                             "kernels_created": int((of == 3).sum().item())}
            nb.nbos_snapshot_destroy(sn)

    rot_mib = n_rot * w.n_snapshots * my_batch * 32 / 2**20
    launches_per_step = 3  # emit (+ validation), rank + finalize (snapshot refresh), placement
    line = {
        "metric": "placement decisions/sec", "value": value, "unit": "decisions/s",
        "pairs_per_s": value * w.n_hosts, "n_gpus": world, "steps": args.steps,
        "warmup": warmup, "rounds": len(round_ms), "timed_ms_total": sum(round_ms),
        "ms_per_step": ms_per_step, "ms_per_step_min_max": [min(round_ms) / args.steps, max(round_ms) / args.steps],
        "higher_is_better": True,
        "scaling": args.scaling if world > 1 else "weak", "vs_baseline": None, "dtype": "int32", "data": "synthetic",
        "config": {"workload": w.name, "n_snapshots": w.n_snapshots, "n_hosts": w.n_hosts,
                   "batch": w.batch, "batch_per_gpu": my_batch, "pairs_per_step_per_gpu": my_pairs,
                   "replicas_R": w.replicas_R,
                   "step": ("snapshot creation (derivation, one host synchronisation) + placement of one batch"
                            if args.fresh_snapshot else
                            "snapshot refresh (all derivation kernels, no read-back) + placement of one batch"),
                   "timing": f"rounds of {args.steps} steps, each bracketed by barrier + synchronise, repeated until "
                             f"{args.min_timed_ms:.0f} ms of device time; ms_per_step is the median round / steps",
                   "snapshot_create_ms": create_ms,
                   "l2": f"inputs rotate over {n_rot} request/result batch sets, {rot_mib:.0f} MiB "
                         f"in total ({'larger' if rot_mib > 126 else 'SMALLER'} than the 126 MiB L2)",
                   "inputs_sha256": w.sha256()},
        "roofline": roofline, "cpu_baseline": cpu_baseline, "e2e": e2e,
        "gpu_launches": launches_per_step * args.steps * len(round_ms), "clocks": clocks,
        "workload_character": character,
    }
    if others is not None:
        line["other_workloads_kernel_only"] = others
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0


def main():
    args = parse_args()
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
