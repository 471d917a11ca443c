"""Multi-GPU use: requests are independent, so a batch is cut across ranks and every rank places
its own slice against its own copy of the (small) snapshot. No collective is on the data path;
`torch.distributed` only gathers results for callers that want them everywhere and reduces
timings. This module holds the bookkeeping, none of the placement arithmetic."""
from __future__ import annotations

import torch
import torch.distributed as dist

ALIGN = 32  # slice starts stay on 512-byte lines of the 16-byte request records


def shard_bounds(total: int, rank: int, world: int, align: int = ALIGN) -> tuple[int, int]:
    """Half-open range [lo, hi) of the flattened request list that `rank` of `world` handles.
    Ranges tile [0, total) exactly, differ by at most `align`, and start on multiples of `align`."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    units = -(-total // align)
    lo = min(total, (units * rank // world) * align)
    hi = min(total, (units * (rank + 1) // world) * align)
    return lo, hi


def gather_results(local_hosts: torch.Tensor, local_found: torch.Tensor, total: int, group=None):
    """All-gather per-rank results ([n_local, 3] and [n_local]) into full [total, 3] / [total]
    tensors on every rank. Works with any backend (gloo on CPU tensors, NCCL on CUDA tensors)."""
    world = dist.get_world_size(group)
    sizes = [shard_bounds(total, r, world) for r in range(world)]
    width = max(hi - lo for lo, hi in sizes)
    pad_h = torch.full((width, 3), -1, dtype=local_hosts.dtype, device=local_hosts.device)
    pad_f = torch.zeros((width,), dtype=local_found.dtype, device=local_found.device)
    pad_h[: local_hosts.shape[0]] = local_hosts
    pad_f[: local_found.shape[0]] = local_found
    all_h = [torch.empty_like(pad_h) for _ in range(world)]
    all_f = [torch.empty_like(pad_f) for _ in range(world)]
    dist.all_gather(all_h, pad_h, group=group)
    dist.all_gather(all_f, pad_f, group=group)
    hosts = torch.cat([all_h[r][: hi - lo] for r, (lo, hi) in enumerate(sizes)])
    found = torch.cat([all_f[r][: hi - lo] for r, (lo, hi) in enumerate(sizes)])
    return hosts, found


def max_over_ranks(value: float, device="cpu", group=None) -> float:
    """The slowest rank's time: what a multi-GPU measurement reports."""
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(t.item())
