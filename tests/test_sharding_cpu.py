"""The multi-GPU path on CPU: two gloo ranks each place their slice of a batch (here with the CPU
checker standing in for the device, since this test runs without GPUs), results are gathered and
must equal the single-process answer; slice bounds tile the batch; timings reduce to the max."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2503_20591_b200 import sharding, workloads as W


def test_shard_bounds_tile_the_batch():
    for total in (0, 1, 31, 32, 33, 1000, 4096, 1_048_576, 1_000_003):
        for world in (1, 2, 3, 4, 8):
            prev = 0
            sizes = []
            for r in range(world):
                lo, hi = sharding.shard_bounds(total, r, world)
                assert lo == prev and lo <= hi <= total
                assert lo % sharding.ALIGN == 0 or lo == total
                sizes.append(hi - lo)
                prev = hi
            assert prev == total
            assert max(sizes) - min(sizes) <= sharding.ALIGN or total < world * sharding.ALIGN
    with pytest.raises(ValueError):
        sharding.shard_bounds(10, 2, 2)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, batch, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = W.make_config(2, batch=batch)          # every rank builds the same seeded workload
        lo, hi = sharding.shard_bounds(w.batch, rank, world)
        hosts, found = oracle.place_workload(w, request_slice=slice(lo, hi))
        full_h, full_f = sharding.gather_results(torch.from_numpy(hosts[0]), torch.from_numpy(found[0]),
                                                 w.batch)
        slowest = sharding.max_over_ranks(1.0 + rank)
        np.save(os.path.join(out_dir, f"hosts{rank}.npy"), full_h.numpy())
        np.save(os.path.join(out_dir, f"found{rank}.npy"), full_f.numpy())
        np.save(os.path.join(out_dir, f"slowest{rank}.npy"), np.array([slowest]))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("batch", [1000, 77])
def test_two_ranks_gather_the_single_process_answer(tmp_path, batch):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), batch, str(tmp_path)), nprocs=world, join=True)
    w = W.make_config(2, batch=batch)
    ref_h, ref_f = oracle.place_workload(w)
    for rank in range(world):
        np.testing.assert_array_equal(np.load(tmp_path / f"hosts{rank}.npy"), ref_h[0])
        np.testing.assert_array_equal(np.load(tmp_path / f"found{rank}.npy"), ref_f[0])
        assert np.load(tmp_path / f"slowest{rank}.npy")[0] == float(world)
