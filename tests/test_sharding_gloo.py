"""N > 1 plumbing on CPU: two gloo ranks shard independent (batch, KV head) units and reduce their timing the
way bench.py does (max of the step time, sum of the units)."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2605_18753_b200.shard import combine_timing, shard_range


def test_shard_range_is_a_balanced_partition():
    for n in (0, 1, 7, 8, 128, 129):
        for world in (1, 2, 3, 8):
            parts = [list(shard_range(n, world, r)) for r in range(world)]
            assert sum(parts, []) == list(range(n))
            assert max(len(p) for p in parts) - min(len(p) for p in parts) <= 1


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    units = shard_range(16 * 8, world, rank)           # 16 sequences x 8 KV heads
    ms, tot = combine_timing(1.0 + rank, float(len(units)))
    out[rank] = (ms, tot, len(units))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_reduce_time_by_max_and_units_by_sum():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    assert out[0][:2] == out[1][:2] == (2.0, 128.0)
    assert out[0][2] + out[1][2] == 128


def test_single_process_passthrough():
    assert combine_timing(3.5, 10.0) == (3.5, 10.0)
