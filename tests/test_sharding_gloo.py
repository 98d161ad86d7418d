"""World-size-2 checks of the multi-GPU host logic on CPU (gloo)."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2602_02711_b200 import sharding


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        b, e = sharding.shard_range(65, rank, world)
        t = 1.0 + rank  # rank 1 is slower
        units = float(e - b)
        sharding.barrier()
        res = {
            "range": (b, e),
            "max": sharding.max_over_ranks(t),
            "sum": sharding.sum_over_ranks(units),
            "tp": sharding.job_throughput(units, t),
        }
        out[rank] = res
    finally:
        dist.destroy_process_group()


def test_two_rank_reductions_and_shards():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    assert out[0]["range"] == (0, 33) and out[1]["range"] == (33, 65)
    for r in range(world):
        assert out[r]["max"] == 2.0
        assert out[r]["sum"] == 65.0
        assert out[r]["tp"] == 65.0 / 2.0


@pytest.mark.parametrize("total,world", [(0, 1), (1, 4), (64, 8), (65, 8), (7, 3)])
def test_shard_ranges_partition_the_rows(total, world):
    parts = [sharding.shard_range(total, r, world) for r in range(world)]
    assert parts[0][0] == 0 and parts[-1][1] == total
    for a, b in zip(parts, parts[1:]):
        assert a[1] == b[0]
    sizes = [e - b for b, e in parts]
    assert max(sizes) - min(sizes) <= 1


def test_single_process_reductions_are_identity():
    assert sharding.max_over_ranks(3.5) == 3.5
    assert sharding.job_throughput(10.0, 2.0) == 5.0
