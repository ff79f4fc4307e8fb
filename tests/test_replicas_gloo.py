"""The multi-GPU path is "replicas only": no data-path collective, only the split of work items
and the max-over-ranks of the timings.  Covered here with two gloo ranks on CPU."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2512_24545_b200 import replicas


def test_shard_units_partitions_everything():
    for n in (0, 1, 7, 128):
        for world in (1, 2, 3, 8):
            parts = [replicas.shard_units(n, r, world) for r in range(world)]
            flat = [i for p in parts for i in p]
            assert flat == list(range(n))
            assert max(len(p) for p in parts) - min(len(p) for p in parts) <= 1
    with pytest.raises(ValueError):
        replicas.shard_units(4, 2, 2)


def test_single_process_aggregation():
    assert replicas.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert replicas.aggregate_throughput(10.0, 4, 2.0) == 20.0
    with pytest.raises(ValueError):
        replicas.aggregate_throughput(1.0, 1, 0.0)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = replicas.shard_units(7, rank, world)
        ms_local = 10.0 + 5.0 * rank                  # rank 1 is the slow replica
        ms_max, e2e_max = replicas.max_over_ranks([ms_local, 100.0 - rank], dist)
        value = replicas.aggregate_throughput(3.0, world, ms_max / 1e3)
        dist.barrier()
        out[rank] = (mine, ms_max, e2e_max, value)
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_max_and_total():
    world = 2
    port = _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == [0, 1, 2, 3] and res[1][0] == [4, 5, 6]
    for r in range(world):
        assert res[r][1] == 15.0 and res[r][2] == 100.0         # every rank sees the slowest time
        assert res[r][3] == pytest.approx(2 * 3.0 / 0.015)      # whole-job units / max time
