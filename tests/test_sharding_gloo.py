"""Multi-process (world size 2, gloo, CPU) test of the batch sharding and of the job-throughput reduction."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2001_07710_b200.sharding import job_throughput, shard_batch


def test_shard_batch_covers_the_batch_exactly():
    for n in (0, 1, 7, 64, 65):
        for world in (1, 2, 3, 8):
            spans = [shard_batch(n, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [b - a for a, b in spans]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        shard_batch(4, 2, 2)


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
        start, stop = shard_batch(65, world, rank)
        ms = 10.0 if rank == 0 else 25.0                      # rank 1 is the slow one
        dist.barrier()
        value, ms_job, units = job_throughput(float(stop - start), ms)
        out[rank] = (value, ms_job, units, stop - start)
    finally:
        dist.destroy_process_group()


def test_job_throughput_world2_gloo():
    world = 2
    mgr = mp.get_context("spawn").Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    assert set(out.keys()) == {0, 1}
    for r in range(world):
        value, ms_job, units, _ = out[r]
        assert ms_job == 25.0                                  # slowest rank's time
        assert units == 65.0                                   # all images counted once
        assert abs(value - 65.0 / 0.025) < 1e-9
    assert out[0][3] + out[1][3] == 65 and abs(out[0][3] - out[1][3]) <= 1


def test_job_throughput_without_process_group():
    value, ms, units = job_throughput(64.0, 8.0)
    assert (value, ms, units) == (8000.0, 8.0, 64.0)
