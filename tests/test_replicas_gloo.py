"""CPU, world_size 2 over gloo: the only cross-rank step of the N-GPU benchmark is the
max-over-ranks reduction of the per-replica device time (tokens shard with no exchange)."""
import os
import socket

import pytest
import torch.distributed as dist
import torch.multiprocessing as mp

import bench


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, "cpu")          # rank 1 is the slow replica
    out.put((rank, ms, bench.replica_throughput(world, 4096, 20, ms)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_time():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, value in got:
        assert ms == 15.0
        assert value == pytest.approx(2 * 4096 * 20 / 15e-3)


def test_single_process_is_identity():
    assert bench.max_over_ranks(3.5, "cpu") == 3.5
    assert bench.replica_throughput(1, 100, 10, 2.0) == pytest.approx(100 * 10 / 2e-3)
