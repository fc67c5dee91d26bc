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


def test_gpus_flag_without_launcher_spawns_replicas():
    """`python bench.py --gpus 2` run directly (no WORLD_SIZE) starts one process per replica itself;
    the launch-path self-check stage needs no GPU (gloo) and prints the job-wide arithmetic."""
    import json
    import subprocess
    import sys
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    res = subprocess.run([sys.executable, bench.__file__, "--gpus", "2", "--stage", "ranks", "--steps", "20"],
                         capture_output=True, text=True, timeout=300, env=env)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                   # rank 0 alone prints
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["ms_max"] == 15.0
    assert line["value"] == pytest.approx(2 * 4096 * 20 / 15e-3)
    cmd = bench.replica_launch_command(4, ["--gpus", "4", "--steps", "7"], 29999)
    assert "--nproc-per-node=4" in cmd and cmd[-4:] == ["--gpus", "4", "--steps", "7"]
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"


def test_gpus_flag_must_agree_with_the_launcher():
    import subprocess
    import sys
    env = dict(os.environ, WORLD_SIZE="1", RANK="0", LOCAL_RANK="0")
    res = subprocess.run([sys.executable, bench.__file__, "--gpus", "8", "--stage", "ranks"],
                         capture_output=True, text=True, timeout=120, env=env)
    assert res.returncode == 2 and "WORLD_SIZE" in res.stderr
