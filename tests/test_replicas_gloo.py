"""The benchmark's multi-GPU mode is independent replicas: the only exchange is the max over ranks
of the elapsed time.  Two CPU processes over gloo check that reduction and the whole-job rate."""

import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = 10.0 + 5.0 * rank            # rank 1 is the slow one
        slowest = bench.max_over_ranks(mine)
        rate = bench.whole_job_rate(1000, 3, world, slowest)
        out.put((rank, slowest, rate))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_rate_two_replicas():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slowest, rate in got:
        assert slowest == 15.0                      # every rank sees the slowest rank's time
        assert abs(rate - 2 * 1000 * 3 / 15e-3) < 1e-6


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    import bench

    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.whole_job_rate(10, 2, 1, 4.0) == 10 * 2 / 4e-3


def test_gpus_flag_builds_a_launch_of_that_many_replicas(monkeypatch):
    """`bench.py --gpus 2` outside a launcher starts two ranks of itself on this node (it used to
    run one replica whatever the flag said); under a launcher a rank count that disagrees with
    the flag is an error."""
    sys.path.insert(0, ROOT)
    import bench

    cmd = bench.replica_launch_command(2, ["--gpus", "2", "--steps", "4"], 29511)
    assert cmd[1:3] == ["-m", "torch.distributed.run"]
    assert cmd[cmd.index("--nproc-per-node") + 1] == "2"
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[cmd.index("--master-port") + 1] == "29511"
    assert cmd[-4:] == ["--gpus", "2", "--steps", "4"] and cmd[-5].endswith("bench.py")

    calls = []
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    monkeypatch.setattr(bench.subprocess, "call", lambda c: calls.append(c) or 0)
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "2", "--steps", "1"])
    try:
        bench.main()
    except SystemExit as e:
        assert e.code == 0
    assert len(calls) == 1 and calls[0][calls[0].index("--nproc-per-node") + 1] == "2"

    monkeypatch.setenv("WORLD_SIZE", "4")
    try:
        bench.main()
        raised = False
    except SystemExit as e:
        raised = e.code not in (0, None)
    assert raised
