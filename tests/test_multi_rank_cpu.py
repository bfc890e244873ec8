"""The multi-GPU form of the benchmark is "replicas only": requests are independent, every rank decodes its own batch
and no collective touches the data path.  What N > 1 adds is the aggregation of the timing -- the job is as slow as its
slowest rank, and its throughput counts every rank's items.  Checked here with two gloo ranks on the CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 100.0 if rank == 0 else 250.0                     # rank 1 is the slow one
    value, worst = bench.whole_job_throughput(dist, local_ms, items_per_rank_step=640, steps=10, world=world)
    # every rank must come to the same answer
    gathered = [None] * world
    dist.all_gather_object(gathered, (value, worst))
    if rank == 0:
        out.put(gathered)
    dist.destroy_process_group()


def test_two_replicas_aggregate_by_the_slowest_rank():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got[0] == got[1]
    value, worst = got[0]
    assert worst == 250.0
    assert abs(value - 2 * 640 * 10 / 0.250) < 1e-6


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    value, worst = bench.whole_job_throughput(None, 50.0, 640, 5, 1)
    assert worst == 50.0 and abs(value - 640 * 5 / 0.05) < 1e-9


def test_gpus_flag_without_a_launcher_starts_one_replica_per_gpu(monkeypatch):
    """`python bench.py --gpus 4` with no WORLD_SIZE in the environment must start 4 ranks itself (one per GPU, rendezvous
    on 127.0.0.1), not run one replica and call it four."""
    sys.path.insert(0, ROOT)
    import argparse
    import bench
    seen = {}
    monkeypatch.setattr(bench.subprocess, "call", lambda cmd: seen.setdefault("cmd", cmd) and 0)
    monkeypatch.setattr(bench.sys, "argv", ["bench.py", "--gpus", "4", "--steps", "3"])
    try:
        bench.relaunch_replicas(argparse.Namespace(gpus=4))
    except SystemExit as e:
        assert e.code == 0
    cmd = seen["cmd"]
    assert "--nproc-per-node=4" in cmd and "--nnodes=1" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[-4:] == ["--gpus", "4", "--steps", "3"] and cmd[-5].endswith("bench.py")
