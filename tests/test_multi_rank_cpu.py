"""Host logic of the multi-GPU bench path, on CPU with the gloo backend (world size 2).

The path shards by replication only (tokens are independent rows, no data-path collective):
each rank times its own replica, the job time is the maximum over ranks, the value is the sum
of the replicas' work over that time.  The reference arm prints on rank 0 only.
"""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    mine = 2.0 + 3.0 * rank                      # rank 1 is the slow replica: 5 ms
    slowest = bench.max_over_ranks(mine, world)
    value = bench.replica_throughput(1e12, world, slowest)
    gathered = [None] * world
    dist.all_gather_object(gathered, (slowest, value))
    if rank == 0:
        out.put(gathered)
    dist.destroy_process_group()


def test_replicas_report_max_time_and_summed_work():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for slowest, value in got:
        assert slowest == 5.0
        assert abs(value - 2 * 1e12 / 5e-3 / 1e12) < 1e-9      # two replicas' ops over the slowest time


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.max_over_ranks(1.25, 1) == 1.25
    assert bench.replica_throughput(2e12, 1, 1.0) == 2000.0


def test_reference_arm_prints_on_rank_0_only():
    env = dict(os.environ, WORLD_SIZE="2", RANK="1", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                        "--gpus", "2", "--steps", "1", "--warmup", "0"], env=env,
                       capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_gpus_flag_is_honoured():
    """--gpus N decides the launch: alone for one GPU, as a rank of a launcher whose world size
    agrees, by starting the ranks itself when no launcher did; a disagreeing launcher is an error."""
    import pytest

    import bench
    assert bench.launch_mode(1, {}) == "single"
    assert bench.launch_mode(1, {"WORLD_SIZE": "1"}) == "single"
    assert bench.launch_mode(4, {"WORLD_SIZE": "4"}) == "rank"
    assert bench.launch_mode(2, {}) == "spawn"
    with pytest.raises(SystemExit):
        bench.launch_mode(8, {"WORLD_SIZE": "2"})
    with pytest.raises(SystemExit):
        bench.launch_mode(1, {"WORLD_SIZE": "2"})
    with pytest.raises(SystemExit):
        bench.launch_mode(0, {})
    cmd = bench.spawn_command(2, ["--gpus", "2", "--steps", "3"], 29511)
    assert "torch.distributed.run" in cmd and "--nproc-per-node=2" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[-4:] == ["--gpus", "2", "--steps", "3"]


def test_reference_arm_does_not_need_the_cuda_library():
    """The CPU-only arm draws its inputs without importing the package that loads libw4a8.so."""
    code = ("import sys, bench; s = bench.load_synth(); "
            "assert s.WORKLOADS[4].shapes[0][:2] == (9216, 36864); "
            "assert 'paper_2311_05161_b200' not in sys.modules")
    r = subprocess.run([sys.executable, "-c", code], cwd=ROOT, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0, r.stderr
