"""The N > 1 path of the benchmark on two gloo ranks (CPU): every rank draws its own sequences, the job's step
time is the slowest rank's, the job's throughput counts every rank's bytes."""

import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2607_09052_b200 import shard, synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = shard.rank_workload(synth.named_workloads()["cfg1_tiny"], rank)
    inp = synth.generate(wl)
    local_ms = 1.0 + rank            # rank 1 is the slow one
    total_ms, e2e = shard.job_times([local_ms, 10.0 - rank])
    gathered = [None] * world
    dist.all_gather_object(gathered, (wl.seed, float(inp["q"].float().sum())))
    out[rank] = (total_ms, e2e, gathered, shard.job_throughput(1000, world, total_ms * 1e-3))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_draw_distinct_sequences_and_time_is_max_over_ranks():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    for rank in range(world):
        total_ms, e2e, gathered, gbs = out[rank]
        assert total_ms == 2.0 and e2e == 10.0              # max over ranks, same on every rank
        seeds = [g[0] for g in gathered]
        sums = [g[1] for g in gathered]
        assert seeds[0] != seeds[1] and sums[0] != sums[1]  # each rank has its own sequences
        assert abs(gbs - 2 * 1000 / 2e-3 / 1e9) < 1e-12


def test_single_process_is_identity():
    assert shard.job_times([3.5, 1.0]) == [3.5, 1.0]
    wl = synth.named_workloads()["cfg2_32k"]
    assert shard.rank_workload(wl, 0).seed == wl.seed and shard.rank_workload(wl, 3).seed == wl.seed + 3000


def test_bench_gpus_flag_starts_that_many_ranks():
    """`python bench.py --gpus 2` with no launcher around it must bring up two ranks by itself (it re-executes
    under torch.distributed.run on 127.0.0.1) and report the real world size and the slowest rank's step time.
    The launch self-test mode runs that path on gloo with a stub step, so it needs no GPU."""
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    res = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--steps", "4", "--launch-selftest"],
                         capture_output=True, text=True, timeout=240, env=env, cwd=root)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, res.stdout                       # rank 0 alone prints
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2
    assert line["ms_per_step"] == 2.0                        # rank 1's stub step takes twice rank 0's: max over ranks
    assert "rank 0 of 2" in res.stderr and "rank 1 of 2" in res.stderr


def test_launcher_command_shape():
    cmd = shard.launcher_command("/x/bench.py", 4, ["--gpus", "4", "--steps", "2"], port=29999)
    assert cmd[1:3] == ["-m", "torch.distributed.run"]
    assert "--nproc-per-node=4" in cmd and "--nnodes=1" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[cmd.index("--master-port") + 1] == "29999"
    assert cmd[-5:] == ["/x/bench.py", "--gpus", "4", "--steps", "2"]
