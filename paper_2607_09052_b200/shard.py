"""Sharding of the decode step over ranks: independent sequences per rank, no data-path collective.

Every (sequence, KV head) unit is independent (one block set per KV head; the paper optimises each KV head on
its own), so N ranks each hold their own batch of sequences.  The only communication is the timing reduction of
the benchmark: the step time of the job is the slowest rank's.
"""

from __future__ import annotations

import socket
import sys

import torch
import torch.distributed as dist


def rank_workload(wl, rank: int):
    """The workload rank `rank` draws: same shapes, its own sequences (seed offset by the rank)."""
    return wl.replace(seed=wl.seed + 1000 * rank)


def job_times(local_values, device="cpu"):
    """Max over ranks of each entry of `local_values` (list of floats); identity without a process group."""
    t = torch.tensor(list(local_values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def job_throughput(bytes_per_rank_step: int, world: int, max_step_seconds: float) -> float:
    """Whole-job GB/s: all ranks' bytes over the slowest rank's step time."""
    return world * bytes_per_rank_step / max_step_seconds / 1e9


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def launcher_command(script: str, n_ranks: int, argv, port: int = 0):
    """The command that starts `n_ranks` ranks of `script` on this node: torch.distributed.run, one process per
    rank (per GPU), rendezvous on 127.0.0.1 (a container's hostname may not resolve)."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_ranks}",
            "--master-addr", "127.0.0.1", "--master-port", str(port or free_port()), script, *argv]
