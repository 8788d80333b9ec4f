"""Multi-GPU plumbing for the replayed layer: token sharding and max-over-ranks timing.

The replayed layer has no exchange step when expert weights are replicated: every token's gate,
rows and output depend on that token alone.  N GPUs therefore each run the whole path on their
own slice of the tokens (weak scaling: the per-GPU batch is fixed), with no data-path
collective; torch.distributed is used only for the start barrier and to reduce the timings.
"""
from __future__ import annotations

import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist


def env_rank_world():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def init(backend: str) -> tuple[int, int]:
    """Joins the process group described by the torchrun environment (no-op for one process)."""
    rank, world = env_rank_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, world


def shard_range(total: int, rank: int, world: int) -> tuple[int, int]:
    """Contiguous [lo, hi) slice of `total` units owned by `rank`; sizes differ by at most one."""
    base, extra = divmod(total, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def barrier():
    if dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device="cpu") -> float:
    """The slowest rank's time decides the job's time."""
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device="cpu") -> float:
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def free_port() -> int:
    """A TCP port of the loopback interface that is free right now."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def launch_command(n_ranks: int, script: str, argv, port: int) -> list:
    """Command line that runs `script argv...` as n_ranks processes of one node under
    torch.distributed.run, rendezvous on the loopback interface (one process per GPU: every rank
    reads RANK / LOCAL_RANK / WORLD_SIZE from its environment)."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1",
            f"--nproc-per-node={n_ranks}", "--master-addr", "127.0.0.1", "--master-port",
            str(port), script, *argv]


def run_ranks(n_ranks: int, script: str, argv, env=None) -> int:
    """Starts the n_ranks processes of a job whose caller gave only a rank count (no launcher
    environment), waits for them and returns the launcher's exit code.  The ranks inherit the
    caller's standard output, so rank 0's one line is the job's line."""
    full_env = dict(os.environ)
    # NCCL's communicator log (rings, NVLS, transports) of every rank, kept out of the job's
    # standard output
    full_env.setdefault("NCCL_DEBUG", "INFO")
    full_env.setdefault("NCCL_DEBUG_FILE", os.path.join(
        os.environ.get("TMPDIR", "/tmp"), "r3_nccl_%h_%p.log"))
    if env:
        full_env.update(env)
    return subprocess.call(launch_command(n_ranks, script, list(argv), free_port()), env=full_env)
