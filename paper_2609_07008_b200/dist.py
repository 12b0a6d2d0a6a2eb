"""Process-group plumbing for the benchmark: one process per GPU, every rank runs its own
independent request (the MLA-Online layer has no exchange step, so nothing of the data path
crosses ranks); the group is used only for the barrier around the timed region and for the
max-over-ranks of the device time."""
from __future__ import annotations

import os
from typing import Tuple

import torch
import torch.distributed as dist


def env_ranks() -> Tuple[int, int, int]:
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init(backend: str, device=None) -> Tuple[int, int, int]:
    """Joins the group described by RANK / WORLD_SIZE / MASTER_ADDR / MASTER_PORT (no-op for one rank)."""
    rank, world, local_rank = env_ranks()
    if world > 1 and not dist.is_initialized():
        kw = {}
        if backend == "nccl" and device is not None:
            kw["device_id"] = device
        dist.init_process_group(backend, rank=rank, world_size=world, **kw)
    return rank, world, local_rank


def barrier() -> None:
    if dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device="cpu") -> float:
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    if dist.is_initialized():
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def rank_seed(base_seed: int, rank: int) -> int:
    """Each rank draws its own request values: independent requests of the same shape."""
    return int(base_seed) * 1000 + int(rank)


def aggregate_throughput(units_per_rank_step: int, steps: int, world: int, max_seconds: float) -> float:
    """Whole-job throughput: units all ranks processed divided by the slowest rank's time."""
    return world * units_per_rank_step * steps / max_seconds


def spawn_ranks(n: int, script_and_args) -> int:
    """Starts `n` ranks of `script_and_args` on this node through torch.distributed.run (one process per GPU,
    rendezvous on 127.0.0.1 at a free port) and returns its exit code.  Rank 0's standard output is the
    caller's: the one JSON line appears once."""
    import socket
    import subprocess
    import sys
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(port)] + list(script_and_args)
    return subprocess.run(cmd).returncode


def shutdown() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()
