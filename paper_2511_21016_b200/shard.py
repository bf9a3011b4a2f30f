"""Data-parallel plumbing: (batch, head) pairs are independent units of the GKA hot path, so N
GPUs run N independent shards with no data-path collective.  The only communication is the
benchmark's barrier and the max-over-ranks of the measured time."""
from __future__ import annotations

import os
from typing import Tuple

import torch
import torch.distributed as dist


def env_rank_world() -> Tuple[int, int, int]:
    """(rank, local_rank, world_size) from the torchrun environment, (0, 0, 1) without it."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def free_port() -> int:
    """A TCP port that is free on the loopback interface right now."""
    import socket
    sk = socket.socket()
    sk.bind(("127.0.0.1", 0))
    port = sk.getsockname()[1]
    sk.close()
    return port


def rank_env(rank: int, world: int, port: int) -> dict:
    """Environment of local rank `rank` of `world` (what torchrun would set), for launching ranks without it."""
    env = dict(os.environ)
    env.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
               MASTER_PORT=str(port))
    return env


def shard_seed(base_seed: int, rank: int) -> int:
    """Seed of a rank's shard: every rank draws its own batch of the same shape (weak scaling)."""
    return base_seed + 1000 * rank


def batch_slice(total_batch: int, rank: int, world: int) -> Tuple[int, int]:
    """[start, stop) of the sequences a rank owns when one global batch is split (strong scaling);
    remainders go to the lowest ranks."""
    base, rem = divmod(total_batch, world)
    start = rank * base + min(rank, rem)
    return start, start + base + (1 if rank < rem else 0)


def init_process_group(backend: str) -> None:
    if not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29511")
        dist.init_process_group(backend=backend)


def barrier() -> None:
    if dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


def max_over_ranks(value: float, device: str = "cpu") -> float:
    """Largest value over all ranks (the time a whole job took is its slowest rank's)."""
    if not (dist.is_initialized() and dist.get_world_size() > 1):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device: str = "cpu") -> float:
    if not (dist.is_initialized() and dist.get_world_size() > 1):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())
