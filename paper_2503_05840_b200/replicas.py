"""Host-side logic for running N independent replicas of the decode path, one
process per GPU.  The path shards by sequence and by layer with no exchange
step, so ranks share nothing but the barrier around the timed region and the
max-over-ranks of its duration.  Works with any torch.distributed backend
(nccl on GPUs, gloo in the CPU tests)."""
from __future__ import annotations

import os


def rank_info():
    """(rank, world_size, local_rank) from the launcher's environment."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def _free_port() -> int:
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        return sk.getsockname()[1]


def _spawned(rank: int, world: int, port: int, target, args) -> None:
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    target(rank, world, *args)


def spawn_replicas(target, world: int, args=(), port: int | None = None) -> None:
    """Start `world` processes on this node, one per GPU (rank = local rank), each with the
    environment a launcher would give it (RANK, LOCAL_RANK, WORLD_SIZE, MASTER_ADDR, MASTER_PORT),
    and run target(rank, world, *args) in each.  Returns when all have exited; raises if one failed.
    `target` must be importable (a module-level function)."""
    import torch.multiprocessing as mp
    mp.spawn(_spawned, args=(world, port or _free_port(), target, tuple(args)), nprocs=world, join=True)


def replica_seed(base_seed: int, rank: int) -> int:
    """Every replica draws its own keys and queries; the ragged length mix is
    the same on all ranks so that per-GPU work is equal (weak scaling)."""
    return base_seed + 100000 * rank


def max_over_ranks(ms: float, dist=None, device=None) -> float:
    """Duration of the slowest rank (the job's duration)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(ms)
    import torch
    t = torch.tensor([float(ms)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank: int, world_size: int, ms_per_step: float) -> float:
    """Whole-job units per second: all ranks' units over the slowest rank's step time."""
    return units_per_rank * world_size / (ms_per_step * 1e-3)
