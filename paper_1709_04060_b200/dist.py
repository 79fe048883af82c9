"""Process-group plumbing for multi-GPU runs: one process per GPU, no data-path
collective.  The hot path partitions over independent problems (columns /
images / GEMM problems are independent, thresholds are per row), so ranks only
meet at a barrier and to take the maximum of their device-side timings."""
import os

import torch
import torch.distributed as dist


def env_rank_world():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def init(backend: str):
    """Initialise the default group from the torchrun environment (no-op for 1 rank)."""
    rank, world = env_rank_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, world


def barrier():
    if dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device="cpu") -> float:
    """Maximum of a per-rank scalar (e.g. elapsed device milliseconds)."""
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


def shard(units, rank: int, world: int):
    """Contiguous, balanced share of a list of independent work units."""
    n = len(units)
    lo = rank * n // world
    hi = (rank + 1) * n // world
    return units[lo:hi]


def finalize():
    if dist.is_initialized():
        dist.destroy_process_group()
