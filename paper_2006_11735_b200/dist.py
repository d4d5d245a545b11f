"""One process per GPU: rendezvous, sharding and the max-over-ranks reduction used for
timing.  Images are independent units through every layer, so the batch is partitioned
across ranks and the data path has no collective; the only communication is the barrier
and the reduction of the measured time."""
import os

import torch
import torch.distributed as dist


def world():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def init(backend: str = None) -> bool:
    """Join the process group described by the environment; returns True when there is one."""
    rank, _, size = world()
    if size <= 1:
        return False
    if not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group(backend or ("nccl" if torch.cuda.is_available() else "gloo"), rank=rank, world_size=size)
    return True


def barrier():
    if dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device="cpu") -> float:
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


def shard(n_units: int, rank: int, size: int):
    """Contiguous [first, first + count) slice of n_units for this rank (strong scaling)."""
    base, extra = divmod(n_units, size)
    first = rank * base + min(rank, extra)
    return first, base + (1 if rank < extra else 0)


def finish():
    if dist.is_initialized():
        dist.destroy_process_group()
