"""Multi-GPU plumbing: one process per GPU, no collective on the data path.

Every (sequence, layer, KV head) slab is an independent unit of the compress path and every
(sequence, KV head) of decode attention, so ranks simply own disjoint units.  The only exchanges
are the barrier around a timed region and the maximum of the per-rank times.  Works with the
`nccl` backend on GPUs and with `gloo` on CPUs (tests)."""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_world():
    """(rank, local_rank, world_size) from the launcher's environment; (0, 0, 1) when run directly."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str, device=None):
    """Join the process group if there is more than one rank.  Returns (rank, world_size)."""
    rank, _, world = env_world()
    if world > 1 and not dist.is_initialized():
        kw = {"device_id": device} if (backend == "nccl" and device is not None) else {}
        dist.init_process_group(backend, **kw)
    return rank, world


def finish():
    if dist.is_initialized():
        dist.destroy_process_group()


def partition(n_units: int, rank: int, world: int):
    """Contiguous, balanced share [begin, end) of n_units for this rank; the first n_units % world ranks get one more."""
    base, extra = divmod(n_units, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def rank_seed(seed: int, rank: int) -> int:
    """Seed of a replica's synthetic inputs: every rank draws its own data."""
    return seed + 7919 * rank


def barrier(device=None):
    """Barrier over the ranks, then drain the device: brackets a timed region on both sides."""
    if dist.is_initialized():
        dist.barrier()
    if device is not None and torch.device(device).type == "cuda":
        torch.cuda.synchronize(device)


def max_over_ranks(value: float, device="cpu") -> float:
    """The slowest rank's time: the time of the whole job."""
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
