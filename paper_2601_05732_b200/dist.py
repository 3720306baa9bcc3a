"""One process per GPU: rank plumbing for runs that shard the tokens over several GPUs.

Tokens are independent, so rank r simply works on its own shard of tokens (shard index = rank) with
its own copy of the parameters; there is no data-path collective.  The only things exchanged are the
barrier that brackets a timed region and the MAX over ranks of the elapsed device time.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_rank_world():
    """(rank, local_rank, world_size) from the torchrun environment; (0, 0, 1) outside it."""
    return (int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1)))


def init(world: int, backend: str = "nccl", device=None):
    if world > 1 and not dist.is_initialized():
        kw = {"device_id": torch.device(device)} if (device is not None and backend == "nccl") else {}
        dist.init_process_group(backend, **kw)


def shutdown():
    if dist.is_initialized():
        dist.destroy_process_group()


def barrier(world: int, cuda: bool = True):
    if world > 1:
        dist.barrier()
    if cuda:
        torch.cuda.synchronize()


def max_over_ranks(value: float, world: int, device="cpu") -> float:
    """The slowest rank's time: every multi-GPU number is the max over ranks."""
    if world == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_tokens_per_s(tokens_per_rank: int, world: int, steps: int, ms_max: float) -> float:
    """Whole-job throughput: all ranks' tokens over the slowest rank's time."""
    return world * tokens_per_rank * steps / (ms_max * 1e-3)


def shard_of(rank: int) -> int:
    """Token shard a rank draws (the parameters are the same on every rank)."""
    return rank
