"""One process per GPU: rank plumbing for runs that shard the tokens over several GPUs.

Tokens are independent, so rank r simply works on its own shard of tokens (shard index = rank) with
its own copy of the parameters; there is no data-path collective.  The only things exchanged are the
barrier that brackets a timed region and the MAX over ranks of the elapsed device time, and, for a
trainer that shards the tokens (data parallelism, paper Appendix A), the sum over ranks of the
parameter gradients dW, db, dalpha, dgain: the only quantities of the layer that add up over tokens.
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


def all_reduce_param_grads(dW: torch.Tensor, db: torch.Tensor, dalpha: torch.Tensor, dgain: torch.Tensor,
                           world: int, bucket: torch.Tensor | None = None) -> torch.Tensor | None:
    """Sums the layer's parameter gradients over the ranks, in place, with ONE all-reduce.

    The four tensors ((nC+1) N + nC + 3 floats, about 0.5 MB at n=4, C=1024) are packed into one flat
    bucket (pass `bucket` to reuse a buffer of that size on the tensors' device), reduced, and copied
    back.  Each rank's gradients cover its own token shard; the sum is the gradient over all tokens.
    Returns the bucket (None when world == 1, where nothing is done).
    """
    if world == 1:
        return None
    parts = (dW, db, dalpha, dgain)
    total = sum(p.numel() for p in parts)
    if bucket is None:
        bucket = torch.empty(total, dtype=dW.dtype, device=dW.device)
    assert bucket.numel() >= total and bucket.dtype == dW.dtype
    off = 0
    for p in parts:
        bucket[off:off + p.numel()].copy_(p.reshape(-1))
        off += p.numel()
    dist.all_reduce(bucket[:total], op=dist.ReduceOp.SUM)
    off = 0
    for p in parts:
        p.copy_(bucket[off:off + p.numel()].view_as(p))
        off += p.numel()
    return bucket
