"""Multi-GPU plumbing: one process per GPU, heads sharded across ranks, no data-path
collective (heads are planned and attended independently: Algorithm 2 loops over heads,
and heads share no K/V blocks).  torch.distributed is used for the rendezvous, the barrier,
the max-over-ranks timing reduction and an optional gather of per-head results."""
from __future__ import annotations

import os
from typing import List, Tuple

import torch
import torch.distributed as dist


def env_rank() -> Tuple[int, int, int]:
    """(rank, world_size, local_rank) from the launcher's environment (1 process if unset)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init(backend: str = "nccl") -> Tuple[int, int, int]:
    """Rendezvous of the launcher's ranks.  WAVEAL_DIST_BACKEND=gloo overrides the backend: the
    control plane (barrier, max / sum of a scalar) then runs over gloo, which lets several ranks
    share one GPU in a functional test - their kernels never wait on one another."""
    rank, world, local = env_rank()
    backend = os.environ.get("WAVEAL_DIST_BACKEND", backend)
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        kw = {}
        if backend == "nccl":
            torch.cuda.set_device(local)
            kw["device_id"] = torch.device("cuda", local)
        dist.init_process_group(backend=backend, rank=rank, world_size=world, **kw)
    return rank, world, local


def head_slice(rank: int, world: int, total_heads: int) -> range:
    """Contiguous, balanced slice of the flattened (batch*heads) axis owned by `rank`."""
    base, rem = divmod(total_heads, world)
    lo = rank * base + min(rank, rem)
    return range(lo, lo + base + (1 if rank < rem else 0))


def barrier():
    if dist.is_initialized():
        dist.barrier()


def _scalar_device(device):
    return "cpu" if dist.get_backend() == "gloo" else device


def max_over_ranks(value: float, device="cpu") -> float:
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=_scalar_device(device))
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device="cpu") -> float:
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=_scalar_device(device))
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def gather_heads(local: torch.Tensor, total_heads: int) -> torch.Tensor:
    """Concatenates per-head results (first axis = this rank's heads) over ranks in head
    order; every rank receives the full [total_heads, ...] tensor."""
    if not dist.is_initialized():
        return local
    world, rank = dist.get_world_size(), dist.get_rank()
    sizes = [len(head_slice(r, world, total_heads)) for r in range(world)]
    mx = max(sizes)
    pad = torch.zeros((mx,) + tuple(local.shape[1:]), dtype=local.dtype, device=local.device)
    pad[: local.shape[0]] = local
    parts: List[torch.Tensor] = [torch.empty_like(pad) for _ in range(world)]
    dist.all_gather(parts, pad)
    return torch.cat([p[:n] for p, n in zip(parts, sizes)], dim=0)


def shutdown():
    if dist.is_initialized():
        dist.destroy_process_group()
