"""Data-parallel sharding of the attention path: host logic only, no arithmetic of the method.

Every (batch, head) pair of Eq. 5-6 / Eq. 9-12 is an independent problem (the sums run over
positions of one sequence of one head), so N processes split the pairs and never exchange
data on the path.  The only collectives are the timing reductions of the benchmark (a
barrier and a MAX over ranks) and, in tests, a gather that reassembles the shards.

One process per GPU, launched by `python -m torch.distributed.run`; the same code runs as
CPU ranks over `gloo` in the tests.
"""
from __future__ import annotations

import dataclasses
import os
from typing import Sequence, Tuple

import torch


def env_ranks() -> Tuple[int, int, int]:
    """(world size, rank, local rank) from the launcher's environment; (1, 0, 0) when absent."""
    return (int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init_process_group(backend: str = "nccl"):
    """Join the job's process group (no-op for a single process).  Returns (world, rank, local)."""
    world, rank, local = env_ranks()
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        if not dist.is_initialized():
            if backend == "nccl":
                torch.cuda.set_device(local)
                dist.init_process_group("nccl", device_id=torch.device("cuda", local))
            else:
                dist.init_process_group(backend, rank=rank, world_size=world)
    return world, rank, local


def pair_range(pairs: int, world: int, rank: int) -> Tuple[int, int]:
    """Contiguous, balanced split of `pairs` independent (batch, head) problems: rank r owns
    [lo, hi); the first `pairs % world` ranks own one more than the others.  A rank may own none."""
    if world < 1 or not 0 <= rank < world:
        raise ValueError(f"rank {rank} outside a world of {world}")
    if pairs < 0:
        raise ValueError("negative number of pairs")
    base, extra = divmod(pairs, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def shard_pairs(tensors: Sequence[torch.Tensor], world: int, rank: int):
    """Strong-scaling shard: each [B, H, ...] tensor becomes the [1, n_r, ...] block of this rank's
    pairs (a view: nothing is copied).  The library treats it as a batch of one with n_r heads."""
    out = []
    for t in tensors:
        B, H = t.shape[:2]
        lo, hi = pair_range(B * H, world, rank)
        out.append(t.reshape(1, B * H, *t.shape[2:])[:, lo:hi])
    return out


def rank_workload(w, world: int, rank: int):
    """Weak-scaling shard: every rank runs a problem of the workload's own shape on its own draw
    (seed + rank); the job's size is `world` times the workload's."""
    if not 0 <= rank < world:
        raise ValueError(f"rank {rank} outside a world of {world}")
    return dataclasses.replace(w, seed=w.seed + rank)


def barrier(world: int, cuda: bool = True):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    if cuda:
        torch.cuda.synchronize()


def max_over_ranks(x: float, world: int, device="cpu") -> float:
    """The job's time for a region is the slowest rank's."""
    if world == 1:
        return float(x)
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(x: float, world: int, device="cpu") -> float:
    """Units processed by the whole job (ranks may own different numbers of pairs)."""
    if world == 1:
        return float(x)
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def gather_pairs(local: torch.Tensor, pairs: int, world: int, rank: int) -> torch.Tensor:
    """Reassemble [1, n_r, ...] shards into [1, pairs, ...] on every rank (tests and result
    collection; the attention path itself never calls this)."""
    if world == 1:
        return local
    import torch.distributed as dist
    sizes = [pair_range(pairs, world, r) for r in range(world)]
    assert local.shape[1] == sizes[rank][1] - sizes[rank][0]
    widest = max(hi - lo for lo, hi in sizes)
    padded = torch.zeros((1, widest, *local.shape[2:]), dtype=local.dtype, device=local.device)
    padded[:, : local.shape[1]] = local
    parts = [torch.empty_like(padded) for _ in range(world)]
    dist.all_gather(parts, padded)
    return torch.cat([p[:, : hi - lo] for p, (lo, hi) in zip(parts, sizes)], dim=1)
