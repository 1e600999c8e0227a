"""Multi-GPU plumbing: candidates are independent units, so the path shards by
candidate with no data-path collective (the paper runs one candidate kernel per
GPU, App. "Kernel Optimization Cost and Runtime Analysis").  Each rank verifies
its own candidates against a reference it holds or regenerates from the seed;
only the tiny results (K pass bits, a time) travel, over torch.distributed.
Works with any backend (nccl on GPUs, gloo on CPU)."""
from __future__ import annotations

import torch
import torch.distributed as dist


def k_range(K: int, world: int, rank: int) -> range:
    """Contiguous, balanced shard of candidate indices for `rank`; shards differ by at most one."""
    if K < 0 or world < 1 or not (0 <= rank < world):
        raise ValueError("bad shard arguments")
    base, extra = divmod(K, world)
    lo = rank * base + min(rank, extra)
    return range(lo, lo + base + (1 if rank < extra else 0))


def _world(group=None) -> int:
    return dist.get_world_size(group) if dist.is_available() and dist.is_initialized() else 1


def max_over_ranks(value: float, device="cpu", group=None) -> float:
    """The slowest rank's time: what a whole-job throughput divides by."""
    if _world(group) == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(t.item())


def sum_over_ranks(value: float, device="cpu", group=None) -> float:
    if _world(group) == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    return float(t.item())


def gather_joint_pass(local_pass, K: int, device="cpu", group=None) -> list:
    """Per-rank pass bits (for the rank's k_range, in order) -> the list for all K candidates."""
    world = _world(group)
    rank = dist.get_rank(group) if world > 1 else 0
    mine = k_range(K, world, rank)
    if len(local_pass) != len(mine):
        raise ValueError(f"rank {rank} holds {len(mine)} candidates, got {len(local_pass)} results")
    if world == 1:
        return [int(v) for v in local_pass]
    width = len(k_range(K, world, 0))                      # the longest shard
    buf = torch.full((width,), -1, dtype=torch.int32, device=device)
    if len(mine):
        buf[:len(mine)] = torch.as_tensor([int(v) for v in local_pass], dtype=torch.int32, device=device)
    parts = [torch.empty_like(buf) for _ in range(world)]
    dist.all_gather(parts, buf, group=group)
    out = []
    for r, p in enumerate(parts):
        out.extend(int(v) for v in p[:len(k_range(K, world, r))].cpu())
    return out
