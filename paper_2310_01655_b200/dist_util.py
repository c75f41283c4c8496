"""Host-side plumbing for running one process per GPU.

Causal Polysketch attention shards over independent (batch, head) problems, so ranks
exchange no tensors on the data path: each rank works on its own batch.  What remains is
rendezvous, a barrier, and taking the maximum over ranks of a timing.

Sharding the SEQUENCE over ranks instead needs one exchange: the state every shard starts from is
the sum of the end states of the shards before it (Section 3.1's prefix sum, one level up).
`exclusive_prefix_over_ranks` is that exchange: an all-gather of the shards' totals into local
memory followed by a local sum, so no rank ever reads another rank's memory inside a kernel."""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_rank():
    """(rank, world_size, local_rank) from the launcher's environment (1 process if unset)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init(backend: str, device=None) -> bool:
    """Joins the process group when WORLD_SIZE > 1; returns whether a group exists."""
    _, world, _ = env_rank()
    if world <= 1:
        return False
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    kwargs = {"device_id": device} if (device is not None and backend == "nccl") else {}
    dist.init_process_group(backend, **kwargs)
    return True


def rank_seed(seed: int, rank: int) -> int:
    """Every rank draws its own batch: distinct, reproducible seeds."""
    return seed + 7919 * rank


def barrier() -> None:
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device="cpu") -> float:
    """Maximum of a per-rank scalar (a step time) over all ranks."""
    t = torch.tensor([value], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized():
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def exclusive_prefix_over_ranks(local_total: torch.Tensor) -> torch.Tensor:
    """Sum of `local_total` over the ranks BEFORE this one (zeros on rank 0): the state a sequence
    shard starts from, given every shard's own total phi'(K_shard)^T [V_shard | 1].  With one process
    the result is zeros.  For the backward's suffix states call it on the reversed rank order."""
    out = torch.zeros_like(local_total)
    if not (dist.is_available() and dist.is_initialized()):
        return out
    world, rank = dist.get_world_size(), dist.get_rank()
    gathered = [torch.empty_like(local_total) for _ in range(world)]
    dist.all_gather(gathered, local_total.contiguous())
    for r in range(rank):
        out += gathered[r]
    return out


def aggregate_throughput(units_per_rank_step: int, steps: int, max_ms: float, world: int) -> float:
    """Whole-job units per second: every rank processes `units_per_rank_step` per step (weak
    scaling), and the job is as slow as its slowest rank."""
    return world * units_per_rank_step * steps / (max_ms / 1e3)


def shutdown() -> None:
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()
