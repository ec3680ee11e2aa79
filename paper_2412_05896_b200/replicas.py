"""Host-side plumbing of the multi-GPU mode: N replicas, one process per GPU, each with its own batch.

The path shards by independent units (sequence x KV head x layer), so no tensor of the method crosses GPUs and
there is no collective on the data path; what the ranks exchange is a barrier and the reductions of the timing.
The functions work on any torch.distributed backend (nccl on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

import os
from dataclasses import replace

import torch
import torch.distributed as dist

SEED_STRIDE = 7919          # rank r draws its batch from seed + r * SEED_STRIDE


def env_ranks() -> tuple[int, int, int]:
    """(rank, world size, local rank) as torchrun exports them; a lone process is rank 0 of 1."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init(backend: str, device: torch.device | None = None) -> tuple[int, int, int]:
    rank, world, local = env_ranks()
    if world > 1 and not dist.is_initialized():
        if device is not None and backend == "nccl":
            dist.init_process_group(backend, device_id=device)
        else:
            dist.init_process_group(backend)
    return rank, world, local


def replica_workload(w, rank: int):
    """The workload of one replica: same shape, its own seed (so ragged lengths and data differ per rank)."""
    return replace(w, seed=w.seed + SEED_STRIDE * rank)


def barrier() -> None:
    if dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


def _reduce(x: float, op, device) -> float:
    if not dist.is_initialized() or dist.get_world_size() == 1:
        return float(x)
    t = torch.tensor([x], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=op)
    return float(t.item())


def max_over_ranks(x: float, device="cpu") -> float:
    return _reduce(x, dist.ReduceOp.MAX, device)


def sum_over_ranks(x: float, device="cpu") -> float:
    return _reduce(x, dist.ReduceOp.SUM, device)


def whole_job_rate(units_local: float, ms_local: float, device="cpu") -> tuple[float, float, float]:
    """(units of all ranks per second, the slowest rank's milliseconds, units of all ranks): weak scaling, every
    rank processes its own units and the job takes as long as the slowest rank."""
    ms_max = max_over_ranks(ms_local, device)
    total = sum_over_ranks(units_local, device)
    return total / (ms_max * 1e-3), ms_max, total


def batch_mean_curves_over_ranks(gains, device="cpu"):
    """One budget list for the sequences of all ranks (instead of one list per replica): the curves the solver
    averages over a batch are averaged over every rank's batch.  gains: float [L, B_local, curve_len] as written by
    xkv_score (torch tensor or array; every rank must use the same L and curve_len).  Returns a torch float64
    tensor [L, 1, curve_len] that xkv.alloc_budgets takes as a batch of one: the mean over all sequences of the
    job.  This is the only exchange a sharded run of the path needs -- L x curve_len numbers, before the host
    solver; K, V and the scores never leave their GPU.
    """
    g = torch.as_tensor(gains).to(device=device, dtype=torch.float64)
    total = g.sum(dim=1, keepdim=True)
    count = torch.tensor([float(g.shape[1])], device=device, dtype=torch.float64)
    if dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(total, op=dist.ReduceOp.SUM)
        dist.all_reduce(count, op=dist.ReduceOp.SUM)
    return total / count
