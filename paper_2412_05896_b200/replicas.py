"""Host-side plumbing of the multi-GPU modes, one process per GPU.

Replicas: every rank has its own batch.  The path shards by independent units (sequence x KV head x layer), so no
tensor of the method crosses GPUs and there is no collective on the data path; what the ranks exchange is a barrier
and the reductions of the timing.

KV-head shards: every rank holds an equal share of the KV heads (with their query heads) of every layer and
sequence, as a tensor-parallel model does.  K, V, scores and caches stay on their GPU; the one exchange is the
layers' curves before the solver (head_shard, sum_curves_over_ranks, gather_unit_curves).

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


def count_over_ranks(n_local: int, device="cpu") -> int:
    """Sum of an integer count over the ranks (e.g. the sequences of the whole job)."""
    return int(round(sum_over_ranks(float(n_local), device)))


def sum_curves_over_ranks(local_curves: torch.Tensor) -> torch.Tensor:
    """One budget list for the units of all ranks (instead of one list per replica).  This is the only exchange a
    sharded run of the path needs -- L x curve_len numbers, before the host solver; K, V and the scores never leave
    their GPU.

    local_curves: float tensor [L, curve_len], this rank's share of the job's curves, already weighted so that the
    shares add up to the job's curve: xkv.batch_curves(..., divisor = sequences of all ranks) when the ranks hold
    different sequences, or the rank's own mean divided by the number of ranks when they hold equal shares of the
    KV heads.  Summed in place over the ranks (all-reduce) and returned; every rank then runs the same
    deterministic host solver on it as a batch of one.  No arithmetic of the method happens here.
    """
    if dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(local_curves, op=dist.ReduceOp.SUM)
    return local_curves


def head_shard(n_q_heads: int, n_kv_heads: int, rank: int, world: int) -> tuple[slice, slice]:
    """(KV heads, query heads) of one of `world` equal shards: consecutive KV heads with the query heads of their
    groups, so that a shard is a smaller model of the same group size."""
    if n_kv_heads % world != 0:
        raise ValueError("the KV heads do not divide evenly over the ranks")
    per = n_kv_heads // world
    group = n_q_heads // n_kv_heads
    return slice(rank * per, (rank + 1) * per), slice(rank * per * group, (rank + 1) * per * group)


def gather_unit_curves(local_curves: torch.Tensor) -> torch.Tensor:
    """Head-level budgets over KV-head shards: the solver's units are (layer, KV head) pairs and every rank holds
    the curves of its own heads.  local_curves [L, Hkv_local, curve_len] -> [L, Hkv, curve_len] with the heads in
    rank order (all-gather); every rank then solves for all units and keeps the budgets of its heads."""
    if not dist.is_initialized() or dist.get_world_size() == 1:
        return local_curves
    parts = [torch.empty_like(local_curves) for _ in range(dist.get_world_size())]
    dist.all_gather(parts, local_curves.contiguous())
    return torch.cat(parts, dim=1)
