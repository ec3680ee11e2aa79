"""The multi-GPU mode is N independent replicas; its host-side plumbing (per-rank batches, barrier, max/sum of the
timing, whole-job rate, rank-0-only reference arm) is exercised here with two gloo ranks on the CPU."""
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2412_05896_b200 import replicas
from paper_2412_05896_b200 import workloads as WL

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    r, w, local = replicas.init("gloo")
    assert (r, w, local) == (rank, world, rank)
    wl = replicas.replica_workload(WL.CONFIGS["llama3_8b_ragged"], rank)
    lengths = WL.prompt_lengths(wl)
    gathered = [None] * world
    dist.all_gather_object(gathered, lengths)
    # this rank processed (rank + 1) * 1000 units in 10 ms (rank 0) or 40 ms (rank 1)
    rate, ms_max, total = replicas.whole_job_rate(1000.0 * (rank + 1), 10.0 + 30.0 * rank)
    replicas.barrier()
    out.put((rank, gathered, replicas.max_over_ranks(float(rank)), replicas.sum_over_ranks(float(rank + 1)), rate,
             ms_max, total))
    dist.destroy_process_group()


def test_two_replicas_draw_their_own_batches_and_report_the_whole_job():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, gathered, mx, sm, rate, ms_max, total in results:
        assert gathered[0] != gathered[1], "the ranks must not share a batch"
        assert len(gathered[0]) == len(gathered[1]) == WL.CONFIGS["llama3_8b_ragged"].batch
        assert mx == 1.0 and sm == 3.0
        assert total == 3000.0 and ms_max == 40.0
        assert abs(rate - 3000.0 / 0.040) < 1e-6       # all ranks' units over the slowest rank's time
    # a lone process is rank 0 of 1 and the reductions are the identity
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        os.environ.pop(k, None)
    assert replicas.env_ranks() == (0, 1, 0)
    assert replicas.whole_job_rate(500.0, 250.0) == (2000.0, 250.0, 500.0)


def _curve_worker(rank: int, world: int, port: int, out):
    import numpy as np
    from oracle import xkv_oracle as O
    from paper_2412_05896_b200 import xkv
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    replicas.init("gloo")
    L, n = 5, 40
    b_local = 2 + rank                                    # the ranks hold batches of different size
    rng = np.random.default_rng(77)
    all_curves = np.stack([[O.head_gains(rng.random(n) ** (2 + l)) for _ in range(5)] for l in range(L)])   # [L, 5, n]
    mine = all_curves[:, :2] if rank == 0 else all_curves[:, 2:]
    assert mine.shape[1] == b_local
    n_seq = replicas.count_over_ranks(b_local)
    assert n_seq == 5
    # this rank's share of the job's curve (on a GPU xkv_batch_curves forms it with divisor = n_seq)
    share = torch.from_numpy(mine.astype(np.float32).astype(np.float64).sum(axis=1) / n_seq)
    shared = replicas.sum_curves_over_ranks(share).numpy()[:, None, :]
    budgets, r = xkv.alloc_budgets(shared.astype(np.float32), [n], total=60, n_min=2)
    whole, r_whole = xkv.alloc_budgets(all_curves.astype(np.float32), [n] * 5, total=60, n_min=2)
    out.put((rank, budgets.tolist(), whole.tolist(), float(np.abs(shared[:, 0] - all_curves.astype(np.float32).mean(1)).max())))
    dist.destroy_process_group()


def test_budget_list_shared_by_all_ranks_equals_the_list_of_the_whole_batch():
    """The one exchange of a sharded run: curves averaged over every rank's sequences before the solver."""
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_curve_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert results[0][1] == results[1][1], "every rank must derive the same list"
    for rank, budgets, whole, err in results:
        assert budgets == whole and sum(budgets) == 60 and err < 1e-6


def _head_shard_worker(rank: int, world: int, port: int, out):
    import numpy as np
    from oracle import xkv_oracle as O
    from paper_2412_05896_b200 import xkv
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    replicas.init("gloo")
    L, Hq, Hkv, n = 4, 8, 4, 30
    rng = np.random.default_rng(91)
    w_heads = [[rng.random(n) ** (2 + l + g) for g in range(Hkv)] for l in range(L)]          # one sequence
    kv, qh = replicas.head_shard(Hq, Hkv, rank, world)
    assert (kv, qh) == (slice(2 * rank, 2 * rank + 2), slice(4 * rank, 4 * rank + 4))
    # layer budgets: this shard's mean over its heads, divided by the number of shards, summed over the ranks
    mine = np.stack([O.layer_gains(w_heads[l][kv], n) for l in range(L)]) / world
    layer = replicas.sum_curves_over_ranks(torch.from_numpy(mine.astype(np.float32).astype(np.float64))).numpy()
    whole = np.stack([O.layer_gains(w_heads[l], n) for l in range(L)])
    b_layer, _ = xkv.alloc_budgets(layer[:, None, :].astype(np.float32), [n], total=40)
    b_whole, _ = xkv.alloc_budgets(whole[:, None, :].astype(np.float32), [n], total=40)
    # head-level budgets: the units' curves are gathered in rank order
    local_units = torch.from_numpy(np.stack([[O.head_gains(w) for w in w_heads[l][kv]] for l in range(L)])
                                   .astype(np.float32))                                        # [L, 2, n]
    units = replicas.gather_unit_curves(local_units).numpy()                                   # [L, 4, n]
    ref_units = np.stack([[O.head_gains(w) for w in w_heads[l]] for l in range(L)]).astype(np.float32)
    b_units, _ = xkv.alloc_budgets(units.reshape(L * Hkv, 1, n), [n], total=160)
    n_ref, _ = O.head_level_allocation(w_heads, N=160)
    out.put((rank, float(np.abs(layer - whole).max()), b_layer.tolist(), b_whole.tolist(),
             bool(np.array_equal(units, ref_units)), b_units.reshape(L, Hkv).tolist(), n_ref))
    dist.destroy_process_group()


def test_kv_head_shards_exchange_curves_before_the_solver():
    """A KV-head-sharded run: the layer curve is the sum over the ranks of each rank's share, the per-head curves
    are gathered in rank order, and both give the budgets of the unsharded problem."""
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_head_shard_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert results[0][2] == results[1][2] and results[0][5] == results[1][5], "every rank derives the same lists"
    for rank, err, b_layer, b_whole, same_units, b_units, n_ref in results:
        assert err < 1e-7 and b_layer == b_whole and sum(b_layer) == 40
        assert same_units and b_units == n_ref
    try:
        replicas.head_shard(8, 4, 0, 3)
        raise AssertionError("uneven shards must be refused")
    except ValueError:
        pass


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, env=env, timeout=120)
    assert res.returncode == 0 and res.stdout.strip() == ""
