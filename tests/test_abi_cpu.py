"""Host-side checks that need no GPU: the library loads, exports every symbol the header declares,
rejects bad arguments before touching CUDA, and its budget solver (Alg. 1) agrees with the oracle."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import xkv_oracle as O
from paper_2412_05896_b200 import build, xkv

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "xkv.h")).read()
    declared = set(re.findall(r"\b(xkv_[a-z_]+)\s*\(", header))
    assert declared == set(xkv.EXPORTS)
    lib = ctypes.CDLL(xkv.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name
    assert xkv.version() >= 100
    assert xkv.status_string(xkv.ERR_WORKSPACE) == "workspace too small"
    assert xkv.launch_count() >= 0


def _dims(**kw):
    base = dict(batch=2, n_q_heads=8, n_kv_heads=2, head_dim=128, window=16, pool_kernel=7, pool_mode=0,
                scale=0.0, kv_stride_token=256, kv_stride_head=128)
    base.update(kw)
    return xkv.Dims(**base)


def test_workspace_sizes_and_rejections():
    d = _dims()
    assert xkv.workspace_bytes(xkv.OP_SCORE, d, max_seqlen=1000, total_tokens=1500) > 0
    assert xkv.workspace_bytes(xkv.OP_SELECT_COMPACT, d, max_seqlen=1000, total_tokens=1500) > 0
    auto = xkv.workspace_bytes(xkv.OP_DECODE_ATTN, d, n_layers=4, max_cache_len=4096)
    forced = xkv.workspace_bytes(xkv.OP_DECODE_ATTN, d, n_layers=4, max_cache_len=4096, chunk_rows=64)
    assert auto > 0 and forced > 0
    lib = xkv.lib()
    assert xkv.workspace_bytes(xkv.OP_SCORE, _dims(window=3), max_seqlen=1000, total_tokens=1500) > 0   # rows are padded
    for bad in (_dims(head_dim=96), _dims(window=0), _dims(n_kv_heads=3), _dims(pool_kernel=4),
                _dims(window=128)):
        assert lib.xkv_workspace_bytes(xkv.OP_SCORE, ctypes.byref(bad), 100, 100, 0, 0, 0) == 0
    assert lib.xkv_workspace_bytes(99, ctypes.byref(d), 100, 100, 1, 1, 0) == 0
    assert lib.xkv_workspace_bytes(xkv.OP_DECODE_ATTN, ctypes.byref(d), 0, 0, 4, 100, 32) == 0


def test_entry_points_reject_bad_arguments_before_any_cuda_call():
    lib = xkv.lib()
    d = _dims()
    # null pointers
    assert lib.xkv_score(ctypes.byref(d), None, None, None, 10, 10, None, None, None, None, 1, None, 0,
                         None) == xkv.ERR_INVALID_ARG
    # unsupported head_dim
    bad = _dims(head_dim=96)
    assert lib.xkv_score(ctypes.byref(bad), 16, 16, 16, 10, 10, 16, None, None, None, 1, 256, 0,
                         None) == xkv.ERR_UNSUPPORTED
    # misaligned pointer
    assert lib.xkv_score(ctypes.byref(d), 24, 16, 16, 10, 10, 16, None, None, None, 1, 256, 1 << 30,
                         None) == xkv.ERR_INVALID_ARG
    # workspace too small
    assert lib.xkv_score(ctypes.byref(d), 16, 16, 16, 1500, 1000, 16, None, None, None, 1, 256, 64,
                         None) == xkv.ERR_WORKSPACE
    cache = xkv.Cache(256, 512, 768, 1024, 4, 16, 8, 100)
    assert lib.xkv_decode_attn(ctypes.byref(d), ctypes.byref(cache), 0, 5, 16, None, None, 16, None, 0, 256,
                               1 << 30, None) == xkv.ERR_INVALID_ARG          # layer range
    assert lib.xkv_decode_attn(ctypes.byref(d), ctypes.byref(cache), 0, 4, 16, 16, None, 16, None, 0, 256,
                               1 << 30, None) == xkv.ERR_INVALID_ARG          # k_new without v_new
    assert lib.xkv_decode_attn(ctypes.byref(d), ctypes.byref(cache), 0, 4, 16, None, None, 16, None, 0, 256,
                               64, None) == xkv.ERR_WORKSPACE
    bad_cache = xkv.Cache(256, 512, 768, 1024, 4, 24, 8, 100)                 # page size not a multiple of 16
    assert lib.xkv_decode_attn(ctypes.byref(d), ctypes.byref(bad_cache), 0, 4, 16, None, None, 16, None, 0,
                               256, 1 << 30, None) == xkv.ERR_INVALID_ARG
    budget = np.array([-1], dtype=np.int32)
    assert lib.xkv_select_compact(ctypes.byref(d), 0, budget.ctypes.data, 0, 16, 16, 16, 16, 16, 1500, 1000,
                                  ctypes.byref(cache), None, 0, 256, 1 << 30, None) == xkv.ERR_BUDGET


def _curves(rng, L, B, n, power=3.0):
    g = np.zeros((L, B, n), dtype=np.float32)
    for l in range(L):
        for b in range(B):
            g[l, b] = O.head_gains(rng.random(n) ** (power + l))
    return g


@pytest.mark.parametrize("seed", range(4))
def test_alloc_budgets_matches_oracle_and_bruteforce(seed):
    rng = np.random.default_rng(seed)
    L, B, n = 3, 2, 6
    g = _curves(rng, L, B, n)
    mean = [c for c in O.batch_mean_gains(g.astype(np.float64))]
    for N in range(0, L * n + 1):
        budgets, r = xkv.alloc_budgets(g, [n] * B, total=N)
        assert budgets.sum() == N
        A, r_o = O.adaptive_allocation(mean, N=N)
        assert abs(r - r_o) < 1e-12 and budgets.tolist() == A
        if N <= 12:
            _, best = O.bruteforce_allocation(mean, N)
            assert abs(r - best) < 1e-12


def test_alloc_budgets_modes():
    rng = np.random.default_rng(7)
    L, B, n = 8, 3, 200
    g = _curves(rng, L, B, n, power=1.5)
    mean = [c for c in O.batch_mean_gains(g.astype(np.float64))]
    # box constraints
    budgets, r = xkv.alloc_budgets(g, [n] * B, total=400, n_min=10, n_max=120)
    A, r_o = O.adaptive_allocation(mean, N=400, n_min=10, n_max=120)
    assert budgets.tolist() == A and abs(r - r_o) < 1e-12 and budgets.min() >= 10 and budgets.max() <= 120
    # R target mode (Eq. 18)
    budgets, r = xkv.alloc_budgets(g, [n] * B, r_target=0.8)
    A, r_o = O.adaptive_allocation(mean, R_avg=0.8)
    assert budgets.tolist() == A and r >= 0.8 and abs(r - r_o) < 1e-12
    # per-sequence lists, ragged capacities
    prefix = [200, 150, 90]
    g2 = g.copy()
    for b, P in enumerate(prefix):
        g2[:, b, P:] = 0
    budgets, r = xkv.alloc_budgets(g2, prefix, per_sequence=True, total=300)
    assert budgets.shape == (B, L)
    for b, P in enumerate(prefix):
        A, r_o = O.adaptive_allocation([g2[l, b].astype(np.float64) for l in range(L)], N=300,
                                       capacity=[P] * L)
        assert budgets[b].tolist() == A and abs(r[b] - r_o) < 1e-12 and budgets[b].max() <= P
    # errors
    for kw in (dict(total=L * n + 1), dict(total=5, n_min=10), dict(r_target=1.5)):
        with pytest.raises(xkv.XkvError) as e:
            xkv.alloc_budgets(g, [n] * B, **kw)
        assert e.value.status == xkv.ERR_BUDGET
    # identical layers: ties go to the lowest layer index
    same = np.tile(O.head_gains(np.array([5.0, 4, 3, 2, 1])).astype(np.float32), (3, 1, 1))
    budgets, _ = xkv.alloc_budgets(same, [5], total=7)
    assert budgets.tolist() == [3, 2, 2]


@pytest.mark.parametrize("seed", range(3))
def test_alloc_budgets_ties_and_unsorted_curves(seed):
    """Sorted curves take the threshold solver, anything else the heap: both must grant like Algorithm 1, also when
    many positions of many layers hold the same value (ties go to the lowest layer, then the next position)."""
    rng = np.random.default_rng(100 + seed)
    L, n = 6, 40
    # few distinct values, non-increasing per layer, trailing zeros
    q = np.sort(rng.integers(0, 5, size=(L, 1, n)), axis=2)[:, :, ::-1].astype(np.float32) / 8.0
    gains = [q[l, 0].astype(np.float64) for l in range(L)]
    for N, n_min, n_max in [(0, 0, 0), (17, 0, 0), (95, 3, 25), (L * n, 0, 0), (60, 10, 10), (101, 2, 0)]:
        if n_max and N > L * n_max:
            continue
        budgets, r = xkv.alloc_budgets(q, [n], total=N, n_min=n_min, n_max=n_max)
        A, r_o = O.adaptive_allocation(gains, N=N, n_min=n_min, n_max=n_max or None)
        assert budgets.tolist() == A and abs(r - r_o) < 1e-12
    # curve shorter than the capacity: the positions beyond it count as zeros
    budgets, r = xkv.alloc_budgets(q[:, :, :10], [30], total=100)
    A, r_o = O.adaptive_allocation([g[:10] for g in gains], N=100, capacity=[30] * L)
    assert budgets.tolist() == A and abs(r - r_o) < 1e-12
    # unsorted curves (not what scoring produces, but the entry point accepts them)
    u = rng.random((L, 1, n)).astype(np.float32)
    for N in (12, 33, 150):
        budgets, r = xkv.alloc_budgets(u, [n], total=N, n_min=2)
        A, r_o = O.adaptive_allocation([u[l, 0].astype(np.float64) for l in range(L)], N=N, n_min=2)
        assert budgets.tolist() == A and abs(r - r_o) < 1e-12


def test_average_budgets_matches_oracle_and_keeps_the_total():
    """Online scenario (Sec. IV-C): layer-wise average of the recorded lists."""
    # by hand: means 4, 14/3, 22/3; recorded totals 16 each -> floors 4, 4, 7 and one slot to the larger fraction 2/3
    assert O.averaged_allocation([[3, 5, 8], [4, 4, 8], [5, 5, 6]]) == [4, 5, 7]
    assert xkv.average_budgets([[3, 5, 8], [4, 4, 8], [5, 5, 6]]).tolist() == [4, 5, 7]
    assert xkv.average_budgets([[1, 1], [2, 2]]).tolist() == [2, 1]            # equal fractions: the lower layer
    rng = np.random.default_rng(5)
    for n_tasks, L, N in [(1, 8, 100), (3, 32, 16384), (7, 5, 33), (10, 32, 65536)]:
        lists = rng.multinomial(N, rng.dirichlet(np.ones(L)), size=n_tasks)
        got = xkv.average_budgets(lists)
        assert got.tolist() == O.averaged_allocation(lists.tolist())
        assert got.sum() == N                                                   # every recorded list adds up to N
        mean = lists.mean(axis=0)
        assert np.all(got >= np.floor(mean)) and np.all(got <= np.floor(mean) + 1)
        if n_tasks == 1:
            assert got.tolist() == lists[0].tolist()
    with pytest.raises(xkv.XkvError):
        xkv.average_budgets([[1, -1]])
