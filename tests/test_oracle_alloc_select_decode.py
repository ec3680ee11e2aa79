"""Pins for the oracle's solver (Alg. 1; Eq. 17, 18, 21), TopK / EvictByIndex (Alg. 2 steps 5-7) and
generation attention (Eq. 1): brute force, invariants, closed forms, library cross-checks."""
import itertools
import math

import numpy as np
import pytest
import torch

from oracle import xkv_oracle as O


def _random_gains(rng, L, lens, power=3.0):
    return [O.head_gains(rng.random(n) ** power) for n in lens[:L]]


# ------------------------------------------------------------------ Algorithm 1
@pytest.mark.parametrize("seed", range(6))
def test_allocation_matches_bruteforce_objective(seed):
    rng = np.random.default_rng(seed)
    L = int(rng.integers(2, 5))
    lens = [int(rng.integers(3, 7)) for _ in range(L)]
    gains = _random_gains(rng, L, lens)
    for N in range(0, min(sum(lens), 14) + 1):
        A, r = O.adaptive_allocation(gains, N=N)
        assert sum(A) == N                                           # constraint of Eq. 17
        best, best_val = O.bruteforce_allocation(gains, N)
        assert abs(r - best_val) < 1e-13
        assert abs(O.allocation_objective(gains, A) - r) < 1e-13


def test_allocation_with_box_matches_bruteforce():
    rng = np.random.default_rng(11)
    gains = _random_gains(rng, 3, [6, 6, 6])
    for N in range(3, 13):
        A, r = O.adaptive_allocation(gains, N=N, n_min=1, n_max=4)
        assert sum(A) == N and all(1 <= a <= 4 for a in A)
        _, best_val = O.bruteforce_allocation(gains, N, n_min=1, n_max=4)
        assert abs(r - best_val) < 1e-13
    with pytest.raises(ValueError):
        O.adaptive_allocation(gains, N=13, n_min=1, n_max=4)
    with pytest.raises(ValueError):
        O.adaptive_allocation(gains, N=2, n_min=1, n_max=4)


def test_allocation_threshold_and_exchange_property():
    rng = np.random.default_rng(12)
    gains = _random_gains(rng, 5, [40, 30, 50, 20, 35])
    N = 60
    A, r = O.adaptive_allocation(gains, N=N)
    granted = [gains[i][A[i] - 1] for i in range(5) if A[i] > 0]
    waiting = [gains[i][A[i]] for i in range(5) if A[i] < len(gains[i])]
    assert min(granted) >= max(waiting)
    # Eq. 21: moving one slot between any two layers never increases the objective
    for i, j in itertools.permutations(range(5), 2):
        if A[i] < len(gains[i]) and A[j] > 0:
            B = list(A); B[i] += 1; B[j] -= 1
            delta = (gains[i][A[i]] - gains[j][A[j] - 1]) / 5
            assert abs(O.allocation_objective(gains, B) - r - delta) < 1e-13
            assert delta <= 1e-15


def test_allocation_r_target_is_shortest_prefix_of_total_mode():
    rng = np.random.default_rng(13)
    gains = _random_gains(rng, 4, [25, 25, 25, 25])
    for target in (0.2, 0.5, 0.9, 1.0):
        A, r = O.adaptive_allocation(gains, R_avg=target)
        n = sum(A)
        assert r >= target
        A_same, r_same = O.adaptive_allocation(gains, N=n)
        assert A_same == A and abs(r_same - r) < 1e-15
        if n > 0:
            _, r_less = O.adaptive_allocation(gains, N=n - 1)
            assert r_less < target
    with pytest.raises(ValueError):
        O.adaptive_allocation(gains, R_avg=1.5)


def test_allocation_identical_layers_split_evenly_lowest_index_first():
    g = O.head_gains(np.array([5.0, 4.0, 3.0, 2.0, 1.0]))
    A, _ = O.adaptive_allocation([g, g, g], N=7)
    assert A == [3, 2, 2]
    A, _ = O.adaptive_allocation([g, g, g], N=15)
    assert A == [5, 5, 5]


def test_allocation_single_layer_and_batch_mean():
    g = O.head_gains(np.array([1.0, 2.0, 3.0]))
    A, r = O.adaptive_allocation([g], N=2)
    assert A == [2] and abs(r - 5.0 / 6.0) < 1e-15
    # batch mean of the curves, numbers written out by hand: 2 layers x 2 sequences x 3 ranks
    x = np.array([[[0.50, 0.25, 0.25], [0.70, 0.20, 0.00]],
                  [[1.00, 0.00, 0.00], [0.40, 0.35, 0.25]]])
    want = np.array([[0.60, 0.225, 0.125],
                     [0.70, 0.175, 0.125]])
    got = O.batch_mean_gains(x)
    assert got.shape == (2, 3) and np.max(np.abs(got - want)) < 1e-15
    # a sequence shorter than the others contributes zeros beyond its prefix: the mean is over all B sequences
    y = np.array([[[0.9, 0.1, 0.0, 0.0], [0.4, 0.3, 0.2, 0.1], [1.0, 0.0, 0.0, 0.0]]])
    assert np.max(np.abs(O.batch_mean_gains(y) - np.array([[2.3 / 3, 0.4 / 3, 0.2 / 3, 0.1 / 3]]))) < 1e-15


# ------------------------------------------------------------------ head-level budgets (Sec. II-C)
def _bruteforce_heads(w_layers, N):
    """Every split of N over the (layer, head) units; best mean over the units of Eq. 4, written out here."""
    units = [np.sort(w)[::-1] / np.sum(w) for heads in w_layers for w in heads]
    best = -1.0
    for split in itertools.product(*[range(len(u) + 1) for u in units]):
        if sum(split) == N:
            best = max(best, sum(float(np.sum(u[:n])) for u, n in zip(units, split)) / len(units))
    return best


@pytest.mark.parametrize("seed", range(4))
def test_head_level_allocation_matches_bruteforce(seed):
    rng = np.random.default_rng(100 + seed)
    w_layers = [[rng.random(int(rng.integers(2, 5))) ** 3 for _ in range(2)] for _ in range(2)]   # 2 layers x 2 heads
    total = sum(len(w) for heads in w_layers for w in heads)
    for N in range(0, total + 1):
        n, r = O.head_level_allocation(w_layers, N=N)
        assert sum(sum(row) for row in n) == N
        assert [len(row) for row in n] == [2, 2]
        assert abs(r - _bruteforce_heads(w_layers, N)) < 1e-13


def test_head_level_allocation_against_the_layer_level_one():
    rng = np.random.default_rng(7)
    L, H, P = 3, 4, 12
    # heads that differ: the head-level optimum is at least the layer-level one spread over the heads (which is a
    # feasible point of the head-level problem with H times the slots), and strictly better for these scores
    w_layers = [[rng.random(P) ** 4 for _ in range(H)] for _ in range(L)]
    layer_curves = [O.layer_gains(heads, P) for heads in w_layers]
    for N in (3, 9, 20):
        A, r_layer = O.adaptive_allocation(layer_curves, N=N)
        n, r_head = O.head_level_allocation(w_layers, N=H * N)
        spread = sum(float(np.sum(O.head_gains(w)[:A[l]])) for l in range(L) for w in w_layers[l]) / (L * H)
        assert abs(spread - r_layer) < 1e-13                       # the layer curve is the mean of its heads' curves
        assert r_head >= r_layer - 1e-15
    assert r_head > r_layer + 1e-6
    # identical heads inside every layer: each head gets exactly its layer's count
    w_same = [[w] * H for w in (rng.random(P) ** 3 for _ in range(L))]
    curves = [O.head_gains(heads[0]) for heads in w_same]
    for N in (1, 7, 15, 30):
        A, r_layer = O.adaptive_allocation(curves, N=N)
        n, r_head = O.head_level_allocation(w_same, N=H * N)
        assert n == [[a] * H for a in A] and abs(r_head - r_layer) < 1e-13
    # by hand: one layer, two heads w0 = (6, 3, 1) and w1 = (5, 5): the curves are (.6, .3, .1) and (.5, .5); three
    # slots go to .6, then .5 (head 1), then .5 (head 1)
    n, r = O.head_level_allocation([[np.array([1.0, 6.0, 3.0]), np.array([5.0, 5.0])]], N=3)
    assert n == [[1, 2]] and abs(r - (0.6 + 1.0) / 2) < 1e-15
    # the box applies per head
    n, _ = O.head_level_allocation([[np.array([1.0, 6.0, 3.0]), np.array([5.0, 5.0])]], N=3, n_min=1, n_max=2)
    assert n == [[1, 2]]


# ------------------------------------------------------------------ TopK / EvictByIndex
def test_topk_matches_bruteforce_sort():
    rng = np.random.default_rng(20)
    for _ in range(20):
        P = int(rng.integers(1, 30))
        w = rng.integers(0, 6, size=P).astype(np.float64)          # many ties
        for n in range(0, P + 2):
            order = sorted(range(P), key=lambda c: (-w[c], c))
            assert O.topk_indices(w, n).tolist() == sorted(order[: min(n, P)])


def test_topk_special_cases():
    assert O.topk_indices(np.full(9, 0.25), 4).tolist() == [0, 1, 2, 3]       # ties -> lowest positions
    e = np.zeros(20); e[11] = 1.0
    plateau = O.pooling(e, 7, "max")                                          # positions 8..14
    assert O.topk_indices(plateau, 3).tolist() == [8, 9, 10]
    assert O.topk_indices(plateau, 7).tolist() == list(range(8, 15))
    assert O.topk_indices(plateau, 9).tolist() == [0, 1] + list(range(8, 15))
    w = np.array([0.1, 0.9, 0.3])
    assert O.topk_indices(w, 5).tolist() == [0, 1, 2] and O.topk_indices(w, 0).tolist() == []
    assert O.kept_positions(w, 1, 5, 2).tolist() == [1, 3, 4]
    assert O.kept_positions(np.zeros(0), 3, 2, 4).tolist() == [0, 1]          # t < ows: keep all


def test_near_tie_band():
    w = np.array([1.0, 0.5, 0.5 * (1 + 5e-6), 0.2, 0.5])
    assert O.near_tie(w, 2) and O.near_tie(w, 3)
    assert not O.near_tie(w, 1)
    assert not O.near_tie(np.array([1.0, 0.5, 0.5, 0.2]), 2)   # exact copies are not near-ties
    assert not O.near_tie(w, 0) and not O.near_tie(w, 5)


def test_evict_by_index_is_bit_exact_and_full_budget_is_identity():
    rng = np.random.default_rng(21)
    X = rng.integers(0, 2 ** 16, size=(12, 4), dtype=np.uint16)
    idx = np.array([0, 3, 4, 11])
    Y = O.evict_by_index(X, idx)
    assert Y.dtype == np.uint16 and np.array_equal(Y, X[[0, 3, 4, 11]])
    w = rng.random(10)
    full = O.kept_positions(w, 99, 12, 2)
    assert np.array_equal(O.evict_by_index(X, full), X)


# ------------------------------------------------------------------ Eq. 1 decode
def test_decode_full_budget_reproduces_full_attention_bitwise():
    rng = np.random.default_rng(30)
    t, d, ows = 50, 16, 4
    K, V, q = rng.normal(size=(t, d)), rng.normal(size=(t, d)), rng.normal(size=d)
    w = rng.random(t - ows)
    idx = O.kept_positions(w, t, t, ows)
    z_full, lse_full = O.decode_attention(q, K, V)
    z_c, lse_c = O.decode_attention(q, O.evict_by_index(K, idx), O.evict_by_index(V, idx))
    assert np.array_equal(z_full, z_c) and lse_full == lse_c


def test_decode_single_row_permutation_and_torch():
    rng = np.random.default_rng(31)
    n, d = 33, 8
    K, V, q = rng.normal(size=(n, d)), rng.normal(size=(n, d)), rng.normal(size=d)
    z1, _ = O.decode_attention(q, K[:1], V[:1])
    assert np.allclose(z1, V[0], atol=1e-15)
    z, lse = O.decode_attention(q, K, V)
    perm = rng.permutation(n)
    zp, lsep = O.decode_attention(q, K[perm], V[perm])
    assert np.allclose(z, zp, atol=1e-12) and abs(lse - lsep) < 1e-12
    s = torch.from_numpy(K) @ torch.from_numpy(q) / math.sqrt(d)
    ref = torch.softmax(s, 0) @ torch.from_numpy(V)
    assert np.allclose(z, ref.numpy(), atol=1e-14)
    assert abs(lse - torch.logsumexp(s, 0).item()) < 1e-13
    z0, lse0 = O.decode_attention(q, K[:0], V[:0])
    assert np.all(z0 == 0) and lse0 == -np.inf


@pytest.mark.parametrize("splits", [2, 3, 7])
def test_decode_split_and_lse_merge_is_invariant(splits):
    rng = np.random.default_rng(32)
    n, d = 61, 8
    K, V, q = rng.normal(size=(n, d)) * 3, rng.normal(size=(n, d)), rng.normal(size=d)
    z, lse = O.decode_attention(q, K, V)
    bounds = np.linspace(0, n, splits + 1).astype(int)
    parts = [O.decode_attention(q, K[a:b], V[a:b]) for a, b in zip(bounds[:-1], bounds[1:])]
    m = max(p[1] for p in parts)
    wts = np.array([math.exp(p[1] - m) for p in parts])
    merged = sum(wi * p[0] for wi, p in zip(wts, parts)) / wts.sum()
    assert np.allclose(merged, z, atol=1e-12)
    assert abs(m + math.log(wts.sum()) - lse) < 1e-12


# ------------------------------------------------------------------ 8-bit rows of a reduced cache (Sec. II-B)
def test_int8_rows_by_hand():
    # one row whose largest entry is 127 so that the scale is exactly 1: the integers are the rounded entries,
    # halves go to the even neighbour, the stored byte is the integer plus 128
    x = np.array([[127.0, -127.0, 0.0, 0.5, 1.5, 2.5, -0.5, -1.5, 3.49, 3.51, -126.5, 100.25]])
    stored, scales = O.quantize_rows_int8(x)
    assert scales.tolist() == [1.0]
    assert (stored.astype(int) - 128).tolist() == [[127, -127, 0, 0, 2, 2, 0, -2, 3, 4, -126, 100]]
    assert np.array_equal(O.dequantize_rows_int8(stored, scales), (stored.astype(np.float64) - 128))
    # scale = max|x| / 127 in fp32; the largest entry maps to +-127 exactly; an all-zero row keeps scale 1
    y = np.array([[0.25, -2.0, 1.0], [0.0, 0.0, 0.0], [3.0, 0.0, -0.01]])
    st, sc = O.quantize_rows_int8(y)
    assert sc.dtype == np.float32 and st.dtype == np.uint8
    assert sc[0] == np.float32(2.0) / np.float32(127) and sc[1] == 1.0 and sc[2] == np.float32(3.0) / np.float32(127)
    assert (st.astype(int) - 128)[:, :2].tolist() == [[16, -127], [0, 0], [127, 0]]        # 0.25 * 63.5 = 15.875 -> 16
    assert (st.astype(int) - 128)[1:, 2].tolist() == [0, 0]


def test_quantized_rows_scale_round_trip_and_error_bound():
    rng = np.random.default_rng(50)
    X = torch.from_numpy(rng.standard_normal((40, 128)) * rng.uniform(0.01, 30, (40, 1))).to(torch.bfloat16)
    X = X.float().numpy().astype(np.float64)
    X[3] = 0.0
    X[5, :] = 0.0
    X[5, 17] = -3.0                                             # a one-hot row: its entry becomes -127 * scale
    stored, scales = O.quantize_rows_int8(X)
    assert scales[3] == 1.0 and np.all(stored[3] == 128)
    assert stored[5, 17] == 1 and np.all(np.delete(stored[5], 17) == 128)
    back = O.dequantize_rows_int8(stored, scales)
    assert abs(back[5, 17] + 3.0) < 1e-6
    amax = np.abs(X).max(axis=1)
    nz = amax > 0
    assert np.allclose(scales[nz], amax[nz] / 127.0, rtol=1e-7)
    assert np.all(np.abs(stored.astype(int) - 128).max(axis=1)[nz] == 127) and stored.min() >= 1
    # the error is half a step of the row's grid (plus the fp32 roundings of scale and quotient)
    assert np.all(np.abs(back - X) <= 0.5 * scales[:, None].astype(np.float64) * (1 + 1e-5))
    # stored rows are a fixed point: quantising what was recovered gives the same bytes and scales
    stored2, scales2 = O.quantize_rows_int8(back)
    assert np.array_equal(stored2, stored) and np.array_equal(scales2, scales)
    # brute force on a small row: the nearest grid point, ties to the even integer
    row = X[7:8, :16]
    st, sc = O.quantize_rows_int8(row)
    for j in range(16):
        y = float(np.float32(row[0, j]) / sc[0])
        cands = sorted(range(-127, 128), key=lambda n: (abs(n - y), n % 2))
        assert int(st[0, j]) - 128 == cands[0]
