"""CPU oracle for the XKV hot path -- TEST INFRASTRUCTURE, not part of the product.

Plain, slow, fp64 numpy restatement of what the paper's method computes, step by step and in the
paper's notation.  Only the tests, the smoke check and the CPU-baseline leg of the benchmark may
import it; the CUDA library never does, and nothing here imports the CUDA library.  No blocking,
fusion or reordering beyond what the cited passage states.

Inputs are the same bf16 tensors the GPU path receives, widened exactly to float64 by the caller.

Readings of the paper used here (each is the place where the paper is silent or garbled):
  * Merge sums over the window rows instead of averaging them (a constant factor: same ranking,
    same retention ratio R).
  * With grouped-query attention the window-summed weights of the G query heads that share one
    KV head are added before pooling; scores, selection and caches are per KV head.
  * Pooling has stride 1, keeps the length, the kernel is centred; max-pooling clips the kernel to
    the prefix, average-pooling pads with zeros and always divides by ps.
  * n_i counts prefix tokens only; the ows window tokens are always kept in addition.
  * TopK orders by (score descending, position ascending).
  * A layer's curve is the rank-wise mean over its heads of each head's sorted, self-normalised
    scores (for one head this is exactly Sort(w_i)/Sum(w_i) of Eq. 21).
  * Algorithm 1's wait value of a layer that holds pos slots is its (pos+1)-th largest normalised
    score (Eq. 21); the listing's slice expression is garbled.  Max(List_W) ties go to the lowest
    layer index.
  * Generation appends the new token's K/V first and then attends over all cached rows.

Parity pins live in tests/test_oracle_*.py; every function below is pinned there except where its
docstring says "parity unpinned".
"""
from __future__ import annotations

import itertools
import math

import numpy as np

NEG_INF = -np.inf


# ----------------------------------------------------------------------------------------------
# Alg. 2 step 1 / Eq. 2: attention weights
# ----------------------------------------------------------------------------------------------
def softmax_rows(S: np.ndarray) -> np.ndarray:
    """Row-wise softmax with the usual max subtraction; -inf entries get weight 0."""
    S = np.asarray(S, dtype=np.float64)
    m = np.max(S, axis=-1, keepdims=True)
    E = np.exp(S - m)
    return E / np.sum(E, axis=-1, keepdims=True)


def attention_weights(Q: np.ndarray, K: np.ndarray, scale: float | None = None) -> np.ndarray:
    """Eq. 2: W_attn = softmax(Q K^T / sqrt(d_k)) of a causal model, full t x t matrix.

    Q, K: [t, d].  Row i sees keys 0..i.
    """
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    t, d = K.shape
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    S = (Q @ K.T) * scale
    mask = np.tril(np.ones((t, t), dtype=bool))
    S = np.where(mask, S, NEG_INF)
    return softmax_rows(S)


def window_attention_weights(Q_win: np.ndarray, K: np.ndarray, scale: float | None = None) -> np.ndarray:
    """The last ows rows of Eq. 2's matrix, computed from the window queries alone.

    Q_win: [ows, d] queries of positions t-ows .. t-1;  K: [t, d].  Returns [ows, t]; row r sees
    keys c <= t - ows + r.  If t < ows only the last t rows are meaningful; earlier rows are 0.
    """
    Q_win = np.asarray(Q_win, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    ows, d = Q_win.shape
    t = K.shape[0]
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    out = np.zeros((ows, t), dtype=np.float64)
    for r in range(ows):
        pos = t - ows + r            # position of this query in the sequence
        if pos < 0:
            continue
        s = (K[: pos + 1] @ Q_win[r]) * scale
        out[r, : pos + 1] = softmax_rows(s[None, :])[0]
    return out


# ----------------------------------------------------------------------------------------------
# Alg. 2 steps 2-4 / Eq. 3: the attention-processing module f
# ----------------------------------------------------------------------------------------------
def select(W_rows: np.ndarray, ows: int) -> np.ndarray:
    """Alg. 2 step 2: rows of the last ows tokens, columns of the first t-ows tokens.

    W_rows holds the last ows rows of W_attn ([ows, t]).  Returns [ows, max(t-ows, 0)].
    """
    t = W_rows.shape[1]
    P = max(t - ows, 0)
    return W_rows[:, :P]


def merge(block: np.ndarray) -> np.ndarray:
    """Alg. 2 step 3: reduce the ows x (t-ows) block along its first dimension (sum)."""
    return np.sum(block, axis=0)


def pooling(u: np.ndarray, ps: int, mode: str = "max") -> np.ndarray:
    """Alg. 2 step 4: 1-D pooling, stride 1, same length, centred kernel of size ps (odd)."""
    u = np.asarray(u, dtype=np.float64)
    assert ps >= 1 and ps % 2 == 1
    P = u.shape[0]
    half = ps // 2
    w = np.empty(P, dtype=np.float64)
    for c in range(P):
        lo = max(c - half, 0)
        hi = min(c + half, P - 1)
        if mode == "max":
            w[c] = np.max(u[lo: hi + 1])
        elif mode == "avg":
            w[c] = np.sum(u[lo: hi + 1]) / ps
        else:
            raise ValueError(mode)
    return w


def column_scores(Q_win_group: np.ndarray, K: np.ndarray, ows: int, scale: float | None = None) -> np.ndarray:
    """Select + Merge for one KV head: u[c] = sum over the group's query heads and window rows.

    Q_win_group: [G, ows, d] (the G query heads sharing this KV head);  K: [t, d].  Returns [t-ows].
    """
    t = K.shape[0]
    P = max(t - ows, 0)
    u = np.zeros(P, dtype=np.float64)
    for Qh in Q_win_group:
        u += merge(select(window_attention_weights(Qh, K, scale), ows))
    return u


def score_vector(Q_win_group: np.ndarray, K: np.ndarray, ows: int, ps: int, mode: str = "max",
                 scale: float | None = None) -> np.ndarray:
    """Eq. 3: w = f(W_attn, ows) for one KV head -- Select, Merge, Pooling."""
    return pooling(column_scores(Q_win_group, K, ows, scale), ps, mode)


# ----------------------------------------------------------------------------------------------
# Eq. 4: importance-retention ratio, and the curves Algorithm 1 consumes
# ----------------------------------------------------------------------------------------------
def sort_descending(w: np.ndarray) -> np.ndarray:
    return np.sort(np.asarray(w, dtype=np.float64))[::-1]


def retention_ratio(w: np.ndarray, n: int) -> float:
    """Eq. 4 as a fraction: R = Sum(TopK(n, w)) / Sum(w)."""
    w = np.asarray(w, dtype=np.float64)
    return float(np.sum(sort_descending(w)[:n]) / np.sum(w))


def head_gains(w: np.ndarray) -> np.ndarray:
    """Sort(w)[-(j+1)] / Sum(w) for j = 0..len-1 (the terms of Eq. 21); empty or all-zero w -> zeros."""
    w = np.asarray(w, dtype=np.float64)
    if w.size == 0:
        return np.zeros(0, dtype=np.float64)
    total = np.sum(w)
    if total <= 0.0:
        return np.zeros(w.size, dtype=np.float64)
    return sort_descending(w) / total


def layer_gains(w_heads: list[np.ndarray], curve_len: int) -> np.ndarray:
    """Rank-wise mean over a layer's heads of head_gains; ranks beyond a head's length count 0."""
    g = np.zeros(curve_len, dtype=np.float64)
    for w in w_heads:
        hg = head_gains(w)[:curve_len]
        g[: hg.size] += hg
    return g / max(len(w_heads), 1)


def retained_mass(gains: np.ndarray) -> np.ndarray:
    """mass[n] = sum_{j<=n} gains[j]: R after keeping n+1 tokens per head."""
    return np.cumsum(np.asarray(gains, dtype=np.float64))


# ----------------------------------------------------------------------------------------------
# Algorithm 1: adaptive allocation
# ----------------------------------------------------------------------------------------------
def adaptive_allocation(gains: list[np.ndarray], N: int | None = None, R_avg: float | None = None,
                        n_min: int = 0, n_max: int | None = None,
                        capacity: list[int] | None = None) -> tuple[list[int], float]:
    """Algorithm 1 (adaptive allocation).  gains[i][j] is layer i's (j+1)-th largest normalised score,
    i.e. the increase of R_i (Eq. 4) when layer i keeps one more token (Eq. 21).

    Every layer offers the gain of the next token it would keep; one slot at a time goes to the layer whose
    offer is largest (the lowest layer among equal offers), and that layer then offers its following token.
    Mode N (Eq. 17): stop after N slots.  Mode R_avg (Eq. 18): stop as soon as the mean over layers of the
    retained ratio reaches R_avg.  Returns (slots per layer, mean over layers of the retained ratio).
    """
    n_layers = len(gains)
    room = [len(g) for g in gains] if capacity is None else list(capacity)
    if n_max is not None:
        room = [min(c, n_max) for c in room]

    def offer(i: int) -> float:
        # gain of the token layer i would keep next; a full layer offers nothing, ranks past the curve add 0
        if held[i] >= room[i]:
            return NEG_INF
        return float(gains[i][held[i]]) if held[i] < len(gains[i]) else 0.0

    held = [min(n_min, room[i]) for i in range(n_layers)]
    retained = sum(float(np.sum(np.asarray(gains[i][: held[i]], dtype=np.float64))) for i in range(n_layers))

    def give_one_slot() -> None:
        nonlocal retained
        offers = [offer(i) for i in range(n_layers)]
        best = max(offers)
        if best == NEG_INF:
            raise ValueError("budget exceeds capacity")
        winner = offers.index(best)            # lowest layer index among equal offers
        held[winner] += 1
        retained += best

    if N is not None:
        if N < sum(held):
            raise ValueError("N below the n_min floor")
        while sum(held) < N:
            give_one_slot()
    elif R_avg is not None:
        if not (0.0 < R_avg <= 1.0 + 1e-12):
            raise ValueError("R_avg target out of range")
        while retained / n_layers < R_avg:
            give_one_slot()
    else:
        raise ValueError("give N or R_avg")
    return held, retained / n_layers


def allocation_objective(gains: list[np.ndarray], List_A: list[int]) -> float:
    """Objective of Eq. 17: mean over layers of R_i(n_i)."""
    return sum(float(np.sum(np.asarray(g[:n], dtype=np.float64))) for g, n in zip(gains, List_A)) / len(gains)


def averaged_allocation(lists: list[list[int]]) -> list[int]:
    """Online scenario (Sec. IV-C): the allocation lists recorded for the sampled tasks are averaged layer by
    layer and the averaged list is applied to later tasks of the same type.

    The paper does not say how the averages become integers.  Reading taken here: every layer gets the floor of
    its mean, and the slots this leaves over (so that the list adds up to the rounded mean of the recorded
    totals) go one each to the layers with the largest fractional parts, lower layer first among equals.
    Exact integer arithmetic throughout.
    """
    n = len(lists)
    L = len(lists[0])
    sums = [sum(int(lst[i]) for lst in lists) for i in range(L)]
    base = [s // n for s in sums]
    rem = [s % n for s in sums]                       # fractional part of layer i's mean is rem[i] / n
    total = sum(sums)
    target = (2 * total + n) // (2 * n)               # mean of the recorded totals, rounded half up
    left = target - sum(base)
    order = sorted(range(L), key=lambda i: (-rem[i], i))
    out = list(base)
    for i in order[:left]:
        out[i] += 1
    return out


def bruteforce_allocation(gains: list[np.ndarray], N: int, n_min: int = 0,
                          n_max: int | None = None) -> tuple[list[int], float]:
    """Enumerate every split of N over the layers (tiny inputs only) and return the best of Eq. 17."""
    L = len(gains)
    cap = [len(g) if n_max is None else min(len(g), n_max) for g in gains]
    best, best_val = None, -1.0
    for split in itertools.product(*[range(min(n_min, cap[i]), cap[i] + 1) for i in range(L)]):
        if sum(split) != N:
            continue
        val = allocation_objective(gains, list(split))
        if val > best_val:
            best, best_val = list(split), val
    if best is None:
        raise ValueError("no feasible split")
    return best, best_val


def head_level_allocation(w_layers: list[list[np.ndarray]], N: int | None = None, R_avg: float | None = None,
                          n_min: int = 0, n_max: int | None = None) -> tuple[list[list[int]], float]:
    """Head-level budgets inside the layers (Sec. II-C: cache sizes pre-set per attention head work together with
    the layer-centric allocation).  Reading taken here: the unit that waits for slots in Algorithm 1 is a
    (layer, KV head) pair instead of a layer, each with its own curve Sort(w)/Sum(w) (Eq. 21 for that head);
    N is then the number of cached prefix tokens summed over all heads of all layers, and the objective is the
    mean over all heads of Eq. 4.  Units are ordered layer-major, so ties go to the lower layer, then the lower
    head.

    w_layers[l][g]: pooled score vector of KV head g of layer l (one sequence).  Returns (n[l][g], mean R).
    """
    flat = [head_gains(w) for heads in w_layers for w in heads]
    held, r = adaptive_allocation(flat, N=N, R_avg=R_avg, n_min=n_min, n_max=n_max)
    out, i = [], 0
    for heads in w_layers:
        out.append(held[i: i + len(heads)])
        i += len(heads)
    return out, r


def batch_mean_gains(gains_lb: np.ndarray) -> np.ndarray:
    """gains_lb [L, B, curve_len] -> [L, curve_len]: mean over the sequences of a batch."""
    return np.mean(np.asarray(gains_lb, dtype=np.float64), axis=1)


# ----------------------------------------------------------------------------------------------
# Alg. 2 steps 5-7: TopK and EvictByIndex
# ----------------------------------------------------------------------------------------------
def topk_indices(w: np.ndarray, n: int) -> np.ndarray:
    """Alg. 2 step 5: positions of the n largest entries, ties to the lower position, ascending."""
    w = np.asarray(w, dtype=np.float64)
    P = w.shape[0]
    n = min(max(n, 0), P)
    order = np.lexsort((np.arange(P), -w))   # primary key: score descending; secondary: position
    return np.sort(order[:n]).astype(np.int64)


def kept_positions(w: np.ndarray, n: int, t: int, ows: int) -> np.ndarray:
    """The retained positions of one head: TopK over the prefix, then the window positions."""
    P = max(t - ows, 0)
    assert w.shape[0] == P
    return np.concatenate([topk_indices(w, n), np.arange(P, t, dtype=np.int64)])


def evict_by_index(X: np.ndarray, index: np.ndarray) -> np.ndarray:
    """Alg. 2 steps 6-7: keep the rows listed in index, in that order (any dtype, bit-exact copy)."""
    return np.asarray(X)[np.asarray(index, dtype=np.int64)].copy()


# ----------------------------------------------------------------------------------------------
# Eq. 1: generation-phase attention over a reduced cache
# ----------------------------------------------------------------------------------------------
def decode_attention(q: np.ndarray, K_c: np.ndarray, V_c: np.ndarray,
                     scale: float | None = None) -> tuple[np.ndarray, float]:
    """Eq. 1 for one query row: z = softmax(q K_c^T / sqrt(d_k)) V_c.  Returns (z, log-sum-exp)."""
    q = np.asarray(q, dtype=np.float64)
    K_c = np.asarray(K_c, dtype=np.float64)
    V_c = np.asarray(V_c, dtype=np.float64)
    d = q.shape[0]
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    if K_c.shape[0] == 0:
        return np.zeros(V_c.shape[1] if V_c.ndim == 2 else d, dtype=np.float64), NEG_INF
    s = (K_c @ q) * scale
    m = np.max(s)
    e = np.exp(s - m)
    return (e / np.sum(e)) @ V_c, float(m + math.log(np.sum(e)))


# ----------------------------------------------------------------------------------------------
# A reduced cache stored with few bits (Sec. II-B: quantisation is compatible with eviction)
# ----------------------------------------------------------------------------------------------
# The paper names no format.  Reading taken here: every cached row (one token of one KV head, K and V separately)
# is stored as 8-bit integers times one fp32 scale per row: scale = max|x| / 127 (1 for an all-zero row),
# q = x / scale rounded to the nearest integer, ties to even, kept within [-127, 127]; the stored byte is q + 128.
# Where floating point decides the integer, the decision is taken in fp32 (the division by 127, the division by the
# scale), which is the precision of the CUDA path.
INT8_MAX = 127


def quantize_rows_int8(X: np.ndarray) -> tuple[np.ndarray, np.ndarray]:
    """Rows of X [n, d] -> (stored bytes uint8 [n, d] = q + 128, scales float32 [n])."""
    X32 = np.asarray(X, dtype=np.float32)
    amax = np.max(np.abs(X32), axis=1) if X32.shape[0] else np.zeros(0, dtype=np.float32)
    scales = np.where(amax > 0, amax / np.float32(INT8_MAX), np.float32(1.0)).astype(np.float32)
    y = (X32 / scales[:, None]).astype(np.float32)              # fp32 division, as on the GPU
    q = np.clip(np.rint(y.astype(np.float64)), -INT8_MAX, INT8_MAX).astype(np.int64)   # rint: ties to even
    return (q + 128).astype(np.uint8), scales


def dequantize_rows_int8(stored: np.ndarray, scales: np.ndarray) -> np.ndarray:
    """What the computation recovers from a stored row: (byte - 128) times the row's scale (float64)."""
    return (np.asarray(stored, dtype=np.int64) - 128).astype(np.float64) * np.asarray(scales, dtype=np.float64)[:, None]


# ----------------------------------------------------------------------------------------------
# Eq. 1 / Eq. 2 over the whole prompt: the prefill attention whose last ows rows are W_attn of Alg. 2 step 1
# ----------------------------------------------------------------------------------------------
def prefill_attention(Q: np.ndarray, K: np.ndarray, V: np.ndarray,
                      scale: float | None = None) -> tuple[np.ndarray, np.ndarray]:
    """Causal attention of one head over a prompt of t tokens: Z = softmax(Q K^T / sqrt(d_k)) V (Eq. 1 with the
    weights of Eq. 2), row i seeing keys 0..i.  Q, K, V: [t, d].  Returns (Z [t, d], lse [t]) where lse[i] is the
    natural log of the sum over the visible keys of exp(scaled logit): the softmax normaliser of row i, which
    for the last ows rows is the normaliser of the observation-window weights (Alg. 2 step 1)."""
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    t, d = K.shape
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    Z = attention_weights(Q, K, scale) @ V
    S = (Q @ K.T) * scale
    lse = np.empty(t, dtype=np.float64)
    for i in range(t):
        row = S[i, : i + 1]
        m = np.max(row)
        lse[i] = m + math.log(np.sum(np.exp(row - m)))
    return Z, lse


def column_scores_from_lse(Q_win_group: np.ndarray, K: np.ndarray, lse_rows: np.ndarray, ows: int,
                           scale: float | None = None) -> np.ndarray:
    """Select + Merge when the prefill attention has already produced the normalisers of the window rows
    (Alg. 2 step 1 takes W_attn from the layer's own attention): u[c] = sum over the group's query heads and
    window rows of exp(scaled logit - lse).  Q_win_group [G, ows, d], K [t, d], lse_rows [G, ows] (rows of
    positions t-ows .. t-1).  Returns [max(t-ows, 0)]."""
    K = np.asarray(K, dtype=np.float64)
    t, d = K.shape
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    P = max(t - ows, 0)
    u = np.zeros(P, dtype=np.float64)
    for Qh, lh in zip(np.asarray(Q_win_group, dtype=np.float64), np.asarray(lse_rows, dtype=np.float64)):
        for r in range(ows):
            if t - ows + r < 0:
                continue
            u += np.exp((K[:P] @ Qh[r]) * scale - lh[r])
    return u


# ----------------------------------------------------------------------------------------------
# The path end to end on packed batches (same layouts the C ABI uses, numpy arrays)
# ----------------------------------------------------------------------------------------------
def score_layer(q_win: np.ndarray, k: np.ndarray, cu_seqlens: np.ndarray, ows: int, ps: int,
                mode: str = "max", scale: float | None = None,
                units: list[tuple[int, int]] | None = None) -> dict[tuple[int, int], np.ndarray]:
    """w for the (b, g) units of one layer.  q_win [B,Hq,ows,d], k [T,Hkv,d] (float64).

    Sequences shorter than ows use the last t_b query rows.
    """
    B, Hq = q_win.shape[0], q_win.shape[1]
    Hkv = k.shape[1]
    G = Hq // Hkv
    out = {}
    for b in range(B):
        lo, hi = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
        for g in range(Hkv):
            if units is not None and (b, g) not in units:
                continue
            out[(b, g)] = score_vector(q_win[b, g * G:(g + 1) * G], k[lo:hi, g], ows, ps, mode, scale)
    return out


def layer_curves(w_units: dict[tuple[int, int], np.ndarray], B: int, Hkv: int,
                 curve_len: int) -> np.ndarray:
    """gains [B, curve_len] of one layer from all its (b, g) score vectors."""
    return np.stack([layer_gains([w_units[(b, g)] for g in range(Hkv)], curve_len) for b in range(B)])


def near_tie(w: np.ndarray, n: int, rel: float = 1e-5) -> bool:
    """True if some score other than exact copies of the n-th largest lies within rel of it.

    Inside that band a path that computes scores in lower precision may legitimately keep a
    different token; outside it the kept set is unique.
    """
    w = np.asarray(w, dtype=np.float64)
    P = w.shape[0]
    if n <= 0 or n >= P:
        return False
    thr = sort_descending(w)[n - 1]
    band = np.abs(w - thr) <= rel * abs(thr)
    return bool(np.any(band & (w != thr)))
