"""Pins for the oracle's scoring half (Eq. 2, Eq. 3, Eq. 4; Alg. 2 steps 1-4): closed forms,
a hand-derived rational example, invariants and torch-fp64 library cross-checks."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import xkv_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            key, *vals = line.split()
            out[key] = np.array([float(v) for v in vals])
    return out


def test_softmax_rows_sum_to_one_and_match_torch():
    rng = np.random.default_rng(0)
    t, d = 37, 16
    Q, K = rng.normal(size=(t, d)), rng.normal(size=(t, d))
    Wa = O.attention_weights(Q, K)
    assert np.allclose(Wa.sum(axis=1), 1.0, atol=1e-12)
    assert np.all(np.triu(Wa, 1) == 0.0)                      # causal
    S = torch.from_numpy(Q) @ torch.from_numpy(K).T / math.sqrt(d)
    S = S.masked_fill(~torch.tril(torch.ones(t, t, dtype=torch.bool)), float("-inf"))
    assert np.allclose(Wa, torch.softmax(S, dim=-1).numpy(), atol=1e-14)


def test_window_rows_are_the_last_rows_of_the_full_matrix():
    rng = np.random.default_rng(1)
    t, d, ows = 29, 8, 5
    Q, K = rng.normal(size=(t, d)), rng.normal(size=(t, d))
    full = O.attention_weights(Q, K)
    win = O.window_attention_weights(Q[t - ows:], K)
    assert np.allclose(win, full[t - ows:], atol=1e-14)
    assert np.allclose(win.sum(axis=1), 1.0, atol=1e-12)
    # the selected ows x (t-ows) block has rows that sum to less than one
    assert np.all(O.select(win, ows).sum(axis=1) < 1.0)
    assert O.select(win, ows).shape == (ows, t - ows)


def test_identical_keys_give_uniform_weights_closed_form():
    t, d, ows, G = 23, 4, 6, 3
    P = t - ows
    K = np.tile(np.array([[0.3, -1.0, 2.0, 0.5]]), (t, 1))
    rng = np.random.default_rng(2)
    Qg = rng.normal(size=(G, ows, d))
    win = O.window_attention_weights(Qg[0], K)
    for r in range(ows):
        assert np.allclose(win[r, : P + r + 1], 1.0 / (P + r + 1), atol=1e-14)
        assert np.all(win[r, P + r + 1:] == 0.0)
    u = O.column_scores(Qg, K, ows)
    expect = G * sum(1.0 / (P + r + 1) for r in range(ows))
    assert u.shape == (P,)
    assert np.allclose(u, expect, atol=1e-13)


def test_single_row_single_head_is_one_softmax_row():
    rng = np.random.default_rng(3)
    t, d = 17, 8
    q, K = rng.normal(size=(1, 1, d)), rng.normal(size=(t, d))
    u = O.column_scores(q, K, 1)
    s = K @ q[0, 0] / math.sqrt(d)
    p = np.exp(s - s.max()); p /= p.sum()
    assert np.allclose(u, p[: t - 1], atol=1e-14)


def test_hand_derived_rational_example():
    g = _golden("window_scores_rational.txt")
    a = g["a"]
    K = np.log(a)[:, None]
    Qw = np.ones((1, 2, 1))
    u = O.column_scores(Qw, K, ows=2, scale=1.0)
    assert np.allclose(u, g["u_num"] / g["u_den"], atol=1e-14)
    wmax = O.pooling(u, 3, "max")
    wavg = O.pooling(u, 3, "avg")
    assert np.allclose(wmax, g["max_num"] / g["max_den"], atol=1e-14)
    assert np.allclose(wavg, g["avg_num"] / g["avg_den"], atol=1e-14)
    for n in range(1, 5):
        assert abs(O.retention_ratio(wmax, n) - g["R_num"][n - 1] / g["R_den"][0]) < 1e-14
    assert O.topk_indices(wmax, 2).tolist() == g["top2_max"].astype(int).tolist()
    assert O.topk_indices(wavg, 2).tolist() == g["top2_avg"].astype(int).tolist()
    assert O.topk_indices(wavg, 1).tolist() == g["top1_avg"].astype(int).tolist()
    assert np.allclose(O.score_vector(Qw, K, 2, 3, "max", 1.0), wmax)


def test_gqa_group_sums_heads_before_pooling():
    rng = np.random.default_rng(4)
    t, d, ows, G = 40, 8, 4, 4
    Qg, K = rng.normal(size=(G, ows, d)), rng.normal(size=(t, d))
    per_head = [O.column_scores(Qg[h:h + 1], K, ows) for h in range(G)]
    assert np.allclose(O.column_scores(Qg, K, ows), np.sum(per_head, axis=0), atol=1e-14)
    # pooling after the sum differs from the sum of pooled vectors (max is not linear)
    a = O.pooling(np.sum(per_head, axis=0), 5, "max")
    b = np.sum([O.pooling(u, 5, "max") for u in per_head], axis=0)
    assert np.all(a <= b + 1e-15) and not np.allclose(a, b)


def test_short_sequence_uses_last_rows_only():
    rng = np.random.default_rng(5)
    d, ows, t = 8, 6, 4
    Qw, K = rng.normal(size=(ows, d)), rng.normal(size=(t, d))
    win = O.window_attention_weights(Qw, K)
    assert np.all(win[: ows - t] == 0.0)
    assert np.allclose(win[ows - t:].sum(axis=1), 1.0)
    assert O.column_scores(Qw[None], K, ows).shape == (0,)


# ------------------------------------------------------------------ pooling
def test_pooling_identity_constant_onehot():
    rng = np.random.default_rng(6)
    u = rng.random(19)
    assert np.array_equal(O.pooling(u, 1, "max"), u)
    assert np.allclose(O.pooling(u, 1, "avg"), u)
    c = np.full(11, 0.7)
    assert np.array_equal(O.pooling(c, 5, "max"), c)
    avg = O.pooling(c, 5, "avg")
    assert np.allclose(avg[2:-2], 0.7)
    assert np.allclose(avg[[0, -1]], 0.7 * 3 / 5) and np.allclose(avg[[1, -2]], 0.7 * 4 / 5)
    e = np.zeros(15); e[7] = 2.0
    m = O.pooling(e, 5, "max")
    assert np.array_equal(np.nonzero(m)[0], np.arange(5, 10)) and np.all(m[5:10] == 2.0)


def test_pooling_hand_computed_six_elements():
    u = np.array([1.0, 5.0, 2.0, 0.0, 3.0, 4.0])
    assert O.pooling(u, 3, "max").tolist() == [5.0, 5.0, 5.0, 3.0, 4.0, 4.0]
    assert np.allclose(O.pooling(u, 3, "avg"), np.array([6.0, 8.0, 7.0, 5.0, 7.0, 7.0]) / 3.0)
    assert O.pooling(u, 5, "max").tolist() == [5.0, 5.0, 5.0, 5.0, 4.0, 4.0]
    assert np.allclose(O.pooling(u, 5, "avg"), np.array([8.0, 8.0, 11.0, 14.0, 9.0, 7.0]) / 5.0)


@pytest.mark.parametrize("ps", [3, 5, 7])
def test_pooling_matches_torch(ps):
    rng = np.random.default_rng(7)
    u = rng.random(53)
    x = torch.from_numpy(u)[None, None]
    mx = torch.nn.functional.max_pool1d(x, ps, stride=1, padding=ps // 2)[0, 0].numpy()
    av = torch.nn.functional.avg_pool1d(x, ps, stride=1, padding=ps // 2,
                                        count_include_pad=True)[0, 0].numpy()
    assert np.array_equal(O.pooling(u, ps, "max"), mx)
    assert np.allclose(O.pooling(u, ps, "avg"), av, atol=1e-15)


# ------------------------------------------------------------------ Eq. 4 and curves
def test_retention_ratio_and_curves():
    rng = np.random.default_rng(8)
    w = rng.random(31) ** 4
    assert abs(O.retention_ratio(w, len(w)) - 1.0) < 1e-14          # 100 % with no eviction
    g = O.head_gains(w)
    mass = O.retained_mass(g)
    assert abs(mass[-1] - 1.0) < 1e-13
    assert np.all(np.diff(mass) >= 0) and np.all(np.diff(g) <= 0)
    for n in (1, 5, 17, 31):
        assert abs(mass[n - 1] - O.retention_ratio(w, n)) < 1e-13
    # library cross-check
    s, _ = torch.sort(torch.from_numpy(w), descending=True)
    assert np.allclose(mass, (torch.cumsum(s, 0) / s.sum()).numpy(), atol=1e-14)
    # one head: the layer curve is the head's own curve
    assert np.allclose(O.layer_gains([w], 31), g)


def test_layer_gains_is_rankwise_mean_with_zero_fill():
    w1 = np.array([4.0, 1.0, 3.0, 2.0])          # gains 0.4 0.3 0.2 0.1
    w2 = np.array([1.0, 3.0])                    # gains 0.75 0.25
    g = O.layer_gains([w1, w2], 5)
    assert np.allclose(g, [(0.4 + 0.75) / 2, (0.3 + 0.25) / 2, 0.1, 0.05, 0.0])
    # equals the mean over heads of each head's own Eq. 4 at every n
    for n in range(1, 5):
        r = (O.retention_ratio(w1, n) + O.retention_ratio(w2, min(n, 2))) / 2
        assert abs(O.retained_mass(g)[n - 1] - r) < 1e-14
    assert np.all(O.head_gains(np.zeros(3)) == 0) and O.head_gains(np.zeros(0)).size == 0


def test_score_layer_packed_batch_matches_per_unit():
    rng = np.random.default_rng(9)
    B, Hq, Hkv, d, ows = 2, 4, 2, 8, 3
    lens = [9, 14]
    cu = np.array([0, 9, 23])
    q = rng.normal(size=(B, Hq, ows, d)); k = rng.normal(size=(23, Hkv, d))
    out = O.score_layer(q, k, cu, ows, 3, "max")
    assert set(out) == {(b, g) for b in range(B) for g in range(Hkv)}
    w = O.score_vector(q[1, 2:4], k[9:23, 1], ows, 3, "max")
    assert np.array_equal(out[(1, 1)], w) and w.shape == (lens[1] - ows,)
    curves = O.layer_curves(out, B, Hkv, 12)
    assert curves.shape == (2, 12)
    assert abs(curves[0].sum() - 1.0) < 1e-13 and abs(curves[1].sum() - 1.0) < 1e-13
    assert np.all(curves[0, 6:] == 0.0)


# ------------------------------------------------------------------ prefill attention (Eq. 1 / Eq. 2 over the prompt)
def test_prefill_attention_closed_forms_and_library():
    rng = np.random.default_rng(40)
    t, d = 37, 16
    Q, K, V = rng.standard_normal((t, d)), rng.standard_normal((t, d)), rng.standard_normal((t, d))
    Z, lse = O.prefill_attention(Q, K, V)
    # library cross-check: torch fp64 causal scaled-dot-product attention on the CPU
    ref = torch.nn.functional.scaled_dot_product_attention(torch.from_numpy(Q)[None], torch.from_numpy(K)[None],
                                                           torch.from_numpy(V)[None], is_causal=True)[0].numpy()
    assert np.max(np.abs(Z - ref)) < 1e-12
    # identical keys: uniform weights over the visible keys, so row i is the running mean of V and lse = s + ln(i+1)
    Kc = np.tile(K[:1], (t, 1))
    Zc, lc = O.prefill_attention(Q, Kc, V)
    running = np.cumsum(V, axis=0) / np.arange(1, t + 1)[:, None]
    assert np.max(np.abs(Zc - running)) < 1e-12
    s_const = (Q @ K[0]) / math.sqrt(d)
    assert np.max(np.abs(lc - (s_const + np.log(np.arange(1, t + 1))))) < 1e-12
    # row 0 sees only itself: z_0 = v_0, lse_0 = its one logit
    assert np.max(np.abs(Z[0] - V[0])) < 1e-15 and abs(lse[0] - (Q[0] @ K[0]) / math.sqrt(d)) < 1e-13
    # the last rows of each decode step: attending with q_i over keys 0..i is decode_attention on that prefix
    for i in (0, 5, t - 1):
        z, l = O.decode_attention(Q[i], K[: i + 1], V[: i + 1])
        assert np.max(np.abs(z - Z[i])) < 1e-13 and abs(l - lse[i]) < 1e-12


def test_window_scores_from_the_prefill_normalisers_equal_the_definition():
    rng = np.random.default_rng(41)
    t, d, ows, G = 53, 8, 6, 2
    K = rng.standard_normal((t, d))
    Qfull = rng.standard_normal((G, t, d)) * 2.0
    lse = np.stack([O.prefill_attention(Qfull[h], K, K)[1] for h in range(G)])            # [G, t]
    Qwin = Qfull[:, t - ows:]
    u_def = O.column_scores(Qwin, K, ows)
    u_lse = O.column_scores_from_lse(Qwin, K, lse[:, t - ows:], ows)
    assert np.max(np.abs(u_def - u_lse)) < 1e-13
    # exp(logit - lse) of a window row is that row of W_attn (Eq. 2): compare with the full matrix
    Wfull = O.attention_weights(Qfull[1], K)
    r = 3
    row = np.exp((K[: t - ows] @ Qwin[1, r]) / math.sqrt(d) - lse[1, t - ows + r])
    assert np.max(np.abs(row - Wfull[t - ows + r, : t - ows])) < 1e-14
    # a wrong normaliser (shifted by ln 2) halves the scores: the function really uses what it is given
    u_half = O.column_scores_from_lse(Qwin, K, lse[:, t - ows:] + math.log(2.0), ows)
    assert np.max(np.abs(u_half - 0.5 * u_def)) < 1e-13
