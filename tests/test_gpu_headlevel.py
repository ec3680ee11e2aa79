"""Head-level budgets inside the layers (Sec. II-C: cache sizes pre-set per attention head work together with the
layer-level allocation): per-head curves, the solver over (layer, KV head) units, selection and compaction into
caches of one KV head each, and decode over them, against the oracle."""
from dataclasses import replace

import numpy as np
import pytest
import torch

from oracle import xkv_oracle as O
from paper_2412_05896_b200 import workloads as WL
from paper_2412_05896_b200 import xkv
from paper_2412_05896_b200.pipeline import XkvSession

from gpu_util import bits, check_attention, f64, require_lib

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

CASES = {
    "gqa": replace(WL.CONFIGS["mistral_7b_gqa"], n_layers=3, n_q_heads=8, n_kv_heads=4, batch=2, prompt=(700, 1500),
                   window=16, avg_budget=160, n_min=8, n_max=1024, decode_steps=3),
    "mha_d64": replace(WL.CONFIGS["tiny"], n_layers=2, n_q_heads=4, n_kv_heads=4, batch=3, prompt=(200, 900),
                       budgets=None, avg_budget=96, decode_steps=2),
    "long_chunked_select": replace(WL.CONFIGS["llama3_8b_long"], n_layers=2, n_q_heads=8, n_kv_heads=2, prompt=9000,
                                   avg_budget=700, n_min=64, n_max=4096, decode_steps=2),
}


def _head_cache_rows(sess, layer, cache_idx, n):
    bt = sess.block_table[layer, cache_idx].cpu().numpy()
    slots = np.arange(n)
    pages = torch.from_numpy(bt[slots // sess.page_size].astype(np.int64)).to(sess.device)
    off = torch.from_numpy(slots % sess.page_size).to(sess.device)
    return sess.k_pages[pages, 0, off], sess.v_pages[pages, 0, off]


@pytest.mark.parametrize("name", list(CASES))
def test_head_level_path_against_oracle(name):
    require_lib()
    w = CASES[name]
    lengths = WL.prompt_lengths(w)
    L, B, Hkv, Hq, G, W, d = w.n_layers, w.batch, w.n_kv_heads, w.n_q_heads, w.group, w.window, w.head_dim
    steps = w.decode_steps
    tens = [WL.layer_tensors(w, l, DEV, lengths, stress=True) for l in range(L)]
    max_prefix = max(t - W for t in lengths)
    n_max = w.n_max or 0
    N = L * Hkv * w.avg_budget                      # prefix tokens over all heads of all layers, per sequence
    sess = XkvSession(L, Hq, Hkv, d, W, w.pool_kernel, lengths, pool_mode=w.pool_mode, max_new_tokens=steps,
                      max_budget=n_max or None, total_budget=N, curve_len=n_max or None, device=DEV,
                      head_level=True)
    sess.score_layers([t[0] for t in tens], [t[1] for t in tens])
    torch.cuda.synchronize()
    assert sess.device_status("score") == xkv.OK

    mode = "max" if w.pool_mode == 0 else "avg"
    w_ref = [O.score_layer(f64(tens[l][0]), f64(tens[l][1]), sess.cu_host, W, w.pool_kernel, mode) for l in range(L)]
    # per-head curves, element by element
    hg = sess.head_gains.cpu().numpy().astype(np.float64)            # [L, Hkv, B, curve_len]
    for l in range(L):
        for b in range(B):
            for g in range(Hkv):
                ref = O.head_gains(w_ref[l][(b, g)])[: sess.curve_len]
                got = hg[l, g, b]
                assert np.allclose(got[: ref.size], ref, rtol=1e-4, atol=1e-9), (l, b, g)
                assert np.all(got[ref.size:] == 0.0)

    # the solver over (layer, KV head) units on the batch-mean curves, compared by objective
    budgets, r_gpu = sess.solve_budgets(total=N, n_min=w.n_min, n_max=n_max)
    assert budgets.shape == (L, Hkv) and int(budgets.sum()) == N
    unit_curves = []
    for l in range(L):
        for g in range(Hkv):
            c = np.zeros(sess.curve_len)
            for b in range(B):
                x = O.head_gains(w_ref[l][(b, g)])[: sess.curve_len]
                c[: x.size] += x
            unit_curves.append(c / B)
    A, r_ref = O.adaptive_allocation(unit_curves, N=N, n_min=w.n_min, n_max=n_max or None,
                                     capacity=[max_prefix] * (L * Hkv))
    assert abs(r_gpu - r_ref) <= 1e-6, (r_gpu, r_ref)
    assert abs(O.allocation_objective(unit_curves, budgets.ravel().tolist()) - r_ref) <= 1e-6
    assert len(set(budgets.ravel().tolist())) > 1                    # heads really get different counts
    if B == 1:
        # one sequence: the oracle's head-level allocation from the score vectors themselves
        n_hl, r_hl = O.head_level_allocation([[w_ref[l][(0, g)] for g in range(Hkv)] for l in range(L)], N=N,
                                             n_min=w.n_min, n_max=n_max or None)
        assert abs(r_gpu - r_hl) <= 1e-6
    sess.assign_pages(budgets)

    # selection and compaction per head (downstream stages use the GPU's budgets on both sides)
    sel = torch.full((B, Hkv, sess.max_seqlen), -1, dtype=torch.int32, device=DEV)
    Kc, Vc = {}, {}
    near = 0
    for l in range(L):
        sel.fill_(-1)
        sess.select_layer(l, budgets[l], tens[l][1], tens[l][2], sel=sel)
        torch.cuda.synchronize()
        assert sess.device_status("select") == xkv.OK
        lens = sess.seq_lens[l].cpu().numpy()                        # [B * Hkv]
        for b, t in enumerate(lengths):
            lo = int(sess.cu_host[b])
            for g in range(Hkv):
                kb = int(budgets[l, g])
                wv = w_ref[l][(b, g)]
                keep = O.kept_positions(wv, kb, t, W)
                assert lens[b * Hkv + g] == len(keep), (l, b, g)
                got = sel[b, g, : len(keep)].cpu().numpy()
                if O.near_tie(wv, kb):
                    near += 1
                    thr = O.sort_descending(wv)[min(kb, len(wv)) - 1]
                    diff = np.setxor1d(got, keep)
                    assert np.all(np.abs(wv[diff] - thr) <= 1e-5 * thr)
                else:
                    assert np.array_equal(got, keep), (l, b, g)
                kc, vc = _head_cache_rows(sess, l, b * Hkv + g, len(keep))
                krows, vrows = tens[l][1][lo: lo + t, g], tens[l][2][lo: lo + t, g]
                assert np.array_equal(bits(kc), O.evict_by_index(bits(krows), got))
                assert np.array_equal(bits(vc), O.evict_by_index(bits(vrows), got))
                Kc[(l, b, g)] = O.evict_by_index(f64(krows), got)
                Vc[(l, b, g)] = O.evict_by_index(f64(vrows), got)
    print(f"{name}: budgets {budgets.tolist()}, near-tie heads {near} of {L * B * Hkv}")

    # generation over caches whose lengths differ per head
    for step in range(steps):
        q, kn, vn = WL.decode_tensors(w, step, DEV, stress=True)
        out = sess.decode(q, kn, vn)
        torch.cuda.synchronize()
        assert sess.device_status("decode") == xkv.OK
        ref = np.zeros((L, B, Hq, d))
        for l in range(L):
            for b in range(B):
                for g in range(Hkv):
                    Kc[(l, b, g)] = np.concatenate([Kc[(l, b, g)], f64(kn[l, b, g])[None]], 0)
                    Vc[(l, b, g)] = np.concatenate([Vc[(l, b, g)], f64(vn[l, b, g])[None]], 0)
                    for h in range(g * G, (g + 1) * G):
                        ref[l, b, h], _ = O.decode_attention(f64(q[l, b, h]), Kc[(l, b, g)], Vc[(l, b, g)])
        check_attention(out, ref, f"{name} step {step}", rel_l2=True)
        lens = sess.seq_lens.cpu().numpy().reshape(L, B, Hkv)
        for l in range(L):
            for b in range(B):
                for g in range(Hkv):
                    assert lens[l, b, g] == Kc[(l, b, g)].shape[0]


def test_head_level_budget_rejections_and_capacity():
    require_lib()
    w = replace(WL.CONFIGS["tiny"], n_layers=1, batch=2, prompt=300)
    lengths = WL.prompt_lengths(w)
    q_win, k, v = WL.layer_tensors(w, 0, DEV, lengths)
    sess = XkvSession(1, w.n_q_heads, w.n_kv_heads, w.head_dim, w.window, w.pool_kernel, lengths, max_new_tokens=1,
                      max_budget=64, device=DEV, head_level=True)
    sess.score_layer(0, q_win, k)
    bad = np.full((w.batch, w.n_kv_heads), 10, dtype=np.int32)
    bad[1, 2] = -1
    with pytest.raises(xkv.XkvError) as e:
        sess.select_layer(0, bad, k, v)
    assert e.value.status == xkv.ERR_BUDGET
    with pytest.raises(xkv.XkvError) as e:
        xkv.select_compact(sess.dims, 0, np.zeros(1, dtype=np.int32), 3, sess.scores[0], sess.sorted[0], k, v, sess.cu,
                           sess.T, sess.max_seqlen, sess.cache, None, 0, sess.ws_select[0])
    assert e.value.status == xkv.ERR_INVALID_ARG
    # one head beyond what its page list holds: that head's cache stays empty, the status says so, the others fit
    sess.assign_pages(np.full((1, w.n_kv_heads), 16, dtype=np.int32))
    over = np.full((w.batch, w.n_kv_heads), 16, dtype=np.int32)
    over[0, 1] = 250
    sess.select_layer(0, over, k, v)
    torch.cuda.synchronize()
    assert sess.device_status("select") == xkv.ERR_CAPACITY
    lens = sess.seq_lens[0].cpu().numpy().reshape(w.batch, w.n_kv_heads)
    assert lens[0, 1] == 0 and lens[0, 0] == 16 + w.window and lens[1, 3] == 16 + w.window
