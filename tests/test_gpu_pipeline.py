"""End-to-end GPU parity of the whole path (score -> budgets -> select/compact -> decode steps) on the
tiny configuration and on scaled-down versions of the larger workload shapes, against the oracle."""
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

SCALED = {
    "tiny": WL.CONFIGS["tiny"],
    "mha": replace(WL.CONFIGS["llama2_7b_mha"], n_layers=3, n_q_heads=4, n_kv_heads=4, batch=2, prompt=1024,
                   avg_budget=128, decode_steps=3),
    "gqa_long_window": replace(WL.CONFIGS["mistral_7b_gqa"], n_layers=3, n_q_heads=8, n_kv_heads=2, batch=2,
                               prompt=3000, avg_budget=300, n_min=32, n_max=1024, decode_steps=3),
    "ragged": replace(WL.CONFIGS["llama3_8b_ragged"], n_layers=2, n_q_heads=8, n_kv_heads=2, batch=6,
                      prompt=(300, 1200), avg_budget=200, decode_steps=3),
    "long": replace(WL.CONFIGS["llama3_8b_long"], n_layers=2, n_q_heads=8, n_kv_heads=2, prompt=10000,
                    avg_budget=512, n_min=64, n_max=2048, decode_steps=2),
}


def _cache_rows(sess, layer, b, g, n):
    bt = sess.block_table[layer, b].cpu().numpy()
    slots = np.arange(n)
    pages = torch.from_numpy(bt[slots // sess.page_size].astype(np.int64)).to(sess.device)
    off = torch.from_numpy(slots % sess.page_size).to(sess.device)
    return sess.k_pages[pages, g, off], sess.v_pages[pages, g, off]


def run_path(w: WL.Workload, stress: bool, full_budget: bool = False):
    require_lib()
    lengths = WL.prompt_lengths(w)
    L, B, Hkv, G, W = w.n_layers, w.batch, w.n_kv_heads, w.group, w.window
    steps = w.decode_steps
    tens = [WL.layer_tensors(w, l, DEV, lengths, stress=stress) for l in range(L)]
    max_prefix = max(t - W for t in lengths)
    n_max = w.n_max if (w.n_max and not full_budget) else 0
    N = None
    if w.budgets is None and not full_budget:
        N = L * w.avg_budget
    sess = XkvSession(L, w.n_q_heads, Hkv, w.head_dim, W, w.pool_kernel, lengths, pool_mode=w.pool_mode,
                      max_new_tokens=steps, max_budget=n_max or None, total_budget=N,
                      curve_len=n_max or None, device=DEV)
    for l in range(L):
        sess.score_layer(l, tens[l][0], tens[l][1])
    torch.cuda.synchronize()

    # oracle scores and curves
    w_ref = [O.score_layer(f64(tens[l][0]), f64(tens[l][1]), sess.cu_host, W, w.pool_kernel,
                           "max" if w.pool_mode == 0 else "avg") for l in range(L)]
    if full_budget:
        budgets = np.full(L, max_prefix, dtype=np.int32)
    elif w.budgets is not None:
        budgets = np.asarray(w.budgets, dtype=np.int32)
    else:
        budgets, r_gpu = sess.solve_budgets(total=N, n_min=w.n_min, n_max=n_max)
        curves = [O.layer_curves(w_ref[l], B, Hkv, sess.curve_len).mean(axis=0) for l in range(L)]
        A, r_ref = O.adaptive_allocation(curves, N=N, n_min=w.n_min, n_max=n_max or None,
                                         capacity=[max_prefix] * L)
        assert budgets.sum() == N
        assert abs(r_gpu - r_ref) <= 1e-6, (r_gpu, r_ref)
        assert abs(O.allocation_objective(curves, budgets.tolist()) - r_ref) <= 1e-6
        print(f"{w.name}: budgets {budgets.tolist()} oracle {A} sum|dk|={int(np.abs(budgets - np.array(A)).sum())}")
    sess.assign_pages(budgets)

    # selection + compaction
    sel = torch.full((B, Hkv, sess.max_seqlen), -1, dtype=torch.int32, device=DEV)
    Kc, Vc = {}, {}
    near = 0
    for l in range(L):
        sel.fill_(-1)
        sess.select_layer(l, int(budgets[l]), tens[l][1], tens[l][2], sel=sel)
        torch.cuda.synchronize()
        assert sess.device_status("select") == xkv.OK
        lens = sess.seq_lens[l].cpu().numpy()
        for b, t in enumerate(lengths):
            lo = int(sess.cu_host[b])
            for g in range(Hkv):
                wv = w_ref[l][(b, g)]
                keep = O.kept_positions(wv, int(budgets[l]), t, W)
                assert lens[b] == len(keep)
                got = sel[b, g, : len(keep)].cpu().numpy()
                if O.near_tie(wv, int(budgets[l])):
                    near += 1
                    thr = O.sort_descending(wv)[min(int(budgets[l]), len(wv)) - 1]
                    diff = np.setxor1d(got, keep)
                    assert np.all(np.abs(wv[diff] - thr) <= 1e-5 * thr)
                else:
                    assert np.array_equal(got, keep), (l, b, g)
                kc, vc = _cache_rows(sess, l, b, g, len(keep))
                krows, vrows = tens[l][1][lo: lo + t, g], tens[l][2][lo: lo + t, g]
                assert np.array_equal(bits(kc), O.evict_by_index(bits(krows), got))
                assert np.array_equal(bits(vc), O.evict_by_index(bits(vrows), got))
                Kc[(l, b, g)] = O.evict_by_index(f64(krows), got)
                Vc[(l, b, g)] = O.evict_by_index(f64(vrows), got)
    print(f"{w.name}: near-tie heads {near} of {L * B * Hkv}")

    # generation steps
    for step in range(steps):
        q, kn, vn = WL.decode_tensors(w, step, DEV, stress=stress)
        out = sess.decode(q, kn, vn)
        torch.cuda.synchronize()
        assert sess.device_status("decode") == xkv.OK
        qf, knf, vnf = f64(q), f64(kn), f64(vn)
        ref = np.zeros((L, B, w.n_q_heads, w.head_dim))
        for l in range(L):
            for b in range(B):
                for g in range(Hkv):
                    Kc[(l, b, g)] = np.concatenate([Kc[(l, b, g)], knf[l, b, g][None]], 0)
                    Vc[(l, b, g)] = np.concatenate([Vc[(l, b, g)], vnf[l, b, g][None]], 0)
                    for h in range(g * G, (g + 1) * G):
                        ref[l, b, h], _ = O.decode_attention(qf[l, b, h], Kc[(l, b, g)], Vc[(l, b, g)])
        check_attention(out, ref, f"{w.name} step {step}", rel_l2=stress)
    return sess, tens, ref


@pytest.mark.parametrize("name", list(SCALED))
@pytest.mark.parametrize("stress", [False, True])
def test_whole_path_matches_oracle(name, stress):
    run_path(SCALED[name], stress)


def test_full_budget_reproduces_full_attention():
    """With k_l >= P_b nothing is evicted: the compacted cache is the prompt and decode equals full
    attention over prompt + new tokens."""
    w = replace(SCALED["long"], prompt=5000, decode_steps=1)
    sess, tens, ref = run_path(w, stress=True, full_budget=True)
    lengths = WL.prompt_lengths(w)
    q, kn, vn = WL.decode_tensors(w, 0, DEV, stress=True)
    for l in range(w.n_layers):
        K = np.concatenate([f64(tens[l][1]), f64(kn[l])], 0)     # B = 1: whole prompt + new token
        V = np.concatenate([f64(tens[l][2]), f64(vn[l])], 0)
        for h in range(w.n_q_heads):
            z, _ = O.decode_attention(f64(q[l, 0, h]), K[:, h // w.group], V[:, h // w.group])
            assert np.allclose(z, ref[l, 0, h], atol=1e-12)
    assert sess.seq_lens.cpu().numpy().tolist() == [[lengths[0] + 1]] * w.n_layers


def test_online_scenario_averaged_list_applied_to_a_new_task():
    """Sec. IV-C: allocation lists recorded on a few sampled tasks are averaged, and a later task of the same type
    is evicted under the averaged list without running the allocation.  Uses the paper's own defaults (observation
    window 8, average pooling of size 7)."""
    require_lib()
    base = replace(WL.CONFIGS["mistral_7b_gqa"], n_layers=4, n_q_heads=8, n_kv_heads=2, batch=1, prompt=1500,
                   window=8, pool_kernel=7, pool_mode=1, avg_budget=160, n_min=16, n_max=600, decode_steps=2)
    N = base.n_layers * base.avg_budget
    recorded = []
    for task in range(3):
        w = replace(base, seed=base.seed + 31 * (task + 1))
        lengths = WL.prompt_lengths(w)
        sess = XkvSession(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.window, w.pool_kernel, lengths,
                          pool_mode=w.pool_mode, max_budget=w.n_max, total_budget=N, curve_len=w.n_max, device=DEV)
        tens = [WL.layer_tensors(w, l, DEV, lengths) for l in range(w.n_layers)]
        sess.score_layers([t[0] for t in tens], [t[1] for t in tens])
        budgets, _ = sess.solve_budgets(total=N, n_min=w.n_min, n_max=w.n_max)
        assert sess.device_status("score") == xkv.OK and budgets.sum() == N
        recorded.append(budgets.tolist())
    averaged = xkv.average_budgets(recorded)
    assert averaged.tolist() == O.averaged_allocation(recorded) and averaged.sum() == N
    assert len({tuple(r) for r in recorded}) > 1, "the sampled tasks should not all give the same list"
    # a new task of the same type: no allocation, eviction under the averaged list, then generation
    run_path(replace(base, seed=base.seed + 1000, budgets=tuple(int(x) for x in averaged)), stress=True)


def test_deterministic_across_runs():
    w = SCALED["ragged"]
    a, _, _ = run_path(w, False)
    sa, ka, oa = a.scores.clone(), a.k_pages.clone(), a.out.clone()
    b, _, _ = run_path(w, False)
    assert torch.equal(sa, b.scores) and torch.equal(oa.view(torch.int16), b.out.view(torch.int16))
    assert torch.equal(ka.view(torch.int16), b.k_pages.view(torch.int16))
