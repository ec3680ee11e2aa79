"""Parity at the full workload sizes, in the launch configuration bench.py uses: every layer is scored,
the solver splits the global budget, every layer is compacted and decode steps run over all layers in one
call.  The oracle checks one whole (layer, sequence) with all its KV heads plus a few units elsewhere, one
by one; properties that hold at any size are checked on every layer."""
from dataclasses import replace

import numpy as np
import pytest
import torch

from oracle import xkv_oracle as O
from paper_2412_05896_b200 import workloads as WL
from paper_2412_05896_b200 import xkv
from paper_2412_05896_b200.pipeline import XkvSession

from gpu_util import bits, f64, require_lib, ATOL, RTOL

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

# name -> (workload, decode steps checked).  Layers are generated one at a time, so every workload runs with all
# of its layers.
FULL = {
    "llama2_7b_mha": (WL.CONFIGS["llama2_7b_mha"], 3),
    "mistral_7b_gqa": (WL.CONFIGS["mistral_7b_gqa"], 2),
    "llama3_8b_ragged": (WL.CONFIGS["llama3_8b_ragged"], 2),
    "llama3_8b_long": (WL.CONFIGS["llama3_8b_long"], 2),
}


def _sample_units(w, lengths, rng, n_extra):
    """Every KV head of one (layer, sequence), plus n_extra units drawn anywhere."""
    l0, b0 = int(rng.integers(w.n_layers)), int(rng.integers(w.batch))
    units = {(l0, b0, g) for g in range(w.n_kv_heads)}
    while len(units) < w.n_kv_heads + n_extra:
        units.add((int(rng.integers(w.n_layers)), int(rng.integers(w.batch)), int(rng.integers(w.n_kv_heads))))
    return sorted(units)


@pytest.mark.parametrize("name", list(FULL))
def test_full_size_sampled_parity(name):
    require_lib()
    w, steps = FULL[name]
    rng = np.random.default_rng(len(name))
    lengths = WL.prompt_lengths(w)
    L, B, Hkv, G, W, d = w.n_layers, w.batch, w.n_kv_heads, w.group, w.window, w.head_dim
    N = L * w.avg_budget
    sess = XkvSession(L, w.n_q_heads, Hkv, d, W, w.pool_kernel, lengths, max_new_tokens=steps,
                      max_budget=w.n_max or None, total_budget=N, curve_len=w.n_max or None, device=DEV)
    units = _sample_units(w, lengths, rng, 4)
    sample_layers = sorted({u[0] for u in units})
    kept_layers = {}
    for l in range(L):
        q_win, k, v = WL.layer_tensors(w, l, DEV, lengths)
        sess.score_layer(l, q_win, k)
        if l in sample_layers:
            kept_layers[l] = (q_win, k, v)
        else:
            del q_win, k, v
    budgets, r_avg = sess.solve_budgets(total=N, n_min=w.n_min, n_max=w.n_max)
    assert int(budgets.sum()) == N and budgets.min() >= w.n_min
    if w.n_max:
        assert budgets.max() <= w.n_max
    assert 0.0 < r_avg <= 1.0 + 1e-6
    sess.assign_pages(budgets)
    cu = sess.cu_host

    # size-independent properties of the scoring outputs, all layers
    for l in range(L):
        srt = sess.sorted[l]
        for b, t in enumerate(lengths):
            P = t - W
            seg = srt[:, cu[b]: cu[b] + P]
            assert bool((seg[:, 1:] <= seg[:, :-1]).all()), "sort is not descending"
            assert bool((sess.scores[l][:, cu[b] + P: cu[b] + t] == 0).all())
        s_sum = sess.scores[l].double().sum(dim=1)
        assert torch.allclose(s_sum, srt.double().sum(dim=1), rtol=1e-9)
        gsum = sess.gains[l].double().sum(dim=1)
        assert bool((gsum <= 1.0 + 1e-4).all()) and bool((sess.gains[l] >= 0).all())

    # selection + compaction, all layers; sampled units against the oracle
    sel = torch.empty(B, Hkv, sess.max_seqlen, dtype=torch.int32, device=DEV)
    Kc, Vc = {}, {}
    near = 0
    for l in range(L):
        if l in kept_layers:
            q_win, k, v = kept_layers[l]
        else:
            q_win, k, v = WL.layer_tensors(w, l, DEV, lengths)
        sess.select_layer(l, int(budgets[l]), k, v, sel=sel)
        torch.cuda.synchronize()
        assert sess.device_status("select") == xkv.OK
        expect_len = [min(int(budgets[l]), t - W) + W for t in lengths]
        assert sess.seq_lens[l].cpu().tolist() == expect_len
        # kept positions are strictly ascending for every unit of this layer
        for b in range(B):
            s = sel[b, :, : expect_len[b]]
            assert bool((s[:, 1:] > s[:, :-1]).all())
        for (ul, b, g) in units:
            if ul != l:
                continue
            t = lengths[b]
            lo = int(cu[b])
            qf = f64(q_win[b:b + 1, g * G:(g + 1) * G])
            kf = f64(k[lo: lo + t, g:g + 1])
            wv = O.score_layer(qf, kf, np.array([0, t]), W, w.pool_kernel, "max")[(0, 0)]
            got_w = sess.scores[l][g, lo: lo + t - W].cpu().numpy().astype(np.float64)
            err = np.abs(got_w - wv)
            assert np.all(err <= 3e-5 * wv + 1e-7 * wv.max()), f"scores of unit {(l, b, g)}"
            keep = O.kept_positions(wv, int(budgets[l]), t, W)
            got = sel[b, g, : len(keep)].cpu().numpy()
            if O.near_tie(wv, int(budgets[l])):
                near += 1
                thr = O.sort_descending(wv)[min(int(budgets[l]), len(wv)) - 1]
                diff = np.setxor1d(got, keep)
                assert np.all(np.abs(wv[diff] - thr) <= 1e-5 * thr)
            else:
                assert np.array_equal(got, keep), (l, b, g)
            bt = sess.block_table[l, b].cpu().numpy()
            slots = np.arange(len(got))
            pages = torch.from_numpy(bt[slots // sess.page_size].astype(np.int64)).to(DEV)
            off = torch.from_numpy(slots % sess.page_size).to(DEV)
            krows, vrows = k[lo: lo + t, g], v[lo: lo + t, g]
            assert np.array_equal(bits(sess.k_pages[pages, g, off]), O.evict_by_index(bits(krows), got))
            assert np.array_equal(bits(sess.v_pages[pages, g, off]), O.evict_by_index(bits(vrows), got))
            Kc[(l, b, g)] = O.evict_by_index(f64(krows), got)
            Vc[(l, b, g)] = O.evict_by_index(f64(vrows), got)
        del q_win, k, v
    kept_layers.clear()
    print(f"{name}: budgets min {budgets.min()} max {budgets.max()}, R_avg {r_avg:.4f}, near-tie units {near}/{len(units)}")

    # decode steps over all layers; sampled heads against the oracle
    for step in range(steps):
        q, kn, vn = WL.decode_tensors(w, step, DEV)
        out = sess.decode(q, kn, vn)
        torch.cuda.synchronize()
        assert sess.device_status("decode") == xkv.OK
        assert bool(torch.isfinite(out.float()).all())
        for (l, b, g) in units:
            Kc[(l, b, g)] = np.concatenate([Kc[(l, b, g)], f64(kn[l, b, g])[None]], 0)
            Vc[(l, b, g)] = np.concatenate([Vc[(l, b, g)], f64(vn[l, b, g])[None]], 0)
            for h in range(g * G, (g + 1) * G):
                z, lse = O.decode_attention(f64(q[l, b, h]), Kc[(l, b, g)], Vc[(l, b, g)])
                got = f64(out[l, b, h])
                assert np.all(np.abs(got - z) <= ATOL + RTOL * np.abs(z)), (step, l, b, h)
                assert abs(float(sess.lse[l, b, h]) - lse) <= 2e-3 + 1e-4 * abs(lse)
        expect = [[min(int(budgets[l]), t - W) + W + step + 1 for t in lengths] for l in range(L)]
        assert sess.seq_lens.cpu().tolist() == expect


def test_uncompressed_long_cache_decode():
    """The in-run comparison for the long-context workload: nothing evicted (k_l >= P), decode over the
    full 131072-token cache of a few layers; sampled heads against the oracle's full attention."""
    require_lib()
    w = replace(WL.CONFIGS["llama3_8b_long"], n_layers=4)
    lengths = WL.prompt_lengths(w)
    L, Hkv, G, W, d = w.n_layers, w.n_kv_heads, w.group, w.window, w.head_dim
    sess = XkvSession(L, w.n_q_heads, Hkv, d, W, w.pool_kernel, lengths, max_new_tokens=2, device=DEV)
    P = lengths[0] - W
    sess.assign_pages([P] * L)
    tens = []
    for l in range(L):
        q_win, k, v = WL.layer_tensors(w, l, DEV, lengths)
        sess.score_layer(l, q_win, k)
        sess.select_layer(l, P, k, v)
        tens.append((k, v))
    q, kn, vn = WL.decode_tensors(w, 0, DEV)
    out = sess.decode(q, kn, vn)
    torch.cuda.synchronize()
    assert sess.device_status("decode") == xkv.OK
    assert sess.seq_lens.cpu().tolist() == [[lengths[0] + 1]] * L
    for (l, h) in [(0, 0), (1, 13), (3, 31)]:
        g = h // G
        K = np.concatenate([f64(tens[l][0][:, g]), f64(kn[l, 0, g])[None]], 0)
        V = np.concatenate([f64(tens[l][1][:, g]), f64(vn[l, 0, g])[None]], 0)
        z, _ = O.decode_attention(f64(q[l, 0, h]), K, V)
        assert np.all(np.abs(f64(out[l, 0, h]) - z) <= ATOL + RTOL * np.abs(z))


@pytest.mark.parametrize("name", ["llama2_7b_mha", "mistral_7b_gqa", "llama3_8b_ragged"])
def test_full_size_prefill_attention_and_scores_from_its_normalisers(name):
    """One layer of a workload at its full size: the causal attention of every prompt (sampled rows against the
    oracle, one row at a time), then the scores from its normalisers (one whole unit against the oracle's two-pass
    definition, every unit against the two-pass kernel)."""
    require_lib()
    w = WL.CONFIGS[name]
    rng = np.random.default_rng(len(name) + 17)
    lengths = WL.prompt_lengths(w)
    B, Hq, Hkv, G, W, d = w.batch, w.n_q_heads, w.n_kv_heads, w.group, w.window, w.head_dim
    sess = XkvSession(1, Hq, Hkv, d, W, w.pool_kernel, lengths, device=DEV)
    layer = 5
    q_win, k, v = WL.layer_tensors(w, layer, DEV, lengths, stress=True)
    T = sess.T
    gen = torch.Generator(device=DEV).manual_seed(99)
    q = torch.empty(T, Hq, d, dtype=torch.bfloat16, device=DEV).normal_(generator=gen)
    for b, t in enumerate(lengths):
        lo = int(sess.cu_host[b])
        q[lo + t - W: lo + t] = q_win[b].transpose(0, 1)                  # the window queries are the last W rows
    out, lse = sess.prefill_attention(q, k, v)
    torch.cuda.synchronize()
    assert sess.device_status("prefill") == xkv.OK
    assert bool(torch.isfinite(out.float()).all()) and bool(torch.isfinite(lse).all())
    # sampled rows: first and last rows of a sequence, tile boundaries, random ones
    for _ in range(3):
        b = int(rng.integers(B))
        t, lo = lengths[b], int(sess.cu_host[b])
        rows = sorted({0, 1, 63, 64, 127, 128, t - W - 1, t - W, t - 1} | {int(x) for x in rng.integers(0, t, 6)})
        h = int(rng.integers(Hq))
        g = h // G
        kf, vf = f64(k[lo: lo + t, g]), f64(v[lo: lo + t, g])
        for i in rows:
            z, l_ref = O.decode_attention(f64(q[lo + i, h]), kf[: i + 1], vf[: i + 1])
            got = f64(out[lo + i, h])
            assert np.all(np.abs(got - z) <= ATOL + RTOL * np.abs(z)), (b, h, i, float(np.abs(got - z).max()))
            assert abs(float(lse[h, lo + i]) - l_ref) <= 2e-4 + 1e-5 * abs(l_ref), (b, h, i)
    # scores from the normalisers
    sess.score_layer(0, q_win, k, lse=lse)
    torch.cuda.synchronize()
    assert sess.device_status("score") == xkv.OK
    one_pass = sess.scores[0].clone()
    b0, g0 = int(rng.integers(B)), int(rng.integers(Hkv))
    t, lo = lengths[b0], int(sess.cu_host[b0])
    wv = O.score_layer(f64(q_win[b0:b0 + 1, g0 * G:(g0 + 1) * G]), f64(k[lo: lo + t, g0:g0 + 1]), np.array([0, t]), W,
                       w.pool_kernel, "max")[(0, 0)]
    got_w = one_pass[g0, lo: lo + t - W].cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got_w - wv) <= 3e-5 * wv + 1e-7 * wv.max()), (b0, g0)
    sess.score_layer(0, q_win, k)                                        # the two-pass kernel on the same inputs
    torch.cuda.synchronize()
    a, b2 = one_pass.double(), sess.scores[0].double()
    assert bool((torch.abs(a - b2) <= 6e-5 * torch.maximum(a, b2) + 2e-7 * a.max()).all())


def test_full_size_int8_cache_decode():
    """The long-batch workload's shape with 8-bit caches (four layers): stored rows of sampled heads bit-exact against
    the oracle's quantisation, decode outputs of those heads against fp64 attention over the rows they stand for."""
    require_lib()
    w = replace(WL.CONFIGS["llama3_8b_ragged"], n_layers=4)
    rng = np.random.default_rng(5)
    lengths = WL.prompt_lengths(w)
    L, B, Hkv, G, W, d = w.n_layers, w.batch, w.n_kv_heads, w.group, w.window, w.head_dim
    N = L * w.avg_budget
    sess = XkvSession(L, w.n_q_heads, Hkv, d, W, w.pool_kernel, lengths, max_new_tokens=2, total_budget=N, device=DEV,
                      kv_format=xkv.KV_INT8)
    tens = [WL.layer_tensors(w, l, DEV, lengths, stress=True) for l in range(L)]
    sess.score_layers([t[0] for t in tens], [t[1] for t in tens])
    budgets, _ = sess.solve_budgets(total=N)
    sess.assign_pages(budgets)
    units = sorted({(int(rng.integers(L)), int(rng.integers(B)), int(rng.integers(Hkv))) for _ in range(6)})
    sel = torch.empty(B, Hkv, sess.max_seqlen, dtype=torch.int32, device=DEV)
    Kq, Vq = {}, {}
    for l in range(L):
        sess.select_layer(l, int(budgets[l]), tens[l][1], tens[l][2], sel=sel)
        torch.cuda.synchronize()
        for (ul, b, g) in units:
            if ul != l:
                continue
            t, lo = lengths[b], int(sess.cu_host[b])
            n = int(sess.seq_lens[l, b])
            kept = sel[b, g, :n].cpu().numpy()
            bt = sess.block_table[l, b].cpu().numpy()
            slots = np.arange(n)
            pages = torch.from_numpy(bt[slots // sess.page_size].astype(np.int64)).to(DEV)
            off = torch.from_numpy(slots % sess.page_size).to(DEV)
            for rows, pg, sc, store in ((tens[l][1], sess.k_pages, sess.k_scales, Kq),
                                        (tens[l][2], sess.v_pages, sess.v_scales, Vq)):
                ref_b, ref_s = O.quantize_rows_int8(O.evict_by_index(f64(rows[lo: lo + t, g]), kept))
                assert np.array_equal(pg[pages, g, off].cpu().numpy(), ref_b), (l, b, g)
                assert np.array_equal(sc[pages, g, off].cpu().numpy(), ref_s), (l, b, g)
                store[(l, b, g)] = O.dequantize_rows_int8(ref_b, ref_s)
    assert sess.device_status("select") == xkv.OK
    for step in range(2):
        q, kn, vn = WL.decode_tensors(w, step, DEV, stress=True)
        out = sess.decode(q, kn, vn)
        torch.cuda.synchronize()
        assert sess.device_status("decode") == xkv.OK
        assert bool(torch.isfinite(out.float()).all())
        for (l, b, g) in units:
            for new, store in ((kn, Kq), (vn, Vq)):
                nb, ns = O.quantize_rows_int8(f64(new[l, b, g])[None])
                store[(l, b, g)] = np.concatenate([store[(l, b, g)], O.dequantize_rows_int8(nb, ns)], 0)
            for h in range(g * G, (g + 1) * G):
                z, _ = O.decode_attention(f64(q[l, b, h]), Kq[(l, b, g)], Vq[(l, b, g)])
                got = f64(out[l, b, h])
                assert np.all(np.abs(got - z) <= ATOL + RTOL * np.abs(z)), (step, l, b, h)
