"""Reduced caches stored with few bits (Sec. II-B: quantisation is compatible with eviction): rows compacted into
8-bit codes with one scale per row, and decode attention over them, against the oracle.  The codes and scales are
integer / bit-exact work; the attention is compared with fp64 attention over the rows the codes stand for."""
from dataclasses import replace

import numpy as np
import pytest
import torch

from oracle import xkv_oracle as O
from paper_2412_05896_b200 import workloads as WL
from paper_2412_05896_b200 import xkv
from paper_2412_05896_b200.pipeline import XkvSession

from gpu_util import check_attention, f64, require_lib

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

CASES = {
    "gqa_d128": replace(WL.CONFIGS["mistral_7b_gqa"], n_layers=3, n_q_heads=8, n_kv_heads=2, batch=2,
                        prompt=(500, 1400), window=16, avg_budget=200, n_min=16, n_max=1024, decode_steps=3),
    "mha_d64": replace(WL.CONFIGS["tiny"], n_layers=2, batch=3, prompt=(150, 700), budgets=None, avg_budget=90,
                       decode_steps=3),
    "long_split": replace(WL.CONFIGS["llama3_8b_long"], n_layers=2, n_q_heads=8, n_kv_heads=2, prompt=9000,
                          avg_budget=3000, n_min=64, n_max=4096, decode_steps=2),
    # with head-level caches: 6 x 12 x 32 = 2304 (layer, cache) units, beyond what the attention kernel plans for
    # itself, so the separate append-and-plan kernel stores the new rows
    "many_units": replace(WL.CONFIGS["tiny"], n_layers=6, n_q_heads=32, n_kv_heads=32, batch=12, prompt=(40, 90),
                          window=8, budgets=None, avg_budget=16, decode_steps=2),
}


def _cache_rows(sess, layer, cache_idx, head_in_page, n):
    bt = sess.block_table[layer, cache_idx].cpu().numpy()
    slots = np.arange(n)
    pages = torch.from_numpy(bt[slots // sess.page_size].astype(np.int64)).to(sess.device)
    off = torch.from_numpy(slots % sess.page_size).to(sess.device)
    return (sess.k_pages[pages, head_in_page, off].cpu().numpy(), sess.k_scales[pages, head_in_page, off].cpu().numpy(),
            sess.v_pages[pages, head_in_page, off].cpu().numpy(), sess.v_scales[pages, head_in_page, off].cpu().numpy())


@pytest.mark.parametrize("name,head_level", [("gqa_d128", False), ("gqa_d128", True), ("mha_d64", False),
                                             ("long_split", False), ("many_units", True)])
def test_quantized_cache_rows_and_decode(name, head_level):
    require_lib()
    w = CASES[name]
    lengths = WL.prompt_lengths(w)
    L, B, Hkv, Hq, G, W, d = w.n_layers, w.batch, w.n_kv_heads, w.n_q_heads, w.group, w.window, w.head_dim
    steps = w.decode_steps
    tens = [WL.layer_tensors(w, l, DEV, lengths, stress=True) for l in range(L)]
    n_max = w.n_max or 0
    N = L * w.avg_budget * (Hkv if head_level else 1)
    sess = XkvSession(L, Hq, Hkv, d, W, w.pool_kernel, lengths, pool_mode=w.pool_mode, max_new_tokens=steps,
                      max_budget=n_max or None, total_budget=N, curve_len=n_max or None, device=DEV,
                      head_level=head_level, kv_format=xkv.KV_INT8)
    sess.score_layers([t[0] for t in tens], [t[1] for t in tens])
    budgets, _ = sess.solve_budgets(total=N, n_min=w.n_min, n_max=n_max)
    sess.assign_pages(budgets)
    sel = torch.full((B, Hkv, sess.max_seqlen), -1, dtype=torch.int32, device=DEV)
    Kq, Vq = {}, {}
    for l in range(L):
        sel.fill_(-1)
        sess.select_layer(l, budgets[l] if head_level else int(budgets[l]), tens[l][1], tens[l][2], sel=sel)
        torch.cuda.synchronize()
        assert sess.device_status("select") == xkv.OK
        lens = sess.seq_lens[l].cpu().numpy()
        for b, t in enumerate(lengths):
            lo = int(sess.cu_host[b])
            for g in range(Hkv):
                cache_idx, hp = (b * Hkv + g, 0) if head_level else (b, g)
                n = int(lens[cache_idx])
                kept = sel[b, g, :n].cpu().numpy()            # the selection itself is checked elsewhere
                assert n > 0 and np.all(kept >= 0)
                kc, ks, vc, vs = _cache_rows(sess, l, cache_idx, hp, n)
                for rows, codes, scales, store in ((tens[l][1], kc, ks, Kq), (tens[l][2], vc, vs, Vq)):
                    x = O.evict_by_index(f64(rows[lo: lo + t, g]), kept)
                    ref_codes, ref_scales = O.quantize_rows_int8(x)
                    assert np.array_equal(scales, ref_scales), (name, l, b, g)
                    assert np.array_equal(codes, ref_codes), (name, l, b, g, int((codes != ref_codes).sum()))
                    store[(l, b, g)] = O.dequantize_rows_int8(ref_codes, ref_scales)

    for step in range(steps):
        q, kn, vn = WL.decode_tensors(w, step, DEV, stress=True)
        out = sess.decode(q, kn, vn)
        torch.cuda.synchronize()
        assert sess.device_status("decode") == xkv.OK
        ref = np.zeros((L, B, Hq, d))
        lens = sess.seq_lens.cpu().numpy()
        for l in range(L):
            for b in range(B):
                for g in range(Hkv):
                    # the appended row is stored the same way: codes and scale of the new K/V row
                    kcode, kscale = O.quantize_rows_int8(f64(kn[l, b, g])[None])
                    vcode, vscale = O.quantize_rows_int8(f64(vn[l, b, g])[None])
                    Kq[(l, b, g)] = np.concatenate([Kq[(l, b, g)], O.dequantize_rows_int8(kcode, kscale)], 0)
                    Vq[(l, b, g)] = np.concatenate([Vq[(l, b, g)], O.dequantize_rows_int8(vcode, vscale)], 0)
                    cache_idx, hp = (b * Hkv + g, 0) if head_level else (b, g)
                    n = int(lens[l, cache_idx])
                    assert n == Kq[(l, b, g)].shape[0]
                    kc, ks, vc, vs = _cache_rows(sess, l, cache_idx, hp, n)
                    assert np.array_equal(kc[-1], kcode[0]) and ks[-1] == kscale[0], (name, step, l, b, g)
                    assert np.array_equal(vc[-1], vcode[0]) and vs[-1] == vscale[0], (name, step, l, b, g)
                    for h in range(g * G, (g + 1) * G):
                        ref[l, b, h], _ = O.decode_attention(f64(q[l, b, h]), Kq[(l, b, g)], Vq[(l, b, g)])
        check_attention(out, ref, f"{name} step {step}", rel_l2=True)


def test_quantized_cache_rejections():
    require_lib()
    w = replace(WL.CONFIGS["tiny"], n_layers=1, batch=1, prompt=200)
    lengths = WL.prompt_lengths(w)
    sess = XkvSession(1, w.n_q_heads, w.n_kv_heads, w.head_dim, w.window, w.pool_kernel, lengths, max_new_tokens=1,
                      device=DEV, kv_format=xkv.KV_INT8)
    q, kn, vn = WL.decode_tensors(w, 0, DEV)
    no_scales = xkv.Cache(sess.k_pages.data_ptr(), sess.v_pages.data_ptr(), sess.block_table.data_ptr(),
                          sess.seq_lens.data_ptr(), 1, sess.page_size, sess.max_pages_per_seq, sess.n_pages, None, None,
                          xkv.KV_INT8, 0)
    with pytest.raises(xkv.XkvError) as e:
        xkv.decode_attn(sess.dims, no_scales, 0, 1, q, kn, vn, sess.out, None, 0, sess.ws_decode)
    assert e.value.status == xkv.ERR_INVALID_ARG
    bad_format = xkv.Cache(sess.k_pages.data_ptr(), sess.v_pages.data_ptr(), sess.block_table.data_ptr(),
                           sess.seq_lens.data_ptr(), 1, sess.page_size, sess.max_pages_per_seq, sess.n_pages,
                           sess.k_scales.data_ptr(), sess.v_scales.data_ptr(), 7, 0)
    with pytest.raises(xkv.XkvError) as e:
        xkv.decode_attn(sess.dims, bad_format, 0, 1, q, kn, vn, sess.out, None, 0, sess.ws_decode)
    assert e.value.status == xkv.ERR_INVALID_ARG
    with pytest.raises(xkv.XkvError) as e:          # the allocation-free variant reads 16-bit caches only
        xkv.decode_attn_static(sess.dims, sess.cache, 0, 1, q, kn, vn, sess.out, None, 64)
    assert e.value.status == xkv.ERR_UNSUPPORTED
