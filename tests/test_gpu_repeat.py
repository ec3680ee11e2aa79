"""The same call many times over the same inputs: every kernel of the path hands work between roles, warps or CTAs
(mbarriers, tickets, a work counter), and a hand-over that depended on timing would sooner or later show as a
difference between two runs.  Outputs must be bit-identical every time."""
from dataclasses import replace

import pytest
import torch

from paper_2412_05896_b200 import workloads as WL
from paper_2412_05896_b200 import xkv
from paper_2412_05896_b200.pipeline import XkvSession

from gpu_util import require_lib

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
REPS = 40

# name -> workload: the three scoring kernel families (single-read cluster kernel, two-pass kernels at 128 and at
# 256 query rows), each with several key tiles per CTA and ragged lengths
CASES = {
    "fused_gw32": replace(WL.CONFIGS["llama2_7b_mha"], n_layers=1, n_q_heads=8, n_kv_heads=8, batch=6,
                          prompt=(1500, 4000), avg_budget=256, decode_steps=1),
    "two_pass_gw128": replace(WL.CONFIGS["llama3_8b_ragged"], n_layers=1, batch=10, prompt=(2048, 8192),
                              avg_budget=512, decode_steps=1),
    "two_pass_gw256": replace(WL.CONFIGS["mistral_7b_gqa"], n_layers=1, batch=2, prompt=(9000, 20000),
                              avg_budget=1024, decode_steps=1),
}


def _same(a: torch.Tensor, b: torch.Tensor) -> bool:
    return torch.equal(a.contiguous().view(torch.uint8), b.contiguous().view(torch.uint8))


@pytest.mark.parametrize("name", list(CASES))
def test_scoring_selection_and_decode_are_repeatable(name):
    require_lib()
    w = CASES[name]
    lengths = WL.prompt_lengths(w)
    W = w.window
    N = w.avg_budget
    sess = XkvSession(1, w.n_q_heads, w.n_kv_heads, w.head_dim, W, w.pool_kernel, lengths, max_new_tokens=1,
                      total_budget=N, device=DEV)
    q_win, k, v = WL.layer_tensors(w, 0, DEV, lengths, stress=True)
    # ---- scoring
    first = None
    for rep in range(REPS):
        sess.scores.fill_(float("nan"))
        sess.sorted.fill_(float("nan"))
        sess.score_layer(0, q_win, k)
        torch.cuda.synchronize()
        assert sess.device_status("score") == xkv.OK
        got = (sess.scores[0].clone(), sess.sorted[0].clone(), sess.gains[0].clone())
        if first is None:
            first = got
        else:
            assert all(_same(a, b) for a, b in zip(got, first)), ("score", rep)
    # ---- selection and compaction
    budgets, _ = sess.solve_budgets(total=N)
    sess.assign_pages(budgets)
    first = None
    for rep in range(REPS):
        sess.k_pages.fill_(float("nan"))
        sess.select_layer(0, int(budgets[0]), k, v)
        torch.cuda.synchronize()
        assert sess.device_status("select") == xkv.OK
        got = (sess.k_pages.clone(), sess.v_pages.clone(), sess.seq_lens.clone())
        if first is None:
            first = got
        else:
            assert all(_same(a, b) for a, b in zip(got, first)), ("select", rep)
    # ---- decode over the same caches, nothing appended, so every call sees the same state
    q, _, _ = WL.decode_tensors(w, 0, DEV, stress=True)
    first = None
    for rep in range(REPS):
        out = torch.full_like(sess.out, float("nan"))
        sess.decode(q, None, None, out=out)
        torch.cuda.synchronize()
        assert sess.device_status("decode") == xkv.OK
        if first is None:
            first = out.clone()
        else:
            assert _same(out, first), ("decode", rep)


def test_int8_cache_decode_is_repeatable():
    require_lib()
    w = CASES["two_pass_gw128"]
    lengths = WL.prompt_lengths(w)
    N = w.avg_budget
    sess = XkvSession(1, w.n_q_heads, w.n_kv_heads, w.head_dim, w.window, w.pool_kernel, lengths, max_new_tokens=1,
                      total_budget=N, device=DEV, kv_format=xkv.KV_INT8)
    q_win, k, v = WL.layer_tensors(w, 0, DEV, lengths, stress=True)
    sess.score_layer(0, q_win, k)
    budgets, _ = sess.solve_budgets(total=N)
    sess.assign_pages(budgets)
    sess.select_layer(0, int(budgets[0]), k, v)
    torch.cuda.synchronize()
    assert sess.device_status("select") == xkv.OK
    q, _, _ = WL.decode_tensors(w, 0, DEV, stress=True)
    first = None
    for rep in range(REPS):
        out = torch.full_like(sess.out, float("nan"))
        sess.decode(q, None, None, out=out)
        torch.cuda.synchronize()
        assert sess.device_status("decode") == xkv.OK
        if first is None:
            first = out.clone()
        else:
            assert _same(out, first), rep
