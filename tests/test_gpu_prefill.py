"""GPU parity of xkv_score and xkv_select_compact (Eq. 2-4; Alg. 2) against the fp64 oracle."""
import numpy as np
import pytest
import torch

from oracle import xkv_oracle as O
from paper_2412_05896_b200 import xkv
from paper_2412_05896_b200.pipeline import XkvSession

from gpu_util import bits, f64, require_lib

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
MODE = {0: "max", 1: "avg"}


def _inputs(seed, lengths, Hq, Hkv, d, W, peaked=True):
    g = torch.Generator(device="cpu").manual_seed(seed)
    T = sum(lengths)
    k = torch.randn(T, Hkv, d, generator=g)
    u = torch.randn(Hkv, d, generator=g)
    u = u / u.norm(dim=-1, keepdim=True)
    heavy = (torch.rand(T, Hkv, generator=g) < 0.03).float()
    k = k + 3.0 * heavy[..., None] * u[None]
    q = torch.randn(len(lengths), Hq, W, d, generator=g)
    if peaked:
        q = (q + d ** 0.5 * u.repeat_interleave(Hq // Hkv, 0)[None, :, None, :]) / 0.7
    v = torch.randn(T, Hkv, d, generator=g)
    return q.to(torch.bfloat16), k.to(torch.bfloat16), v.to(torch.bfloat16)


def _oracle_scores(q, k, cu, W, ps, mode):
    return O.score_layer(f64(q), f64(k), cu, W, ps, MODE[mode])


def _check_scores(sess, layer, w_ref, lengths, Hkv, W):
    got = sess.scores[layer].cpu().numpy().astype(np.float64)
    srt = sess.sorted[layer].cpu().numpy()
    cu = sess.cu_host
    worst = 0.0
    for b, t in enumerate(lengths):
        P = max(t - W, 0)
        for g in range(Hkv):
            seg = got[g, cu[b]: cu[b] + t]
            ref = w_ref[(b, g)]
            assert np.all(seg[P:] == 0.0) and np.all(srt[g, cu[b] + P: cu[b] + t] == 0.0)
            if P == 0:
                continue
            err = np.abs(seg[:P] - ref)
            tol = 3e-5 * ref + 1e-7 * ref.max()
            worst = max(worst, float((err / np.maximum(ref, 1e-300))[ref > 1e-4 * ref.max()].max()))
            assert np.all(err <= tol), f"unit {(b, g)}: score error {float((err - tol).max()):.3e} over tolerance"
            # the sort is exact: same multiset, descending
            s = srt[g, cu[b]: cu[b] + P]
            assert np.array_equal(s, np.sort(sess.scores[layer][g, cu[b]: cu[b] + P].cpu().numpy())[::-1])
    return worst


CASES = [
    # lengths, Hq, Hkv, d, W, ps, mode
    ([300, 1000, 9], 4, 4, 64, 16, 5, 0),
    ([513, 128], 8, 2, 128, 32, 7, 0),
    ([700], 8, 2, 128, 8, 7, 1),
    ([2500, 1200], 8, 2, 128, 32, 7, 0),         # G*W = 128 query rows
    ([1500], 16, 4, 128, 64, 3, 0),              # G*W = 256 query rows
    ([9000, 4097], 2, 2, 128, 16, 7, 0),         # several sort chunks and merge passes
    ([33, 17, 16, 1], 2, 1, 64, 16, 1, 0),       # at and below the window length
    ([8192, 4500, 130], 2, 2, 128, 32, 7, 0),    # G*W = 32, single-read kernel with clusters of eight
    ([4096, 31, 32, 33, 160], 3, 3, 64, 32, 5, 1),   # G*W = 32, clusters of four, lengths around the window
    ([300, 1000, 5], 4, 4, 64, 8, 7, 1),         # G*W = 8 (MHA with the paper's window of 8): padded to 16 rows
    ([700, 129], 6, 2, 128, 8, 7, 0),            # G*W = 24: padded to 32 rows
    # the two-pass tensor-core kernels in every shape the dispatcher can pick (query rows x head dimension)
    ([2300, 900], 8, 1, 128, 8, 7, 1),           # G*W = 64, d = 128 (eight query heads per KV head, the paper's window of 8)
    ([1800, 2600], 4, 2, 64, 32, 5, 0),          # G*W = 64, d = 64
    ([9100, 300], 2, 2, 128, 32, 7, 0),          # G*W = 32, d = 128, a prompt beyond what the single-read kernel holds
    ([8300, 1000], 1, 1, 64, 32, 3, 0),          # G*W = 32, d = 64, likewise
    ([2100, 640], 8, 2, 64, 32, 7, 0),           # G*W = 128, d = 64
    ([1700, 130], 8, 1, 64, 32, 5, 1),           # G*W = 256, d = 64
]


@pytest.mark.parametrize("lengths,Hq,Hkv,d,W,ps,mode", CASES)
def test_score_sort_and_curves(lengths, Hq, Hkv, d, W, ps, mode):
    require_lib()
    q, k, v = _inputs(len(lengths) * 7 + W, lengths, Hq, Hkv, d, W)
    sess = XkvSession(1, Hq, Hkv, d, W, ps, lengths, pool_mode=mode, device=DEV)
    mass = torch.empty(len(lengths), sess.curve_len, dtype=torch.float32, device=DEV)
    sess.score_layer(0, q.to(DEV), k.to(DEV), mass=mass)
    torch.cuda.synchronize()
    assert sess.device_status("score") == xkv.OK
    w_ref = _oracle_scores(q, k, sess.cu_host, W, ps, mode)
    _check_scores(sess, 0, w_ref, lengths, Hkv, W)
    curves = O.layer_curves(w_ref, len(lengths), Hkv, sess.curve_len)
    got = sess.gains[0].cpu().numpy().astype(np.float64)
    assert np.allclose(got, curves, rtol=1e-4, atol=1e-7)
    got_mass = mass.cpu().numpy().astype(np.float64)
    assert np.allclose(got_mass, np.cumsum(curves, axis=1), rtol=0, atol=2e-5)
    for b, t in enumerate(lengths):
        if t > W:
            assert abs(got_mass[b, min(t - W, sess.curve_len) - 1] - 1.0) < 2e-5 or t - W > sess.curve_len


@pytest.mark.parametrize("Hq,Hkv,W", [(2, 2, 32), (8, 2, 32), (4, 2, 8)])
@pytest.mark.parametrize("profile", ["ramp", "jumps", "falling"])
def test_scores_with_logit_profiles_along_the_keys_and_across_rows(profile, Hq, Hkv, W):
    """Logits that rise, jump or fall along the key axis, with query rows of very different scale: the running
    softmax reference of a row is then raised often, rarely or never, and the rows of one tile sit hundreds of
    units apart (log2 domain)."""
    require_lib()
    d, ps, lengths = 128, 5, [3000, 777]
    T = sum(lengths)
    gen = torch.Generator(device="cpu").manual_seed(4242)
    u = (torch.randint(0, 2, (Hkv, d), generator=gen) * 2 - 1).to(torch.float32)           # q.k = a * c * d exactly
    unit = np.sqrt(d) * 1.4426950408889634                                                 # log2 units per a*c
    pos = torch.cat([torch.arange(t, dtype=torch.float32) / max(t - 1, 1) for t in lengths])
    if profile == "ramp":
        c = 60.0 / unit * pos
    elif profile == "jumps":
        c = 15.0 / unit * torch.floor(pos * 7.0)
    else:
        c = -60.0 / unit * pos
    k = c[:, None, None] * u[None] + 0.05 * torch.randn(T, Hkv, d, generator=gen)
    a = 0.25 * (1.0 + torch.arange(W, dtype=torch.float32))                                # row scale 0.25 .. W/4
    q = a[None, None, :, None] * u.repeat_interleave(Hq // Hkv, 0)[None, :, None, :] + \
        0.05 * torch.randn(len(lengths), Hq, W, d, generator=gen)
    q, k = q.to(torch.bfloat16), k.to(torch.bfloat16)
    sess = XkvSession(1, Hq, Hkv, d, W, ps, lengths, device=DEV)
    sess.score_layer(0, q.to(DEV), k.to(DEV))
    torch.cuda.synchronize()
    assert sess.device_status("score") == xkv.OK
    w_ref = _oracle_scores(q, k, sess.cu_host, W, ps, 0)
    _check_scores(sess, 0, w_ref, lengths, Hkv, W)


def _cache_rows(sess, layer, b, g, n):
    bt = sess.block_table[layer, b].cpu().numpy()
    slots = np.arange(n)
    pages = torch.from_numpy(bt[slots // sess.page_size].astype(np.int64)).to(sess.device)
    off = torch.from_numpy(slots % sess.page_size).to(sess.device)
    return bits(sess.k_pages[pages, g, off]), bits(sess.v_pages[pages, g, off])


@pytest.mark.parametrize("quantised", [True, False])
@pytest.mark.parametrize("d,page_size,lengths", [(128, 16, [1000, 4000, 40, 12, 3100]),       # one sweep step per unit
                                                 (64, 64, [1000, 13000, 40, 12, 4200])])      # chunked selection
def test_select_compact_is_bit_exact_on_given_scores(quantised, d, page_size, lengths):
    """Selection and compaction alone: scores are inputs, so the kept sets must equal the oracle's
    exactly (ties to the lower position) and the cache must hold the oracle's rows bit for bit."""
    require_lib()
    Hkv, W = 2, 16
    B, T = len(lengths), sum(lengths)
    g = torch.Generator(device="cpu").manual_seed(11 + d)
    scores = torch.rand(Hkv, T, generator=g) ** 4
    if quantised:
        scores = torch.round(scores * 12) / 12          # many exact ties, including at the threshold
    sess = XkvSession(1, Hkv, Hkv, d, W, 1, lengths, page_size=page_size, device=DEV)
    cu = sess.cu_host
    srt = torch.zeros_like(scores)
    for b, t in enumerate(lengths):
        P = max(t - W, 0)
        scores[:, cu[b] + P: cu[b] + t] = 0
        srt[:, cu[b]: cu[b] + P] = torch.sort(scores[:, cu[b]: cu[b] + P], dim=1, descending=True).values
    k = torch.randn(T, Hkv, d, generator=g).to(torch.bfloat16)
    v = torch.randn(T, Hkv, d, generator=g).to(torch.bfloat16)
    sess.scores[0].copy_(scores)
    sess.sorted[0].copy_(srt)
    for budget in (0, 1, 7, 300, 984, 985, 3999, 4183, 4184, 4185, 8200, 12983, 12984, 10 ** 6):
        sess.assign_pages([budget])
        sess.k_pages.fill_(float("nan"))
        sel = torch.full((B, Hkv, sess.max_seqlen), -1, dtype=torch.int32, device=DEV)
        sess.select_layer(0, budget, k.to(DEV), v.to(DEV), sel=sel)
        torch.cuda.synchronize()
        assert sess.device_status("select") == xkv.OK
        lens = sess.seq_lens[0].cpu().numpy()
        for b, t in enumerate(lengths):
            P = max(t - W, 0)
            for h in range(Hkv):
                keep = O.kept_positions(scores[h, cu[b]: cu[b] + P].double().numpy(), budget, t, W)
                assert lens[b] == len(keep)
                assert np.array_equal(sel[b, h, : len(keep)].cpu().numpy(), keep), (budget, b, h)
                kb, vb = _cache_rows(sess, 0, b, h, len(keep))
                assert np.array_equal(kb, O.evict_by_index(bits(k[cu[b]: cu[b] + t, h]), keep))
                assert np.array_equal(vb, O.evict_by_index(bits(v[cu[b]: cu[b] + t, h]), keep))


def test_select_per_sequence_budgets_and_capacity_status():
    require_lib()
    lengths, Hkv, W, d = [600, 900], 2, 16, 64
    q, k, v = _inputs(3, lengths, Hkv, Hkv, d, W)
    sess = XkvSession(1, Hkv, Hkv, d, W, 5, lengths, device=DEV, max_budget=200)
    sess.score_layer(0, q.to(DEV), k.to(DEV))
    budgets = np.array([[50], [120]], dtype=np.int32)
    sess.assign_pages(budgets)
    sess.select_layer(0, budgets[:, 0], k.to(DEV), v.to(DEV), per_sequence=True)
    torch.cuda.synchronize()
    assert sess.seq_lens[0].cpu().tolist() == [50 + W, 120 + W]
    # a budget beyond the page table is reported through the status word, nothing is written
    sess.select_layer(0, 800, k.to(DEV), v.to(DEV))
    torch.cuda.synchronize()
    assert sess.device_status("select") == xkv.ERR_CAPACITY
    assert sess.seq_lens[0].cpu().tolist() == [0, 0]


@pytest.mark.parametrize("lengths,Hq,Hkv,d,W,ps,mode", CASES[:5] + CASES[11:])
def test_selection_from_gpu_scores_matches_oracle_outside_near_ties(lengths, Hq, Hkv, d, W, ps, mode):
    """End to end through scoring: kept sets equal the oracle's wherever no other score lies within
    1e-5 (relative) of the k-th largest; inside that band only the band itself may differ."""
    require_lib()
    q, k, v = _inputs(5 + W, lengths, Hq, Hkv, d, W)
    sess = XkvSession(1, Hq, Hkv, d, W, ps, lengths, pool_mode=mode, device=DEV)
    sess.score_layer(0, q.to(DEV), k.to(DEV))
    w_ref = _oracle_scores(q, k, sess.cu_host, W, ps, mode)
    near, total = 0, 0
    for budget in (16, 100, 257):
        sess.assign_pages([budget])
        sel = torch.full((len(lengths), Hkv, sess.max_seqlen), -1, dtype=torch.int32, device=DEV)
        sess.select_layer(0, budget, k.to(DEV), v.to(DEV), sel=sel)
        torch.cuda.synchronize()
        for b, t in enumerate(lengths):
            for g in range(Hkv):
                w = w_ref[(b, g)]
                keep = O.kept_positions(w, budget, t, W)
                got = sel[b, g, : len(keep)].cpu().numpy()
                total += 1
                if O.near_tie(w, budget):
                    near += 1
                    thr = O.sort_descending(w)[min(budget, len(w)) - 1]
                    diff = np.setxor1d(got, keep)
                    assert np.all(np.abs(w[diff] - thr) <= 1e-5 * thr)
                else:
                    assert np.array_equal(got, keep), (budget, b, g)
    print(f"near-tie heads: {near} of {total}")


def test_status_of_an_early_layer_survives_the_later_layers_of_the_phase():
    """Layers share a few workspaces.  A layer whose budget does not fit its page table must still show in the
    phase's status after later layers, which fit, have run on the same workspace."""
    require_lib()
    lengths, Hkv, W, d, L = [600, 900], 2, 16, 64, 6
    q, k, v = _inputs(3, lengths, Hkv, Hkv, d, W)
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    sess = XkvSession(L, Hkv, Hkv, d, W, 5, lengths, device=DEV, max_budget=200, n_lanes=2)
    sess.score_layers([qd] * L, [kd] * L)
    assert sess.device_status("score") == xkv.OK
    budgets = np.array([50, 800, 60, 70, 80, 90], dtype=np.int32)       # layer 1 overflows its 200-token page table
    sess.assign_pages(np.minimum(budgets, 200))
    sess.select_layers(budgets, [kd] * L, [vd] * L)
    torch.cuda.synchronize()
    assert sess.device_status("select") == xkv.ERR_CAPACITY
    assert sess.device_status("select") == xkv.OK                        # read once, then clean
    lens = sess.seq_lens.cpu().numpy()
    assert lens[1].tolist() == [0, 0] and lens[0].tolist() == [50 + W, 50 + W] and lens[5].tolist() == [90 + W, 90 + W]


def test_prompt_longer_than_max_seqlen_is_reported_not_waited_for():
    """max_seqlen sizes the grids; a longer prompt on the device is cut to it and flagged, with no stall."""
    require_lib()
    lengths, Hq, Hkv, d, W = [1500, 400], 4, 2, 128, 16
    q, k, v = _inputs(9, lengths, Hq, Hkv, d, W)
    sess = XkvSession(1, Hq, Hkv, d, W, 5, lengths, device=DEV)
    sess.max_seqlen = 1024                                                # a wrong bound, below the first prompt
    sess.score_layer(0, q.to(DEV), k.to(DEV))
    torch.cuda.synchronize()
    assert sess.device_status("score") == xkv.ERR_INVALID_ARG
