"""GPU parity of xkv_prefill_attn (Eq. 1 with the weights of Eq. 2 over the whole prompt) and of xkv_score_lse
(Alg. 2 steps 1-4 from the normalisers the prefill attention produced) against the fp64 oracle."""
import numpy as np
import pytest
import torch

from oracle import xkv_oracle as O
from paper_2412_05896_b200 import xkv
from paper_2412_05896_b200.pipeline import XkvSession

from gpu_util import check_attention, f64, require_lib

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _prompt(seed, lengths, Hq, Hkv, d, W, temp=0.7):
    """Keys with heavy hitters and a sink, queries that look along the heavy direction (peaked attention), values
    shifted by +1 so that outputs are O(1).  The last W query rows of every sequence are the window queries."""
    g = torch.Generator(device="cpu").manual_seed(seed)
    T = sum(lengths)
    k = torch.randn(T, Hkv, d, generator=g)
    u = torch.randn(Hkv, d, generator=g)
    u = u / u.norm(dim=-1, keepdim=True)
    heavy = (torch.rand(T, Hkv, generator=g) < 0.03).float()
    k = k + 3.0 * heavy[..., None] * u[None]
    q = (torch.randn(T, Hq, d, generator=g) + d ** 0.5 * u.repeat_interleave(Hq // Hkv, 0)[None]) / temp
    v = torch.randn(T, Hkv, d, generator=g) + 1.0
    q, k, v = q.to(torch.bfloat16), k.to(torch.bfloat16), v.to(torch.bfloat16)
    q_win = torch.zeros(len(lengths), Hq, W, d, dtype=torch.bfloat16)
    lo = 0
    for b, t in enumerate(lengths):
        n = min(W, t)
        q_win[b, :, W - n:] = q[lo + t - n: lo + t].transpose(0, 1)
        lo += t
    return q, k, v, q_win


CASES = [
    # lengths, Hq, Hkv, d, W
    ([300, 515], 4, 2, 128, 16),          # G*W = 32; partial last tiles
    ([700], 2, 2, 64, 32),                # d = 64, MHA
    ([1100, 400, 128], 8, 2, 128, 32),    # G*W = 128
    ([129, 1, 127], 2, 1, 128, 32),       # G*W = 64; one-token and sub-tile sequences, a sequence shorter than the window
    ([2200], 4, 1, 128, 64),              # G*W = 256; many key tiles per query tile
]


@pytest.mark.parametrize("lengths,Hq,Hkv,d,W", CASES)
def test_prefill_attention_and_scores_from_its_normalisers(lengths, Hq, Hkv, d, W):
    require_lib()
    G, B, T = Hq // Hkv, len(lengths), sum(lengths)
    q, k, v, q_win = _prompt(11 * len(lengths) + W + d, lengths, Hq, Hkv, d, W)
    ps = 5
    sess = XkvSession(1, Hq, Hkv, d, W, ps, lengths, device=DEV)
    qd, kd, vd, qwd = q.to(DEV), k.to(DEV), v.to(DEV), q_win.to(DEV)
    out = torch.full((T, Hq, d), float("nan"), dtype=torch.bfloat16, device=DEV)
    lse = torch.full((Hq, T), float("nan"), dtype=torch.float32, device=DEV)
    ws = torch.zeros(xkv.workspace_bytes(xkv.OP_PREFILL_ATTN, sess.dims), dtype=torch.uint8, device=DEV)
    xkv.prefill_attn(sess.dims, qd, kd, vd, sess.cu, T, max(lengths), out, lse, ws)
    torch.cuda.synchronize()
    assert xkv.read_device_status(ws) == xkv.OK

    # ---- attention outputs and normalisers, every row of every head
    qf, kf, vf = f64(q), f64(k), f64(v)
    ref = np.zeros((T, Hq, d))
    ref_lse = np.zeros((Hq, T))
    cu = sess.cu_host
    for b, t in enumerate(lengths):
        lo = int(cu[b])
        for h in range(Hq):
            z, l = O.prefill_attention(qf[lo: lo + t, h], kf[lo: lo + t, h // G], vf[lo: lo + t, h // G])
            ref[lo: lo + t, h] = z
            ref_lse[h, lo: lo + t] = l
    check_attention(out, ref, "prefill attention", rel_l2=True)
    got_lse = lse.cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(got_lse))
    assert np.all(np.abs(got_lse - ref_lse) <= 2e-4 + 1e-5 * np.abs(ref_lse)), float(np.abs(got_lse - ref_lse).max())

    # ---- scores from those normalisers against the definition (window queries alone, two passes in the oracle)
    w_ref = O.score_layer(f64(q_win), kf, cu, W, ps, "max")
    for given, what in ((lse, "normalisers of the GPU attention"),
                        (torch.from_numpy(ref_lse.astype(np.float32)).to(DEV), "normalisers of the oracle")):
        sess.scores.fill_(float("nan"))
        xkv.score_lse(sess.dims, qwd, kd, sess.cu, T, max(lengths), given, sess.scores[0], sess.sorted[0],
                      sess.gains[0], None, sess.curve_len, sess.ws_score[0])
        torch.cuda.synchronize()
        assert sess.device_status("score") == xkv.OK
        got = sess.scores[0].cpu().numpy().astype(np.float64)
        for b, t in enumerate(lengths):
            P = max(t - W, 0)
            for g in range(Hkv):
                seg = got[g, cu[b]: cu[b] + t]
                assert np.all(seg[P:] == 0.0)
                if P == 0:
                    continue
                r = w_ref[(b, g)]
                err = np.abs(seg[:P] - r)
                assert np.all(err <= 3e-5 * r + 1e-7 * r.max()), (what, b, g, float((err / r.max()).max()))
        curves = O.layer_curves(w_ref, B, Hkv, sess.curve_len)
        assert np.allclose(sess.gains[0].cpu().numpy().astype(np.float64), curves, rtol=1e-4, atol=1e-7), what

    # ---- the one-pass scores agree with the two-pass xkv_score on the same inputs (same tolerance, both ways)
    two_pass = torch.empty_like(sess.scores[0])
    xkv.score(sess.dims, qwd, kd, sess.cu, T, max(lengths), two_pass, None, None, None, 1, sess.ws_score[0])
    torch.cuda.synchronize()
    a, b2 = sess.scores[0].cpu().numpy().astype(np.float64), two_pass.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(a - b2) <= 6e-5 * np.maximum(a, b2) + 2e-7 * a.max())


def test_score_lse_rejections():
    require_lib()
    lengths, Hq, Hkv, d, W = [400], 3, 1, 128, 8                    # G*W = 24: not a shape the one-pass kernel covers
    q, k, v, q_win = _prompt(5, lengths, Hq, Hkv, d, W)
    sess = XkvSession(1, Hq, Hkv, d, W, 5, lengths, device=DEV)
    lse = torch.zeros(Hq, 400, dtype=torch.float32, device=DEV)
    with pytest.raises(xkv.XkvError) as e:
        xkv.score_lse(sess.dims, q_win.to(DEV), k.to(DEV), sess.cu, 400, 400, lse, sess.scores[0], None, None, None, 1,
                      sess.ws_score[0])
    assert e.value.status == xkv.ERR_UNSUPPORTED
    sess2 = XkvSession(1, 4, 1, d, W, 5, lengths, device=DEV)         # G*W = 32
    with pytest.raises(xkv.XkvError) as e:
        xkv.score_lse(sess2.dims, q_win.to(DEV), k.to(DEV), sess2.cu, 400, 400, None, sess2.scores[0], None, None, None,
                      1, sess2.ws_score[0])
    assert e.value.status == xkv.ERR_INVALID_ARG
    ws = torch.zeros(256, dtype=torch.uint8, device=DEV)
    out = torch.empty(400, 4, d, dtype=torch.bfloat16, device=DEV)
    with pytest.raises(xkv.XkvError) as e:
        xkv.prefill_attn(sess2.dims, None, k.to(DEV), v.to(DEV), sess2.cu, 400, 400, out, None, ws)
    assert e.value.status == xkv.ERR_INVALID_ARG


def test_prefill_attention_is_repeatable():
    """The same call, many times: outputs and normalisers must be bit-identical every time (a hand-over between the
    kernel's roles that depended on timing would show as a difference sooner or later)."""
    require_lib()
    lengths, Hq, Hkv, d, W = [3000, 1700, 900], 8, 2, 128, 32
    q, k, v, _ = _prompt(123, lengths, Hq, Hkv, d, W)
    T = sum(lengths)
    sess = XkvSession(1, Hq, Hkv, d, W, 5, lengths, device=DEV)
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    ws = torch.zeros(xkv.workspace_bytes(xkv.OP_PREFILL_ATTN, sess.dims), dtype=torch.uint8, device=DEV)
    first = None
    for rep in range(100):
        out = torch.full((T, Hq, d), float("nan"), dtype=torch.bfloat16, device=DEV)
        lse = torch.full((Hq, T), float("nan"), dtype=torch.float32, device=DEV)
        xkv.prefill_attn(sess.dims, qd, kd, vd, sess.cu, T, max(lengths), out, lse, ws)
        torch.cuda.synchronize()
        assert xkv.read_device_status(ws) == xkv.OK
        if first is None:
            first = (out.clone(), lse.clone())
        else:
            assert torch.equal(out.view(torch.int16), first[0].view(torch.int16)), rep
            assert torch.equal(lse.view(torch.int32), first[1].view(torch.int32)), rep
