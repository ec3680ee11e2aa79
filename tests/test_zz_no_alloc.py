"""xkv_decode_attn_static: the decode step for callers that cannot pass a workspace (a fixed memory
plan, a plug-in that only gets its inputs and outputs, a path where allocating would stall the GPU).
Its scratch is a fixed array inside the library, so the check here is simple: on the same cache and
the same inputs it must give what xkv_decode_attn gives, on two calls in a row (the second call
reuses the scratch the first one left behind), and it must refuse problems that do not fit."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import xkv_oracle as O
from paper_2412_05896_b200 import xkv

from gpu_util import ATOL, RTOL, DirectCache, check_attention, f64, require_lib

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_static_scratch_decode_matches_workspace_decode_twice():
    require_lib()
    L, B, Hq, Hkv, d, ps = 3, 4, 8, 2, 128, 16
    lens = [[700, 64, 1, 0], [2050, 129, 640, 63], [15, 16, 17, 300]]
    # two identical caches: every call appends, so each entry point needs its own copy
    ref_cache = DirectCache(L, B, Hkv, d, lens, ps, extra_rows=3, device=DEV, seed=77)
    sta_cache = DirectCache(L, B, Hkv, d, lens, ps, extra_rows=3, device=DEV, seed=77)
    dims = xkv.Dims(B, Hq, Hkv, d, 16, 1, 0, 0.0, Hkv * d, d)
    chunk_rows = 128                                   # several chunks per long sequence: partials + tickets in use
    need = xkv.workspace_bytes(xkv.OP_DECODE_ATTN, dims, n_layers=L, max_cache_len=ref_cache.max_pages * ps,
                               chunk_rows=chunk_rows)
    assert need <= xkv.STATIC_SCRATCH_BYTES
    ws = torch.zeros(need, dtype=torch.uint8, device=DEV)
    out_ref = torch.empty(L, B, Hq, d, dtype=torch.bfloat16, device=DEV)
    out_sta = torch.empty_like(out_ref)
    lse_ref = torch.empty(L, B, Hq, dtype=torch.float32, device=DEV)
    lse_sta = torch.empty_like(lse_ref)
    status = torch.full((1,), -99, dtype=torch.int32, device=DEV)
    g = torch.Generator(device="cpu").manual_seed(5)
    for call in range(2):
        q = torch.randn(L, B, Hq, d, generator=g).to(torch.bfloat16).to(DEV)
        kn = torch.randn(L, B, Hkv, d, generator=g).to(torch.bfloat16).to(DEV)
        vn = torch.randn(L, B, Hkv, d, generator=g).to(torch.bfloat16).to(DEV)
        xkv.decode_attn(dims, ref_cache.handle(), 0, L, q, kn, vn, out_ref, lse_ref, chunk_rows, ws)
        xkv.decode_attn_static(dims, sta_cache.handle(), 0, L, q, kn, vn, out_sta, lse_sta, chunk_rows, status)
        torch.cuda.synchronize()
        assert xkv.read_device_status(ws) == xkv.OK
        assert int(status.item()) == xkv.OK
        a, b = out_ref.float().cpu().numpy(), out_sta.float().cpu().numpy()
        assert np.all(np.isfinite(b))
        assert np.all(np.abs(a - b) <= ATOL + RTOL * np.abs(a)), f"call {call}: outputs differ"
        la, lb = lse_ref.cpu().numpy(), lse_sta.cpu().numpy()
        fin = np.isfinite(la)
        assert np.array_equal(fin, np.isfinite(lb)) and np.allclose(la[fin], lb[fin], atol=2e-3, rtol=1e-4)
        assert torch.equal(ref_cache.seq_lens, sta_cache.seq_lens)
        # and against the fp64 attention of Eq. 1 over the same rows, so that this file stands on its own
        sta_cache.append_host(kn, vn)
        want = np.zeros((L, B, Hq, d))
        for l in range(L):
            for bb in range(B):
                K, V = f64(sta_cache.K[(l, bb)]), f64(sta_cache.V[(l, bb)])
                for h in range(Hq):
                    want[l, bb, h], _ = O.decode_attention(f64(q[l, bb, h]), K[:, h // (Hq // Hkv)], V[:, h // (Hq // Hkv)])
        check_attention(out_sta, want, f"call {call} against the oracle")


def test_static_scratch_rejects_problems_beyond_its_size():
    require_lib()
    L, B, Hq, Hkv, d, ps = 64, 64, 64, 8, 128, 16
    dims = xkv.Dims(B, Hq, Hkv, d, 16, 1, 0, 0.0, Hkv * d, d)
    assert xkv.workspace_bytes(xkv.OP_DECODE_ATTN, dims, n_layers=L, max_cache_len=4096) > xkv.STATIC_SCRATCH_BYTES
    # pointers only need to be well-formed: the size check refuses the call before anything is launched
    buf = torch.zeros(1 << 16, dtype=torch.uint8, device=DEV)
    p = buf.data_ptr()
    cache = xkv.Cache(p, p, p, p, L, ps, 256, 8)
    rc = xkv.lib().xkv_decode_attn_static(ctypes.byref(dims), ctypes.byref(cache), 0, L, p, None, None, p, None, 0,
                                          None, None)
    assert rc == xkv.ERR_WORKSPACE
    with pytest.raises(xkv.XkvError):
        xkv.decode_attn_static(dims, cache, 0, L, p, None, None, p, None, 0)
