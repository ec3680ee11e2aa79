"""GPU parity of xkv_decode_attn (Eq. 1, generation phase) against the fp64 oracle, on ragged caches
built directly with torch so that this step is tested alone."""
import numpy as np
import pytest
import torch

from oracle import xkv_oracle as O
from paper_2412_05896_b200 import xkv

from gpu_util import DirectCache, check_attention, f64, require_lib

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _run_case(L, B, Hq, Hkv, d, lens, page_size, chunk_rows, append, seed, stress=False, steps=1):
    require_lib()
    G = Hq // Hkv
    cache = DirectCache(L, B, Hkv, d, lens, page_size, extra_rows=steps + 1, device=DEV, seed=seed,
                        v_shift=1.0 if stress else 0.0)
    dims = xkv.Dims(B, Hq, Hkv, d, 16, 1, 0, 0.0, Hkv * d, d)
    handle = cache.handle()
    ws_bytes = xkv.workspace_bytes(xkv.OP_DECODE_ATTN, dims, n_layers=L,
                                   max_cache_len=cache.max_pages * page_size, chunk_rows=chunk_rows)
    ws = torch.zeros(ws_bytes, dtype=torch.uint8, device=DEV)
    out = torch.empty(L, B, Hq, d, dtype=torch.bfloat16, device=DEV)
    lse = torch.empty(L, B, Hq, dtype=torch.float32, device=DEV)
    g = torch.Generator(device="cpu").manual_seed(seed + 1000)
    for step in range(steps):
        q = (torch.randn(L, B, Hq, d, generator=g) * (4.0 if stress else 1.0)).to(torch.bfloat16)
        k_new = torch.randn(L, B, Hkv, d, generator=g).to(torch.bfloat16)
        v_new = (torch.randn(L, B, Hkv, d, generator=g) + (1.0 if stress else 0.0)).to(torch.bfloat16)
        qd = q.to(DEV)
        if append:
            xkv.decode_attn(dims, handle, 0, L, qd, k_new.to(DEV), v_new.to(DEV), out, lse, chunk_rows, ws)
            cache.append_host(k_new, v_new)
        else:
            xkv.decode_attn(dims, handle, 0, L, qd, None, None, out, lse, chunk_rows, ws)
        torch.cuda.synchronize()
        assert xkv.read_device_status(ws) == xkv.OK
        ref = np.zeros((L, B, Hq, d))
        ref_lse = np.zeros((L, B, Hq))
        for l in range(L):
            for b in range(B):
                K, V = f64(cache.K[(l, b)]), f64(cache.V[(l, b)])
                for h in range(Hq):
                    ref[l, b, h], ref_lse[l, b, h] = O.decode_attention(f64(q[l, b, h]), K[:, h // G], V[:, h // G])
        check_attention(out, ref, f"step {step}", rel_l2=stress)
        got_lse = lse.cpu().numpy().astype(np.float64)
        finite = np.isfinite(ref_lse)
        assert np.array_equal(np.isfinite(got_lse), finite)
        assert np.allclose(got_lse[finite], ref_lse[finite], atol=2e-3, rtol=1e-4)
        if append:
            expect = np.array([[cache.K[(l, b)].shape[0] for b in range(B)] for l in range(L)])
            assert np.array_equal(cache.seq_lens.cpu().numpy(), expect)


@pytest.mark.parametrize("d,Hq,Hkv", [(64, 4, 4), (128, 4, 4), (128, 8, 2), (128, 8, 1), (64, 4, 2)])
def test_decode_ragged_lengths_with_append(d, Hq, Hkv):
    lens = [[0, 1, 15], [16, 17, 63], [64, 65, 300], [1000, 129, 33]]
    _run_case(4, 3, Hq, Hkv, d, lens, 16, 0, True, seed=d + Hq, steps=2)


@pytest.mark.parametrize("chunk_rows", [64, 128, 0])
@pytest.mark.parametrize("page_size", [16, 64])
def test_decode_split_invariance_and_page_sizes(chunk_rows, page_size):
    lens = [[700, 64, 1, 0], [2050, 129, 640, 63]]
    _run_case(2, 4, 8, 2, 128, lens, page_size, chunk_rows, False, seed=chunk_rows + page_size)


def test_decode_peaked_attention_and_shifted_values():
    lens = [[2000, 513], [777, 4096]]
    _run_case(2, 2, 8, 2, 128, lens, 16, 0, True, seed=5, stress=True, steps=2)
    _run_case(2, 2, 4, 4, 64, lens, 32, 256, True, seed=6, stress=True)


@pytest.mark.parametrize("profile", ["ramp", "jumps", "falling", "late_peak"])
def test_decode_score_profiles_along_the_cache(profile):
    """Scores that rise slowly, jump, fall or peak at the very end along the cache: the running softmax
    maximum is then raised often, rarely, never after the first tile, or once at the last row."""
    require_lib()
    L, B, Hq, Hkv, d, ps = 1, 3, 8, 2, 128, 16
    lens = [[700, 333, 2049]]
    gen = torch.Generator(device="cpu").manual_seed(77)
    u = (torch.randint(0, 2, (Hkv, d), generator=gen) * 2 - 1).to(torch.float32)      # +-1: q.k = c * d exactly
    unit = np.sqrt(d) * 1.4426950408889634                                            # log2-domain score per unit c

    def k_rows(l, b, n):
        j = torch.arange(n, dtype=torch.float32)
        if profile == "ramp":
            c = 60.0 / unit * j / max(n - 1, 1)                       # about +0.03 .. +0.2 per row, +60 overall
        elif profile == "jumps":
            c = 20.0 / unit * torch.floor(j / 97.0)                   # +20 every 97 rows
        elif profile == "falling":
            c = -40.0 / unit * j / max(n - 1, 1)
        else:
            c = torch.zeros(n)
            c[-1] = 30.0 / unit                                        # one dominant row at the end
        noise = 0.05 * torch.randn(n, Hkv, d, generator=gen)
        return c[:, None, None] * u[None] + noise

    cache = DirectCache(L, B, Hkv, d, lens, ps, extra_rows=1, device=DEV, seed=8, k_rows=k_rows)
    dims = xkv.Dims(B, Hq, Hkv, d, 16, 1, 0, 0.0, Hkv * d, d)
    G = Hq // Hkv
    q = torch.stack([u[h // G] for h in range(Hq)])[None, None].repeat(L, B, 1, 1).to(torch.bfloat16)
    for chunk_rows in (0, 128):
        ws = torch.zeros(xkv.workspace_bytes(xkv.OP_DECODE_ATTN, dims, n_layers=L, max_cache_len=cache.max_pages * ps,
                                             chunk_rows=chunk_rows), dtype=torch.uint8, device=DEV)
        out = torch.empty(L, B, Hq, d, dtype=torch.bfloat16, device=DEV)
        lse = torch.empty(L, B, Hq, dtype=torch.float32, device=DEV)
        xkv.decode_attn(dims, cache.handle(), 0, L, q.to(DEV), None, None, out, lse, chunk_rows, ws)
        torch.cuda.synchronize()
        assert xkv.read_device_status(ws) == xkv.OK
        ref = np.zeros((L, B, Hq, d))
        ref_lse = np.zeros((L, B, Hq))
        for b in range(B):
            K, V = f64(cache.K[(0, b)]), f64(cache.V[(0, b)])
            for h in range(Hq):
                ref[0, b, h], ref_lse[0, b, h] = O.decode_attention(f64(q[0, b, h]), K[:, h // G], V[:, h // G])
        check_attention(out, ref, f"{profile} chunk {chunk_rows}", rel_l2=True)
        assert np.allclose(lse.cpu().numpy().astype(np.float64), ref_lse, atol=2e-3, rtol=1e-4)


def test_decode_many_units_long_chunks():
    rng = np.random.default_rng(3)
    lens = rng.integers(1, 900, size=(6, 16)).tolist()
    _run_case(6, 16, 8, 8, 128, lens, 16, 0, True, seed=9)


def test_decode_more_units_than_the_attention_kernel_plans_for_itself():
    """Above 2048 (layer, sequence) units a separate kernel appends and writes the work-item table."""
    rng = np.random.default_rng(11)
    lens = rng.integers(0, 70, size=(8, 300)).tolist()
    _run_case(8, 300, 2, 1, 64, lens, 16, 0, True, seed=21, steps=2)
    _run_case(8, 300, 2, 1, 64, lens, 16, 64, False, seed=22)


def test_decode_capacity_overflow_is_reported_not_faulted():
    require_lib()
    L, B, Hq, Hkv, d, ps = 1, 2, 4, 4, 64, 16
    cache = DirectCache(L, B, Hkv, d, [[16, 5]], ps, extra_rows=0, device=DEV, seed=1)
    assert cache.max_pages == 1                      # sequence 0 is exactly full
    dims = xkv.Dims(B, Hq, Hkv, d, 16, 1, 0, 0.0, Hkv * d, d)
    ws = torch.zeros(xkv.workspace_bytes(xkv.OP_DECODE_ATTN, dims, n_layers=L, max_cache_len=ps),
                     dtype=torch.uint8, device=DEV)
    q = torch.randn(L, B, Hq, d, device=DEV).to(torch.bfloat16)
    kn = torch.randn(L, B, Hkv, d, device=DEV).to(torch.bfloat16)
    out = torch.empty_like(q)
    xkv.decode_attn(dims, cache.handle(), 0, L, q, kn, kn, out, None, 0, ws)
    torch.cuda.synchronize()
    assert xkv.read_device_status(ws) == xkv.ERR_CAPACITY
    assert cache.seq_lens.cpu().tolist() == [[16, 6]]


def test_bounded_wait_expires_with_a_status_and_the_workspace_stays_usable():
    """Failure detection without a fault: the split-K merge of one head waits for a chunk whose ticket a test
    hook withholds, with the wait limit shortened to a millisecond.  The kernel must return, the status word
    must read XKV_ERR_TIMEOUT, and the next ordinary call on the same workspace must be clean and correct."""
    require_lib()
    L, B, Hq, Hkv, d, ps, chunk_rows = 1, 2, 4, 2, 128, 16, 64
    lens = [[300, 40]]
    cache = DirectCache(L, B, Hkv, d, lens, ps, extra_rows=1, device=DEV, seed=31)
    dims = xkv.Dims(B, Hq, Hkv, d, 16, 1, 0, 0.0, Hkv * d, d)
    ws = torch.zeros(xkv.workspace_bytes(xkv.OP_DECODE_ATTN, dims, n_layers=L, max_cache_len=cache.max_pages * ps,
                                         chunk_rows=chunk_rows), dtype=torch.uint8, device=DEV)
    q = torch.randn(L, B, Hq, d, generator=torch.Generator().manual_seed(3)).to(torch.bfloat16).to(DEV)
    out = torch.zeros(L, B, Hq, d, dtype=torch.bfloat16, device=DEV)
    try:
        xkv.test_hooks(wait_limit_ns=1_000_000, withhold_decode_item=2)    # a chunk of sequence 0, KV head 0
        xkv.decode_attn(dims, cache.handle(), 0, L, q, None, None, out, None, chunk_rows, ws)
        torch.cuda.synchronize()
    finally:
        xkv.test_hooks()
    assert xkv.read_device_status(ws) == xkv.ERR_TIMEOUT
    assert xkv.read_device_status(ws) == xkv.OK                            # reading reset the word
    xkv.decode_attn(dims, cache.handle(), 0, L, q, None, None, out, None, chunk_rows, ws)
    torch.cuda.synchronize()
    assert xkv.read_device_status(ws) == xkv.OK
    G = Hq // Hkv
    ref = np.zeros((L, B, Hq, d))
    for b in range(B):
        K, V = f64(cache.K[(0, b)]), f64(cache.V[(0, b)])
        for h in range(Hq):
            ref[0, b, h], _ = O.decode_attention(f64(q[0, b, h]), K[:, h // G], V[:, h // G])
    check_attention(out, ref, "call after the expired wait")
