"""Helpers shared by the GPU parity tests: exact widening of bf16 tensors for the oracle and a
direct (torch indexing) construction of ragged paged caches for tests of the decode step alone."""
from __future__ import annotations

import math

import numpy as np
import torch

from paper_2412_05896_b200 import build, xkv

ATOL, RTOL = 2e-2, 1e-2          # attention outputs in bf16
REL_L2 = 1e-2                    # per-head relative L2 error on O(1) outputs


def require_lib():
    build.build()
    return xkv.lib()


def f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


def bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


class DirectCache:
    """A ragged paged cache filled by torch indexing (not by the library): K/V rows of every
    (layer, sequence) are scattered into randomly ordered pages."""

    def __init__(self, L, B, Hkv, d, lens, page_size, extra_rows, device, seed=0, v_shift=0.0, k_rows=None):
        g = torch.Generator(device="cpu").manual_seed(seed)
        self.L, self.B, self.Hkv, self.d, self.page_size = L, B, Hkv, d, page_size
        self.lens = np.asarray(lens, dtype=np.int64).reshape(L, B)
        self.max_pages = max(1, math.ceil((int(self.lens.max()) + extra_rows) / page_size))
        need = L * B * self.max_pages
        self.n_pages = need + 3
        perm = torch.randperm(self.n_pages, generator=g)[:need].to(torch.int32).reshape(L, B, self.max_pages)
        self.block_table = perm.to(device)
        # poison pages with NaN patterns so that rows beyond a sequence's end must be ignored
        self.k_pages = torch.full((self.n_pages, Hkv, page_size, d), float("nan"), dtype=torch.bfloat16, device=device)
        self.v_pages = torch.full((self.n_pages, Hkv, page_size, d), float("nan"), dtype=torch.bfloat16, device=device)
        self.K, self.V = {}, {}
        for l in range(L):
            for b in range(B):
                n = int(self.lens[l, b])
                k = torch.randn(n, Hkv, d, generator=g).to(torch.bfloat16)
                if k_rows is not None:                      # caller-made keys: k_rows(l, b, n) -> [n, Hkv, d]
                    k = k_rows(l, b, n).to(torch.bfloat16)
                v = (torch.randn(n, Hkv, d, generator=g) + v_shift).to(torch.bfloat16)
                self.K[(l, b)], self.V[(l, b)] = k, v
                if n == 0:
                    continue
                slots = torch.arange(n)
                pages = perm[l, b][slots // page_size].long()
                self.k_pages[pages.to(device), :, (slots % page_size).to(device)] = k.to(device)
                self.v_pages[pages.to(device), :, (slots % page_size).to(device)] = v.to(device)
        self.seq_lens = torch.tensor(self.lens, dtype=torch.int32, device=device)

    def handle(self) -> xkv.Cache:
        return xkv.Cache(self.k_pages.data_ptr(), self.v_pages.data_ptr(), self.block_table.data_ptr(),
                         self.seq_lens.data_ptr(), self.L, self.page_size, self.max_pages, self.n_pages)

    def append_host(self, k_new: torch.Tensor, v_new: torch.Tensor):
        for l in range(self.L):
            for b in range(self.B):
                self.K[(l, b)] = torch.cat([self.K[(l, b)], k_new[l, b].cpu()[None]], 0)
                self.V[(l, b)] = torch.cat([self.V[(l, b)], v_new[l, b].cpu()[None]], 0)


def check_attention(out: torch.Tensor, ref: np.ndarray, what: str = "", rel_l2: bool = False):
    """out bf16 [..., d] against the fp64 oracle within 2e-2 abs / 1e-2 rel."""
    got = f64(out)
    assert np.all(np.isfinite(got)), f"{what}: non-finite output"
    err = np.abs(got - ref)
    bound = ATOL + RTOL * np.abs(ref)
    worst = float((err - bound).max())
    assert worst <= 0, f"{what}: |err| exceeds 2e-2 + 1e-2|ref| by {worst:.3e} (max err {err.max():.3e})"
    if rel_l2:
        num = np.linalg.norm(got - ref, axis=-1)
        den = np.linalg.norm(ref, axis=-1)
        r = float((num / np.maximum(den, 1e-30)).max())
        assert r <= REL_L2, f"{what}: relative L2 error {r:.3e} > {REL_L2}"
