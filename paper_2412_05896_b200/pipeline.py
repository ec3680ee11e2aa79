"""The call a user makes: one object that owns the device buffers of a batch (torch tensors for
memory and streams only) and drives the four library entry points in order.

    sess = XkvSession(...); sess.prefill(q_win, k, v, total_budget=...); sess.decode(q, k_new, v_new)

Every computation happens inside libxkv.so; this file allocates, copies and calls.
"""
from __future__ import annotations

import math

import numpy as np
import torch

from . import xkv


class XkvSession:
    def __init__(self, n_layers: int, n_q_heads: int, n_kv_heads: int, head_dim: int, window: int,
                 pool_kernel: int, lengths: list[int], pool_mode: int = xkv.POOL_MAX, page_size: int = 16,
                 max_new_tokens: int = 0, max_budget: int | None = None, total_budget: int | None = None,
                 curve_len: int | None = None, device="cuda:0", scale: float = 0.0,
                 decode_chunk_rows: int = 0):
        self.L, self.Hq, self.Hkv, self.d, self.W = n_layers, n_q_heads, n_kv_heads, head_dim, window
        self.B = len(lengths)
        self.lengths = list(lengths)
        self.device = torch.device(device)
        self.page_size = page_size
        self.max_new = max_new_tokens
        cu = [0]
        for t in lengths:
            cu.append(cu[-1] + t)
        self.T = cu[-1]
        self.max_seqlen = max(lengths)
        self.prefix = [max(t - window, 0) for t in lengths]
        self.max_prefix = max(self.prefix)
        self.cu_host = np.asarray(cu, dtype=np.int32)
        self.cu = torch.tensor(cu, dtype=torch.int32, device=self.device)
        self.dims = xkv.Dims(self.B, n_q_heads, n_kv_heads, head_dim, window, pool_kernel, pool_mode, scale,
                             n_kv_heads * head_dim, head_dim)

        # per-layer scores, their sort and the curves (kept for all layers: the solver needs every curve
        # before the first layer can be compacted)
        self.curve_len = max(1, min(curve_len or self.max_prefix, max(self.max_prefix, 1)))
        f32 = dict(dtype=torch.float32, device=self.device)
        self.scores = torch.empty(n_layers, n_kv_heads, self.T, **f32)
        self.sorted = torch.empty(n_layers, n_kv_heads, self.T, **f32)
        self.gains = torch.empty(n_layers, self.B, self.curve_len, **f32)
        self.gains_host = torch.empty(n_layers, self.B, self.curve_len, dtype=torch.float32, pin_memory=True)
        self.ws_score = self._ws(xkv.workspace_bytes(xkv.OP_SCORE, self.dims, self.max_seqlen, self.T))
        self.ws_select = self._ws(xkv.workspace_bytes(xkv.OP_SELECT_COMPACT, self.dims, self.max_seqlen, self.T))

        # ragged paged cache: a pool large enough for any split of the global budget
        per_layer_cap = min(max_budget if max_budget else self.max_prefix, self.max_prefix)
        self.max_cache_len = per_layer_cap + window + max_new_tokens
        self.max_pages_per_seq = max(1, math.ceil(self.max_cache_len / page_size))
        if total_budget is None:
            total_budget = n_layers * per_layer_cap
        total_budget = min(total_budget, n_layers * per_layer_cap)
        n_pages = 0
        for P, t in zip(self.prefix, lengths):
            rows = min(total_budget, n_layers * P) + n_layers * (min(window, t) + max_new_tokens + page_size)
            n_pages += math.ceil(rows / page_size)
        self.n_pages = max(n_pages, 1)
        bf16 = dict(dtype=torch.bfloat16, device=self.device)
        self.k_pages = torch.zeros(self.n_pages, n_kv_heads, page_size, head_dim, **bf16)
        self.v_pages = torch.zeros(self.n_pages, n_kv_heads, page_size, head_dim, **bf16)
        self.block_table = torch.zeros(n_layers, self.B, self.max_pages_per_seq, dtype=torch.int32,
                                       device=self.device)
        self.block_table_host = torch.zeros(n_layers, self.B, self.max_pages_per_seq, dtype=torch.int32,
                                            pin_memory=(self.device.type == "cuda"))
        self.seq_lens = torch.zeros(n_layers, self.B, dtype=torch.int32, device=self.device)
        self.cache = xkv.Cache(self.k_pages.data_ptr(), self.v_pages.data_ptr(), self.block_table.data_ptr(),
                               self.seq_lens.data_ptr(), n_layers, page_size, self.max_pages_per_seq,
                               self.n_pages)
        self.chunk_rows = decode_chunk_rows
        self.ws_decode = self._ws(xkv.workspace_bytes(xkv.OP_DECODE_ATTN, self.dims, n_layers=n_layers,
                                                      max_cache_len=self.max_pages_per_seq * page_size,
                                                      chunk_rows=decode_chunk_rows))
        self.out = torch.empty(n_layers, self.B, n_q_heads, head_dim, **bf16)
        self.lse = torch.empty(n_layers, self.B, n_q_heads, **f32)
        self.budgets: np.ndarray | None = None
        self.r_avg: float | None = None

    def _ws(self, nbytes: int) -> torch.Tensor:
        return torch.empty(nbytes, dtype=torch.uint8, device=self.device)

    # ------------------------------------------------------------------ prefill
    def score_layer(self, layer: int, q_win: torch.Tensor, k: torch.Tensor, want_curves: bool = True,
                    mass: torch.Tensor | None = None) -> None:
        xkv.score(self.dims, q_win, k, self.cu, self.T, self.max_seqlen, self.scores[layer],
                  self.sorted[layer] if want_curves else None, self.gains[layer] if want_curves else None,
                  mass, self.curve_len, self.ws_score)

    def solve_budgets(self, total: int | None = None, r_target: float = 0.0, n_min: int = 0, n_max: int = 0,
                      per_sequence: bool = False):
        """Curves device -> host (the one crossing of the prefill), then Algorithm 1 on the host."""
        self.gains_host.copy_(self.gains, non_blocking=True)
        torch.cuda.current_stream().synchronize()
        budgets, r_avg = xkv.alloc_budgets(self.gains_host.numpy(), np.asarray(self.prefix, dtype=np.int32),
                                           per_sequence=per_sequence, total=-1 if total is None else total,
                                           r_target=r_target, n_min=n_min, n_max=n_max)
        self.budgets, self.r_avg = budgets, r_avg
        return budgets, r_avg

    def assign_pages(self, budgets) -> None:
        """Hand consecutive pool pages to every (layer, sequence) for its kept rows plus new tokens."""
        budgets = np.asarray(budgets)
        k_lb = budgets.T if budgets.ndim == 2 else np.broadcast_to(budgets[:, None], (self.L, self.B))   # [L, B]
        prefix = np.asarray(self.prefix)[None, :]
        window = np.minimum(self.W, np.asarray(self.lengths))[None, :]
        rows = np.minimum(k_lb, prefix) + window + self.max_new
        n = np.minimum(-(-rows // self.page_size), self.max_pages_per_seq).astype(np.int64)               # pages
        start = np.concatenate([[0], np.cumsum(n.ravel())[:-1]]).reshape(self.L, self.B)
        if int(start.ravel()[-1] + n.ravel()[-1]) > self.n_pages:
            raise RuntimeError("page pool too small for these budgets")
        idx = np.arange(self.max_pages_per_seq, dtype=np.int64)[None, None, :]
        bt = self.block_table_host.numpy()
        bt[:] = np.where(idx < n[:, :, None], start[:, :, None] + idx, 0).astype(np.int32)
        self.block_table.copy_(self.block_table_host, non_blocking=True)

    def select_layer(self, layer: int, budget, k: torch.Tensor, v: torch.Tensor, sel: torch.Tensor | None = None,
                     per_sequence: bool = False) -> None:
        xkv.select_compact(self.dims, layer, budget, per_sequence, self.scores[layer], self.sorted[layer], k, v,
                           self.cu, self.T, self.max_seqlen, self.cache, sel,
                           0 if sel is None else sel.shape[-1], self.ws_select)

    def prefill(self, q_win: list[torch.Tensor], k: list[torch.Tensor], v: list[torch.Tensor],
                budgets=None, total: int | None = None, n_min: int = 0, n_max: int = 0):
        """Score every layer, split the budget (unless given), evict and compact every layer."""
        for l in range(self.L):
            self.score_layer(l, q_win[l], k[l])
        if budgets is None:
            budgets, _ = self.solve_budgets(total=total, n_min=n_min, n_max=n_max)
        else:
            self.budgets = np.asarray(budgets, dtype=np.int32)
        self.assign_pages(budgets)
        for l in range(self.L):
            self.select_layer(l, int(budgets[l]), k[l], v[l])
        return budgets

    # ------------------------------------------------------------------ generation
    def decode(self, q: torch.Tensor, k_new: torch.Tensor | None, v_new: torch.Tensor | None,
               out: torch.Tensor | None = None, lse: torch.Tensor | None = None, layer_begin: int = 0,
               layer_end: int | None = None, chunk_rows: int | None = None) -> torch.Tensor:
        out = self.out if out is None else out
        layer_end = self.L if layer_end is None else layer_end
        xkv.decode_attn(self.dims, self.cache, layer_begin, layer_end, q, k_new, v_new, out,
                        self.lse if lse is None else lse,
                        self.chunk_rows if chunk_rows is None else chunk_rows, self.ws_decode)
        return out

    def device_status(self, which: str = "decode") -> int:
        ws = {"decode": self.ws_decode, "score": self.ws_score, "select": self.ws_select}[which]
        return xkv.read_device_status(ws)
