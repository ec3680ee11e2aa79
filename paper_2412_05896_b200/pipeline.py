"""The call a user makes: one object that owns the device buffers of a batch (torch tensors for
memory and streams only) and drives the four library entry points in order.

    sess = XkvSession(...); sess.prefill(q_win, k, v, total=...); sess.decode(q, k_new, v_new)

Every computation happens inside libxkv.so; this file allocates, copies and calls.
"""
from __future__ import annotations

import ctypes
import math
import time

import numpy as np
import torch

from . import xkv


class XkvSession:
    def __init__(self, n_layers: int, n_q_heads: int, n_kv_heads: int, head_dim: int, window: int,
                 pool_kernel: int, lengths: list[int], pool_mode: int = xkv.POOL_MAX, page_size: int = 16,
                 max_new_tokens: int = 0, max_budget: int | None = None, total_budget: int | None = None,
                 curve_len: int | None = None, device="cuda:0", scale: float = 0.0,
                 decode_chunk_rows: int = 0, n_lanes: int = 6, head_level: bool = False,
                 kv_format: int = xkv.KV_BF16):
        """head_level: budgets, cache lengths and page lists per (layer, sequence, KV head) instead of per (layer,
        sequence); total_budget and the solver's total then count prefix tokens over all heads of all layers, and
        max_budget bounds one head."""
        self.L, self.Hq, self.Hkv, self.d, self.W = n_layers, n_q_heads, n_kv_heads, head_dim, window
        self.head_level = bool(head_level)
        self.kv_format = kv_format                 # xkv.KV_INT8: the reduced caches hold 8-bit codes and row scales
        self.G = n_q_heads // n_kv_heads
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
        # (a multiple of four ranks, so that every layer's slice of the stacked arrays starts on a 16-byte boundary;
        # ranks beyond the longest prefix read zero)
        self.curve_len = (max(1, min(curve_len or self.max_prefix, max(self.max_prefix, 1))) + 3) // 4 * 4
        f32 = dict(dtype=torch.float32, device=self.device)
        self._layer_stride = (n_kv_heads * self.T + 3) // 4 * 4           # floats between the layers' score arrays
        self.scores = torch.empty(n_layers, self._layer_stride, **f32)[:, : n_kv_heads * self.T].view(
            n_layers, n_kv_heads, self.T)
        self.sorted = torch.empty(n_layers, self._layer_stride, **f32)[:, : n_kv_heads * self.T].view(
            n_layers, n_kv_heads, self.T)
        self.gains = torch.empty(n_layers, self.B, self.curve_len, **f32)
        # what crosses to the host for the solver: one curve per layer (the batch mean, formed on the device);
        # the per-sequence curves cross only when every sequence gets its own list
        # units of the solver: layers, or (layer, KV head) pairs with head-level budgets
        self.n_solver_units = n_layers * (n_kv_heads if self.head_level else 1)
        self.head_gains = torch.empty(n_layers, n_kv_heads, self.B, self.curve_len, **f32) if self.head_level else None
        self.layer_gains = torch.empty(self.n_solver_units, self.curve_len, **f32)
        self.layer_gains_host = torch.empty(self.n_solver_units, self.curve_len, dtype=torch.float32, pin_memory=True)
        self.gains_host = None
        # Layers are independent in the scoring and in the eviction phase, so consecutive layers go to
        # n_lanes side streams, each with its own workspace: the short latency-bound kernels of one layer
        # (sort, curves, selection) then run under the HBM-bound ones of the next.
        self.n_lanes = max(1, n_lanes)
        self.lanes = [torch.cuda.Stream(device=self.device) for _ in range(self.n_lanes)] if self.n_lanes > 1 else []
        n_ws = max(1, self.n_lanes)
        self.ws_score = [self._ws(xkv.workspace_bytes(xkv.OP_SCORE, self.dims, self.max_seqlen, self.T))
                         for _ in range(n_ws)]
        self.ws_select = [self._ws(xkv.workspace_bytes(xkv.OP_SELECT_COMPACT, self.dims, self.max_seqlen, self.T))
                          for _ in range(n_ws)]
        self._lanes_busy = False
        self.ws_prefill = None

        # ragged paged cache: a pool large enough for any split of the global budget
        per_layer_cap = min(max_budget if max_budget else self.max_prefix, self.max_prefix)
        self.max_cache_len = per_layer_cap + window + max_new_tokens
        self.max_pages_per_seq = max(1, math.ceil(self.max_cache_len / page_size))
        n_units = self.n_solver_units
        if total_budget is None:
            total_budget = n_units * per_layer_cap
        total_budget = min(total_budget, n_units * per_layer_cap)
        # caches per layer and the KV heads one page holds: B caches of Hkv heads, or B*Hkv caches of one head
        self.n_caches = self.B * (n_kv_heads if self.head_level else 1)
        page_heads = 1 if self.head_level else n_kv_heads
        n_pages = 0
        for P, t in zip(self.prefix, lengths):
            rows = min(total_budget, n_units * P) + n_units * (min(window, t) + max_new_tokens + page_size)
            n_pages += math.ceil(rows / page_size)
        self.n_pages = max(n_pages, 1)
        bf16 = dict(dtype=torch.bfloat16, device=self.device)
        page_dtype = torch.uint8 if kv_format == xkv.KV_INT8 else torch.bfloat16
        self.k_pages = torch.zeros(self.n_pages, page_heads, page_size, head_dim, dtype=page_dtype, device=self.device)
        self.v_pages = torch.zeros(self.n_pages, page_heads, page_size, head_dim, dtype=page_dtype, device=self.device)
        self.k_scales = self.v_scales = None
        if kv_format == xkv.KV_INT8:
            self.k_scales = torch.zeros(self.n_pages, page_heads, page_size, **f32)
            self.v_scales = torch.zeros(self.n_pages, page_heads, page_size, **f32)
        self.block_table = torch.zeros(n_layers, self.n_caches, self.max_pages_per_seq, dtype=torch.int32,
                                       device=self.device)
        # page runs of every (layer, cache): [0] first page, [1] number of pages; expanded on the device
        self.page_runs_host = [torch.zeros(n_layers, self.n_caches, dtype=torch.int32, pin_memory=True)
                               for _ in range(2)]
        self.page_runs = [torch.zeros(n_layers, self.n_caches, dtype=torch.int32, device=self.device)
                          for _ in range(2)]
        self.seq_lens = torch.zeros(n_layers, self.n_caches, dtype=torch.int32, device=self.device)
        self.cache = xkv.Cache(self.k_pages.data_ptr(), self.v_pages.data_ptr(), self.block_table.data_ptr(),
                               self.seq_lens.data_ptr(), n_layers, page_size, self.max_pages_per_seq,
                               self.n_pages, None if self.k_scales is None else self.k_scales.data_ptr(),
                               None if self.v_scales is None else self.v_scales.data_ptr(), kv_format, 0)
        # decode sees the head-level caches as B*Hkv sequences of one KV head with G query heads each
        self.dec_dims = self.dims if not self.head_level else xkv.Dims(
            self.n_caches, self.G, 1, head_dim, window, pool_kernel, pool_mode, scale, head_dim, head_dim)
        self.chunk_rows = decode_chunk_rows
        self.ws_decode = self._ws(xkv.workspace_bytes(xkv.OP_DECODE_ATTN, self.dec_dims, n_layers=n_layers,
                                                      max_cache_len=self.max_pages_per_seq * page_size,
                                                      chunk_rows=decode_chunk_rows))
        self.out = torch.empty(n_layers, self.B, n_q_heads, head_dim, **bf16)
        self.lse = torch.empty(n_layers, self.B, n_q_heads, **f32)
        self.budgets: np.ndarray | None = None
        self.last_solver_ms: float | None = None      # host time of the last xkv_alloc_budgets call
        self.r_avg: float | None = None

    def _ws(self, nbytes: int) -> torch.Tensor:
        return torch.zeros(nbytes, dtype=torch.uint8, device=self.device)   # status word reads OK before first use

    # ------------------------------------------------------------------ prefill
    def _lane(self, layer: int, *tensors):
        """(stream, workspace index) of a layer; the side stream first waits for what the caller's stream holds,
        and the caller's tensors are marked as in use on it (they may be temporaries)."""
        if not self.lanes:
            return torch.cuda.current_stream(), 0
        i = layer % self.n_lanes
        self.lanes[i].wait_stream(torch.cuda.current_stream())
        for t in tensors:
            if isinstance(t, torch.Tensor) and t.is_cuda:
                t.record_stream(self.lanes[i])
        self._lanes_busy = True
        return self.lanes[i], i

    def join(self) -> None:
        """The caller's stream waits for the layers queued on the side streams."""
        if self._lanes_busy:
            cur = torch.cuda.current_stream()
            for s in self.lanes:
                cur.wait_stream(s)
            self._lanes_busy = False

    def score_layer(self, layer: int, q_win: torch.Tensor, k: torch.Tensor, want_curves: bool = True,
                    mass: torch.Tensor | None = None, lse: torch.Tensor | None = None) -> None:
        """lse: fp32 [Hq, T] row normalisers of the layer's prefill attention (prefill_attention's second result);
        with them the scores take one pass over the keys instead of two."""
        stream, i = self._lane(layer, q_win, k, mass, lse)
        srt = self.sorted[layer] if want_curves else None
        gains = self.gains[layer] if want_curves else None
        if lse is None:
            xkv.score(self.dims, q_win, k, self.cu, self.T, self.max_seqlen, self.scores[layer], srt, gains, mass,
                      self.curve_len, self.ws_score[i], stream=stream)
        else:
            xkv.score_lse(self.dims, q_win, k, self.cu, self.T, self.max_seqlen, lse, self.scores[layer], srt, gains,
                          mass, self.curve_len, self.ws_score[i], stream=stream)
        if self.head_level and want_curves:
            xkv.head_curves(self.dims, self.scores[layer], self.sorted[layer], self.cu, self.T, self.max_seqlen,
                            self.head_gains[layer], self.curve_len, stream=stream)

    def score_layers(self, q_win: list[torch.Tensor], k: list[torch.Tensor],
                     lse: list[torch.Tensor] | None = None) -> None:
        """score_layer for every layer, with one fork and one join of the side streams for the whole phase (the
        inputs of all layers must be ready on the caller's stream at the call)."""
        cur = torch.cuda.current_stream()
        streams = self.lanes if self.lanes else [cur]
        for s in self.lanes:
            s.wait_stream(cur)
        lib, dims, cu = xkv.lib(), ctypes.byref(self.dims), self.cu.data_ptr()
        esz = self._layer_stride * 4
        gsz = self.gains[0].numel() * 4
        for l in range(self.L):
            i = l % len(streams)
            ws = self.ws_score[i]
            if lse is None:
                st = lib.xkv_score(dims, q_win[l].data_ptr(), k[l].data_ptr(), cu, self.T, self.max_seqlen,
                                   self.scores.data_ptr() + l * esz, self.sorted.data_ptr() + l * esz,
                                   self.gains.data_ptr() + l * gsz, None, self.curve_len, ws.data_ptr(), ws.numel(),
                                   streams[i].cuda_stream)
            else:
                st = lib.xkv_score_lse(dims, q_win[l].data_ptr(), k[l].data_ptr(), cu, self.T, self.max_seqlen,
                                       lse[l].data_ptr(), self.scores.data_ptr() + l * esz,
                                       self.sorted.data_ptr() + l * esz, self.gains.data_ptr() + l * gsz, None,
                                       self.curve_len, ws.data_ptr(), ws.numel(), streams[i].cuda_stream)
            if st < 0:
                raise xkv.XkvError(st, "xkv_score")
            if self.head_level:
                xkv.head_curves(self.dims, self.scores[l], self.sorted[l], self.cu, self.T, self.max_seqlen,
                                self.head_gains[l], self.curve_len, stream=streams[i])
        self._lanes_busy = bool(self.lanes)
        self.join()

    def prefill_attention(self, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, out: torch.Tensor | None = None,
                          lse: torch.Tensor | None = None):
        """Causal attention of one layer's prompt: q [T, Hq, d], k/v [T, Hkv, d] -> (out [T, Hq, d] bf16,
        lse [Hq, T] fp32).  The lse goes to score_layer(..., lse=) of that layer."""
        if out is None:
            out = torch.empty_like(q)
        if lse is None:
            lse = torch.empty(self.Hq, self.T, dtype=torch.float32, device=self.device)
        if self.ws_prefill is None:
            self.ws_prefill = self._ws(xkv.workspace_bytes(xkv.OP_PREFILL_ATTN, self.dims))
        xkv.prefill_attn(self.dims, q, k, v, self.cu, self.T, self.max_seqlen, out, lse, self.ws_prefill)
        return out, lse

    def select_layers(self, budgets, k: list[torch.Tensor], v: list[torch.Tensor]) -> None:
        """select_layer for every layer under one budget per layer ([L]), or per (layer, KV head) ([L, Hkv]) with
        head-level budgets; forked and joined once like score_layers."""
        cur = torch.cuda.current_stream()
        streams = self.lanes if self.lanes else [cur]
        for s in self.lanes:
            s.wait_stream(cur)
        lib, dims, cu, cache = xkv.lib(), ctypes.byref(self.dims), self.cu.data_ptr(), ctypes.byref(self.cache)
        esz = self._layer_stride * 4
        if self.head_level:
            # the same count for every sequence: [L, Hkv] -> [L, B, Hkv]; kept alive until the streams are joined
            b32 = np.ascontiguousarray(np.broadcast_to(np.asarray(budgets, dtype=np.int32).reshape(self.L, 1, self.Hkv),
                                                       (self.L, self.B, self.Hkv)))
            mode, step = xkv.BUDGET_PER_HEAD, 4 * self.B * self.Hkv
        else:
            b32 = np.ascontiguousarray(budgets, dtype=np.int32)
            mode, step = xkv.BUDGET_PER_LAYER, 4
        self._budget_keepalive = b32
        for l in range(self.L):
            i = l % len(streams)
            ws = self.ws_select[i]
            st = lib.xkv_select_compact(dims, l, b32.ctypes.data + step * l, mode, self.scores.data_ptr() + l * esz,
                                        self.sorted.data_ptr() + l * esz, k[l].data_ptr(), v[l].data_ptr(), cu,
                                        self.T, self.max_seqlen, cache, None, 0, ws.data_ptr(), ws.numel(),
                                        streams[i].cuda_stream)
            if st < 0:
                raise xkv.XkvError(st, "xkv_select_compact")
        self._lanes_busy = bool(self.lanes)
        self.join()

    def solve_budgets(self, total: int | None = None, r_target: float = 0.0, n_min: int = 0, n_max: int = 0,
                      per_sequence: bool = False, head_shards: int = 1, exchange=None):
        """Curves device -> host (the one crossing of the prefill), then Algorithm 1 on the host.  For one list per
        batch the curves are averaged over the sequences on the device first, so L x curve_len numbers cross.

        head_shards > 1: this session holds one of that many equal shares of the model's KV heads (one rank of a
        KV-head-sharded run).  The layers' curves are then combined over the shards before the solver -- summed
        (every shard contributes its heads' share of the layer mean), or with head-level budgets gathered, since
        each (layer, KV head) unit lives on one shard -- and every shard solves the same problem; `total` counts
        the whole model.  exchange(tensor) -> tensor does the combining: by default the torch.distributed
        collectives of `replicas`; a test on one GPU passes a function that stands in for the other shards.
        Returns this shard's budgets ([L], or [L, Hkv_local] with head-level budgets)."""
        self.join()
        if per_sequence and (self.head_level or head_shards > 1):
            raise ValueError("per-sequence lists are not combined with head-level budgets or head shards here")
        if per_sequence:
            if self.gains_host is None:
                self.gains_host = torch.empty(self.L, self.B, self.curve_len, dtype=torch.float32, pin_memory=True)
            self.gains_host.copy_(self.gains, non_blocking=True)
            torch.cuda.current_stream().synchronize()
            gains, prefix = self.gains_host.numpy(), np.asarray(self.prefix, dtype=np.int32)
        else:
            from . import replicas
            src = self.head_gains if self.head_level else self.gains        # [units, B, curve_len] either way
            # layer curves: a shard's mean over its heads is 1/head_shards of the layer's mean over all heads
            divisor = self.B * (1 if self.head_level else head_shards)
            xkv.batch_curves(src, self.n_solver_units, self.B, self.curve_len, divisor, self.layer_gains)
            curves = self.layer_gains
            if head_shards > 1:
                if self.head_level:
                    local = curves.view(self.L, self.Hkv, self.curve_len)
                    curves = (exchange or replicas.gather_unit_curves)(local).reshape(-1, self.curve_len)
                else:
                    curves = (exchange or replicas.sum_curves_over_ranks)(curves)
            n_units = curves.shape[0]
            if n_units == self.n_solver_units:
                self.layer_gains_host.copy_(curves, non_blocking=True)
                host = self.layer_gains_host
            else:
                host = torch.empty(n_units, self.curve_len, dtype=torch.float32, pin_memory=True)
                host.copy_(curves, non_blocking=True)
            torch.cuda.current_stream().synchronize()
            gains = host.numpy().reshape(n_units, 1, self.curve_len)
            prefix = np.asarray([self.max_prefix], dtype=np.int32)
        t0 = time.perf_counter()
        budgets, r_avg = xkv.alloc_budgets(gains, prefix, per_sequence=per_sequence,
                                           total=-1 if total is None else total,
                                           r_target=r_target, n_min=n_min, n_max=n_max)
        self.last_solver_ms = 1e3 * (time.perf_counter() - t0)
        if self.head_level:
            budgets = budgets.reshape(self.L, -1)                # one count per (layer, KV head of the whole model)
            if head_shards > 1:
                from . import replicas
                rank = replicas.env_ranks()[0] if exchange is None else getattr(exchange, "rank", 0)
                budgets = np.ascontiguousarray(budgets[:, rank * self.Hkv: (rank + 1) * self.Hkv])
        self.budgets, self.r_avg = budgets, r_avg
        return budgets, r_avg

    def assign_pages(self, budgets) -> None:
        """Hand consecutive pool pages to every (layer, sequence) for its kept rows plus new tokens: the runs are
        computed here (2 x L x B integers), the page table is expanded from them on the device."""
        budgets = np.asarray(budgets)
        prefix = np.asarray(self.prefix)[None, :]
        window = np.minimum(self.W, np.asarray(self.lengths))[None, :]
        if self.head_level:                                  # budgets [L, Hkv] -> one cache per (layer, b, g)
            k_lb = np.broadcast_to(budgets.reshape(self.L, 1, self.Hkv), (self.L, self.B, self.Hkv))
            rows = (np.minimum(k_lb, prefix[:, :, None]) + window[:, :, None] + self.max_new).reshape(self.L, -1)
        else:
            k_lb = budgets.T if budgets.ndim == 2 else np.broadcast_to(budgets[:, None], (self.L, self.B))   # [L, B]
            rows = np.minimum(k_lb, prefix) + window + self.max_new
        n = np.minimum(-(-rows // self.page_size), self.max_pages_per_seq).astype(np.int64)               # pages
        start = np.concatenate([[0], np.cumsum(n.ravel())[:-1]]).reshape(self.L, self.n_caches)
        if int(start.ravel()[-1] + n.ravel()[-1]) > self.n_pages:
            raise RuntimeError("page pool too small for these budgets")
        for dst, host, src in zip(self.page_runs, self.page_runs_host, (start, n)):
            host.numpy()[:] = src
            dst.copy_(host, non_blocking=True)
        xkv.build_block_table(self.page_runs[0], self.page_runs[1], self.cache, self.n_caches)

    def select_layer(self, layer: int, budget, k: torch.Tensor, v: torch.Tensor, sel: torch.Tensor | None = None,
                     per_sequence: bool = False) -> None:
        """budget: one count, [B] with per_sequence, or [Hkv] / [B, Hkv] in a head-level session."""
        stream, i = self._lane(layer, k, v, sel)
        if self.head_level:
            budget = np.ascontiguousarray(np.broadcast_to(np.asarray(budget, dtype=np.int32), (self.B, self.Hkv)))
            per_sequence = xkv.BUDGET_PER_HEAD
        xkv.select_compact(self.dims, layer, budget, per_sequence, self.scores[layer], self.sorted[layer], k, v,
                           self.cu, self.T, self.max_seqlen, self.cache, sel,
                           0 if sel is None else sel.shape[-1], self.ws_select[i], stream=stream)

    def prefill(self, q_win: list[torch.Tensor], k: list[torch.Tensor], v: list[torch.Tensor],
                budgets=None, total: int | None = None, n_min: int = 0, n_max: int = 0):
        """Score every layer, split the budget (unless given), evict and compact every layer."""
        self.score_layers(q_win, k)
        if budgets is None:
            budgets, _ = self.solve_budgets(total=total, n_min=n_min, n_max=n_max)
        else:
            self.budgets = np.asarray(budgets, dtype=np.int32)
        self.assign_pages(budgets)
        self.select_layers(budgets, k, v)
        return budgets

    # ------------------------------------------------------------------ generation
    def decode(self, q: torch.Tensor, k_new: torch.Tensor | None, v_new: torch.Tensor | None,
               out: torch.Tensor | None = None, lse: torch.Tensor | None = None, layer_begin: int = 0,
               layer_end: int | None = None, chunk_rows: int | None = None) -> torch.Tensor:
        self.join()
        out = self.out if out is None else out
        layer_end = self.L if layer_end is None else layer_end
        xkv.decode_attn(self.dec_dims, self.cache, layer_begin, layer_end, q, k_new, v_new, out,
                        self.lse if lse is None else lse,
                        self.chunk_rows if chunk_rows is None else chunk_rows, self.ws_decode)
        return out

    def device_status(self, which: str = "decode") -> int:
        """First error any call of that kind recorded since the last check (the status words are sticky and
        reading resets them), XKV_OK otherwise."""
        self.join()
        ws = {"decode": [self.ws_decode], "score": self.ws_score, "select": self.ws_select,
              "prefill": [] if self.ws_prefill is None else [self.ws_prefill]}[which]
        first = xkv.OK
        for w in ws:
            st = xkv.read_device_status(w)
            if st != xkv.OK and first == xkv.OK:
                first = st
        return first
