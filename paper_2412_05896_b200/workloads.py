"""Seeded synthetic workloads shaped like the paper's long-context Llama/Mistral inference tasks.

This module only draws random tensors; it holds none of the method's arithmetic and is the one
piece shared by the CUDA path's tests/benchmark and the CPU oracle's tests (both get the same
bf16 tensors).  It stands in for the LongBench prompts and Llama-3-8B-Instruct activations the
paper measures on (Sec. V-A), which are not available offline.

Per layer l (sub-stream seed = base*1000003 + l*101 + tensor id):
  * temperature tau_l, log-uniform in the config's interval (layers differ in how peaked their
    attention is, the cross-layer variation the paper calls DDID);
  * per (layer, KV head) a random unit direction u;
  * keys  k = z,  z ~ N(0,1)^d;  every prefix position is a heavy hitter with probability 0.02 per
    (sequence, KV head): k += 3u;  position 0 of every sequence is a sink: k = 4 (z + 3u);
  * window queries  q = (z + sqrt(d) u_group) / tau_l, so a heavy hitter's expected logit is
    3/tau_l and the sink's about 12/tau_l above the bulk;
  * values  v ~ N(0,1);
  * decode-step q / k_new / v_new ~ N(0,1);
all rounded to bf16 once.  Prompt lengths are fixed, or uniform integers in an interval.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    batch: int
    prompt: int | tuple[int, int]          # fixed length, or (lo, hi) inclusive
    window: int
    pool_kernel: int
    temperature: tuple[float, float]
    decode_steps: int
    seed: int
    budgets: tuple[int, ...] | None = None  # fixed per-layer budgets (prefix tokens per head)
    avg_budget: int | None = None           # else: global budget = n_layers * avg_budget via the solver
    n_min: int = 0
    n_max: int = 0                          # 0 = unbounded
    pool_mode: int = 0                      # 0 max, 1 avg

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads


_BASE = 20241205

CONFIGS: dict[str, Workload] = {
    # Tiny case the CPU oracle finishes in seconds.
    "tiny": Workload("tiny", 4, 4, 4, 64, 1, 512, 16, 5, (0.5, 2.0), 16, _BASE + 1,
                     budgets=(64, 128, 96, 32)),
    # Llama-2-7B-shaped MHA.
    "llama2_7b_mha": Workload("llama2_7b_mha", 32, 32, 32, 128, 8, 4096, 32, 7, (0.3, 3.0), 128,
                              _BASE + 2, avg_budget=512),
    # Mistral-7B-shaped GQA, long prompts.
    "mistral_7b_gqa": Workload("mistral_7b_gqa", 32, 32, 8, 128, 4, 32768, 64, 7, (0.3, 3.0), 256,
                               _BASE + 3, avg_budget=2048, n_min=128, n_max=8192),
    # Llama-3-8B-shaped GQA, large ragged batch.
    "llama3_8b_ragged": Workload("llama3_8b_ragged", 32, 32, 8, 128, 64, (2048, 8192), 32, 7,
                                 (0.3, 3.0), 512, _BASE + 4, avg_budget=1024),
    # Llama-3-8B-shaped GQA, one very long prompt.
    "llama3_8b_long": Workload("llama3_8b_long", 32, 32, 8, 128, 1, 131072, 64, 7, (0.3, 3.0), 256,
                               _BASE + 5, avg_budget=4096, n_min=256, n_max=16384),
}


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed % (2 ** 63 - 1))
    return g


def _sub_seed(base: int, layer: int, tensor_id: int) -> int:
    return base * 1000003 + layer * 101 + tensor_id


def prompt_lengths(w: Workload) -> list[int]:
    """Prompt length of every sequence (host ints)."""
    if isinstance(w.prompt, int):
        return [w.prompt] * w.batch
    lo, hi = w.prompt
    g = _gen(_sub_seed(w.seed, 0, 99), "cpu")
    return torch.randint(lo, hi + 1, (w.batch,), generator=g).tolist()


def cu_seqlens(lengths: list[int]) -> list[int]:
    out = [0]
    for t in lengths:
        out.append(out[-1] + t)
    return out


def temperature(w: Workload, layer: int) -> float:
    g = _gen(_sub_seed(w.seed, layer, 0), "cpu")
    lo, hi = w.temperature
    x = torch.rand((), generator=g).item()
    return math.exp(math.log(lo) + x * (math.log(hi) - math.log(lo)))


def layer_tensors(w: Workload, layer: int, device="cpu", lengths: list[int] | None = None,
                  stress: bool = False):
    """(q_win [B,Hq,W,d], k [T,Hkv,d], v [T,Hkv,d]) in bf16 for one layer.

    stress=True shifts the values by +1 (see decode_tensors).
    """
    if lengths is None:
        lengths = prompt_lengths(w)
    cu = cu_seqlens(lengths)
    T, d, Hkv, Hq, G, W = cu[-1], w.head_dim, w.n_kv_heads, w.n_q_heads, w.group, w.window
    tau = temperature(w, layer)

    g = _gen(_sub_seed(w.seed, layer, 1), device)
    u = torch.randn(Hkv, d, generator=g, device=device, dtype=torch.float32)
    u = u / u.norm(dim=-1, keepdim=True)

    g = _gen(_sub_seed(w.seed, layer, 2), device)
    k = torch.randn(T, Hkv, d, generator=g, device=device, dtype=torch.float32)
    g = _gen(_sub_seed(w.seed, layer, 3), device)
    heavy = torch.rand(T, Hkv, generator=g, device=device) < 0.02
    starts = torch.tensor(cu[:-1], device=device, dtype=torch.long)
    for b, t in enumerate(lengths):          # window positions are never heavy hitters
        heavy[cu[b] + max(t - W, 0): cu[b + 1]] = False
    heavy[starts] = False
    k = k + 3.0 * heavy.unsqueeze(-1).to(torch.float32) * u.unsqueeze(0)
    k[starts] = 4.0 * (k[starts] + 3.0 * u.unsqueeze(0))

    g = _gen(_sub_seed(w.seed, layer, 4), device)
    q = torch.randn(w.batch, Hq, W, d, generator=g, device=device, dtype=torch.float32)
    u_group = u.repeat_interleave(G, dim=0)                    # [Hq, d]
    q = (q + math.sqrt(d) * u_group.view(1, Hq, 1, d)) / tau

    g = _gen(_sub_seed(w.seed, layer, 5), device)
    v = torch.randn(T, Hkv, d, generator=g, device=device, dtype=torch.float32)
    if stress:
        v = v + 1.0
    return q.to(torch.bfloat16), k.to(torch.bfloat16), v.to(torch.bfloat16)


def decode_tensors(w: Workload, step: int, device="cpu", layers: int | None = None,
                   stress: bool = False):
    """(q [L,B,Hq,d], k_new [L,B,Hkv,d], v_new [L,B,Hkv,d]) in bf16 for one generation step.

    stress=True makes the step numerically demanding for parity checks: queries scaled up so the
    attention is peaked, and values shifted by +1 so outputs are O(1) instead of near zero.
    """
    L = w.n_layers if layers is None else layers
    d = w.head_dim
    g = _gen(_sub_seed(w.seed, 7000 + step, 6), device)
    q = torch.randn(L, w.batch, w.n_q_heads, d, generator=g, device=device, dtype=torch.float32)
    k = torch.randn(L, w.batch, w.n_kv_heads, d, generator=g, device=device, dtype=torch.float32)
    v = torch.randn(L, w.batch, w.n_kv_heads, d, generator=g, device=device, dtype=torch.float32)
    if stress:
        q = q * 4.0
        v = v + 1.0
    return q.to(torch.bfloat16), k.to(torch.bfloat16), v.to(torch.bfloat16)
