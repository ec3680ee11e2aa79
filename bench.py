#!/usr/bin/env python
"""Benchmark of the XKV hot path on B200.

One "step" is one pass of the whole path over one batch of a seeded synthetic workload: score
every layer, split the global budget across layers on the host, evict/compact every layer into the
ragged paged cache, then run the workload's decode steps (append + attention over all layers).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--table a,b,c|none]
                    [--impl xkv|reference]

Prints one JSON line.  The headline workload (default: the largest single-GPU one) is timed with
K steps after W warm-up steps; `value` is its decode-attention throughput over the retained cache
(bytes of retained K and V read per decode step / decode time), device-resident inputs; `e2e` is
the same with host inputs and outputs; `roofline` is the attention kernel alone against the
measured HBM bandwidth; `cpu_baseline` is the fp64 oracle timed on the host cores; `parity`
compares the CUDA path with that oracle on a stated sample, outside the timed region.  `workloads`
holds the same measurements (a few steps each) for the other workloads.
With N > 1 (launched by torch.distributed.run) every rank runs its own batch: no data-path
collective, weak scaling.
"""
from __future__ import annotations

import argparse
import gc
import json
import os
import subprocess
import sys
import threading
import time
from dataclasses import replace

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

DEFAULT_WORKLOAD = "llama3_8b_ragged"
TABLE = ("llama2_7b_mha", "mistral_7b_gqa", "llama3_8b_ragged", "llama3_8b_long")
METRIC = "ragged-KV decode-attn GB/s"
DEC_DISTINCT = 64          # distinct sets of decode-step inputs held in memory; later steps reuse them in turn

# (dram__bytes_read.sum + dram__bytes_write.sum) / algorithmic bytes of one decode_attn_kernel launch, taken from
# an ncu capture of a smaller case of the same kernel; traffic grows in proportion to the retained rows, so a full
# launch's traffic is this ratio times its algorithmic bytes.  None whenever the kernel has changed since the capture.
NCU_TRAFFIC_RATIO = 1.033


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json)"
    except Exception:
        return 6650.0, "fallback (earlier measurement on this pool)"


def measured_tflops():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            j = json.load(f)
        return float(j["bf16_tflops"]), float(j["bf16_tflops_sustained"]), "measured (MEASURED_PEAKS.json)"
    except Exception:
        return 1590.0, 1400.0, "fallback (earlier measurement on this pool)"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], {}
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons[name] = reasons.get(name, 0) + 1
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons), "reason_samples": reasons}


# ----------------------------------------------------------------------------------------------
# Oracle leg (CPU baseline, parity sample and --impl reference)
# ----------------------------------------------------------------------------------------------
def oracle_sample(w, tensors_cpu, t0: int, budget: int, seconds: float, dec_cpu, keep_outputs: int = 0):
    """Runs the oracle, as it stands, on one (layer, sequence) with every KV head: scoring, top-k, compaction,
    then decode steps over its own compacted cache; decode passes repeat until `seconds` have elapsed.

    tensors_cpu: (q_win [1,Hq,W,d], k [t0,Hkv,d], v [t0,Hkv,d]) bf16 on the CPU; dec_cpu: list of per-step
    (q [Hq,d], k_new [Hkv,d], v_new [Hkv,d]).  Returns a dict with the timings and, for the first `keep_outputs`
    decode steps, the oracle's attention outputs.
    """
    import numpy as np
    from oracle import xkv_oracle as O

    def f64(t):
        return t.float().numpy().astype(np.float64)

    q_win, k, v = tensors_cpu
    qf, kf, vf = f64(q_win[0:1]), f64(k[:t0]), f64(v[:t0])
    cu = np.array([0, t0])
    wall0, cpu0 = time.perf_counter(), time.process_time()
    t_score = time.perf_counter()
    w_units = O.score_layer(qf, kf, cu, w.window, w.pool_kernel, "max" if w.pool_mode == 0 else "avg")
    score_s = time.perf_counter() - t_score
    caches, kept = {}, {}
    t_evict = time.perf_counter()
    for g in range(w.n_kv_heads):
        kept[g] = O.kept_positions(w_units[(0, g)], budget, t0, w.window)
        caches[g] = (O.evict_by_index(kf[:, g], kept[g]), O.evict_by_index(vf[:, g], kept[g]))
    evict_s = time.perf_counter() - t_evict
    G, d = w.group, w.head_dim
    bytes_read, dec_s, step = 0, 0.0, 0
    outputs = []
    deadline = time.perf_counter() + seconds
    while True:
        qd, knd, vnd = (f64(x) for x in dec_cpu[step % len(dec_cpu)])
        t1 = time.perf_counter()
        z_step = np.zeros((w.n_q_heads, d))
        for g in range(w.n_kv_heads):
            Kc = np.concatenate([caches[g][0], knd[g][None]], 0)
            Vc = np.concatenate([caches[g][1], vnd[g][None]], 0)
            caches[g] = (Kc, Vc)
            for h in range(g * G, (g + 1) * G):
                z_step[h], _ = O.decode_attention(qd[h], Kc, Vc)
            bytes_read += Kc.shape[0] * 2 * d * 2          # the bf16 bytes this KV head's step stands for
        dec_s += time.perf_counter() - t1
        if step < keep_outputs:
            outputs.append(z_step)
        step += 1
        if time.perf_counter() > deadline and step >= max(4, keep_outputs):
            break
    wall, cpu = time.perf_counter() - wall0, time.process_time() - cpu0
    return {"bytes": bytes_read, "decode_s": dec_s, "score_s": score_s, "evict_s": evict_s, "steps": step,
            "cores": max(1, round(cpu / max(wall, 1e-9))), "w_units": w_units, "kept": kept, "outputs": outputs}


def run_reference(args):
    """--impl reference: the oracle timed on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from paper_2412_05896_b200 import workloads as WL
    w = WL.CONFIGS[args.workload]
    lengths = WL.prompt_lengths(w)
    one_seq = replace(w, batch=1, prompt=lengths[0])
    tensors = WL.layer_tensors(one_seq, 0, "cpu", [lengths[0]])
    budget = w.avg_budget if w.budgets is None else w.budgets[0]
    dec_cpu = []
    for s in range(8):
        q, kn, vn = WL.decode_tensors(one_seq, s, "cpu", layers=1)
        dec_cpu.append((q[0, 0], kn[0, 0], vn[0, 0]))
    per_step_s = max(2.0, min(20.0, 60.0 / max(args.steps + args.warmup, 1)))
    vals, cores, samples = [], 1, 0
    t_all = time.perf_counter()
    for i in range(args.warmup + args.steps):
        r = oracle_sample(w, tensors, lengths[0], budget, per_step_s, dec_cpu)
        cores = r["cores"]
        if i >= args.warmup:
            vals.append((r["bytes"], r["decode_s"]))
            samples = r["steps"]
    total_b = sum(b for b, _ in vals)
    total_s = sum(s for _, s in vals)
    value = total_b / total_s / 1e9
    sample = (f"layer 0, sequence 0, all {w.n_kv_heads} KV heads: oracle scoring + top-k + compaction, then "
              f"{samples} decode steps per bench step (~{per_step_s:.0f} s)")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": 1e3 * (time.perf_counter() - t_all) / max(args.steps + args.warmup, 1),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": w.name, "sample": sample},
            "cpu_baseline": {"value": value, "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------------
# The CUDA path: one workload
# ----------------------------------------------------------------------------------------------
class Ctx:
    """What every workload run needs: the rank layout, the device and the imported modules."""

    def __init__(self, args):
        import numpy as np
        import torch
        import torch.distributed as dist

        from paper_2412_05896_b200 import build as _build
        from paper_2412_05896_b200 import replicas
        from paper_2412_05896_b200 import workloads as WL
        from paper_2412_05896_b200 import xkv
        from paper_2412_05896_b200.pipeline import XkvSession
        self.np, self.torch, self.dist, self.replicas, self.WL, self.xkv, self.XkvSession = \
            np, torch, dist, replicas, WL, xkv, XkvSession
        self.args = args
        self.rank, self.world, self.local = replicas.env_ranks()
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device: the XKV path has no CPU fallback")
        torch.cuda.set_device(self.local)
        self.dev = f"cuda:{self.local}"
        replicas.init("nccl", torch.device(self.dev))
        if self.rank == 0:
            _build.build()
        replicas.barrier()
        xkv.lib()
        self.peak, self.peak_src = measured_peak()
        self.tf_burst, self.tf_sustained, self.tf_src = measured_tflops()
        self.sms = torch.cuda.get_device_properties(self.local).multi_processor_count

    def sync_all(self):
        self.torch.cuda.synchronize()
        if self.world > 1:
            self.dist.barrier()
            self.torch.cuda.synchronize()

    def max_over_ranks(self, x: float) -> float:
        return self.replicas.max_over_ranks(x, self.dev)

    def sum_over_ranks(self, x: float) -> float:
        return self.replicas.sum_over_ranks(x, self.dev)


def run_workload(ctx: Ctx, name: str, steps: int, warmup: int, headline: bool) -> dict:
    np, torch, xkv, WL, args = ctx.np, ctx.torch, ctx.xkv, ctx.WL, ctx.args
    dev, rank, world = ctx.dev, ctx.rank, ctx.world
    w0 = WL.CONFIGS[name]
    if args.decode_steps:
        w0 = replace(w0, decode_steps=args.decode_steps)
    if args.layers:
        w0 = replace(w0, n_layers=args.layers)
    w = ctx.replicas.replica_workload(w0, rank)              # every rank draws its own batch
    L, B, Hkv, d, W = w.n_layers, w.batch, w.n_kv_heads, w.head_dim, w.window
    M = w.group * W
    lengths = WL.prompt_lengths(w)
    n_dec = w.decode_steps
    n_distinct = min(n_dec, DEC_DISTINCT)
    tens = [WL.layer_tensors(w, l, dev, lengths) for l in range(L)]
    q_win = [t[0] for t in tens]
    k = [t[1] for t in tens]
    v = [t[2] for t in tens]
    dec = [WL.decode_tensors(w, s, dev) for s in range(n_distinct)]
    N_total = None if w.budgets is not None else L * w.avg_budget
    sess = ctx.XkvSession(L, w.n_q_heads, Hkv, d, W, w.pool_kernel, lengths, pool_mode=w.pool_mode,
                          max_new_tokens=n_dec, max_budget=w.n_max or None, total_budget=N_total,
                          curve_len=w.n_max or None, device=dev, decode_chunk_rows=args.chunk_rows,
                          **({} if args.lanes is None else {"n_lanes": args.lanes}))
    prefix = sess.prefix

    ev = lambda: torch.cuda.Event(enable_timing=True)
    k_start = [ev() for _ in range(n_dec)]
    k_stop = [ev() for _ in range(n_dec)]
    for e in k_start + k_stop:
        e.record()

    def decode_bytes(budgets) -> list[int]:
        """Retained K and V bytes one decode step reads, per decode step (the cache grows by one row)."""
        base = sum(min(int(budgets[l]), P) + min(W, t) for l in range(L) for P, t in zip(prefix, lengths))
        return [(base + (s + 1) * L * B) * Hkv * 2 * d * 2 for s in range(n_dec)]

    def prefill_bytes(budgets) -> int:
        """Algorithmic bytes of score + select + compact: K once, score out, kept rows in and out."""
        tot = 0
        for l in range(L):
            for P, t in zip(prefix, lengths):
                kept = min(int(budgets[l]), P) + min(W, t)
                tot += Hkv * (t * (2 * d + 8) + kept * (8 * d + 4))
        return tot

    def prefill(host_upload=None):
        e = [ev() for _ in range(4)]
        e[0].record()
        if host_upload is not None:
            host_upload()
        sess.score_layers(q_win, k)
        e[1].record()
        if w.budgets is not None:
            budgets = np.asarray(w.budgets, dtype=np.int32)
        else:
            budgets, _ = sess.solve_budgets(total=N_total, n_min=w.n_min, n_max=w.n_max)
        sess.assign_pages(budgets)
        e[2].record()
        sess.select_layers(budgets, k, v)
        e[3].record()
        return e, budgets

    def step(kernel_events=False):
        """One pass of the whole path, inputs resident on the device."""
        e, budgets = prefill()
        for s in range(n_dec):
            q, kn, vn = dec[s % n_distinct]
            if kernel_events:
                xkv.profile_events(k_start[s], k_stop[s])
            sess.decode(q, kn, vn)
        e.append(ev())
        e[4].record()
        xkv.profile_events(None, None)
        return e, budgets

    def check_status(where: str):
        for which in ("score", "select", "decode"):
            st = sess.device_status(which)
            if st != xkv.OK:
                raise SystemExit(f"{name}: device status of {which} after {where}: {xkv.status_string(st)}")

    for _ in range(warmup):
        step()
    ctx.sync_all()
    check_status("warm-up")

    sampler = ClockSampler(ctx.local)
    if rank == 0:
        sampler.start()
    launches0 = xkv.launch_count()
    first, last = ev(), ev()
    ctx.sync_all()
    first.record()
    recs = []
    for _ in range(steps):
        recs.append(step(kernel_events=True))
        torch.cuda.current_stream().synchronize()    # kernel events of this step are read below
        recs[-1] = recs[-1] + ([a.elapsed_time(b) for a, b in zip(k_start, k_stop)],)
    last.record()
    ctx.sync_all()
    launches = xkv.launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    check_status("the timed steps")

    budgets = recs[-1][1]
    dbytes = decode_bytes(budgets)
    phase = np.array([[e[i].elapsed_time(e[i + 1]) for i in range(4)] for e, _, _ in recs])   # ms
    step_ms = np.array([e[0].elapsed_time(e[4]) for e, _, _ in recs])
    dec_ms_total = float(phase[:, 3].sum())
    region_ms = first.elapsed_time(last)
    kern_ms = np.array([r[2] for r in recs])                       # [steps, n_dec]

    rate, dec_ms_max, _ = ctx.replicas.whole_job_rate(float(sum(dbytes)) * steps, dec_ms_total, dev)
    region_ms_max = ctx.max_over_ranks(region_ms)
    value = rate / 1e9
    tokens_per_s = world * B * n_dec * steps / (dec_ms_max * 1e-3)

    peak = ctx.peak
    kern_avg_ms = float(kern_ms.mean())
    launch_bytes = float(np.mean(dbytes))
    achieved = launch_bytes / (kern_avg_ms * 1e-3) / 1e9
    roofline = {"kernel": "decode_attn_kernel", "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "frac_of_nominal_8000": achieved / 8000.0, "peak_source": ctx.peak_src,
                "bytes_per_launch": launch_bytes, "avg_launch_ms": kern_avg_ms,
                "traffic": None if NCU_TRAFFIC_RATIO is None else NCU_TRAFFIC_RATIO * launch_bytes,
                "traffic_source": "ncu capture of a smaller case of the same kernel, scaled by the retained rows"
                                  if NCU_TRAFFIC_RATIO is not None else "none since the kernel last changed"}
    pre_bytes = prefill_bytes(budgets)
    score_evict_ms = float((phase[:, 0] + phase[:, 2]).mean() / L)
    se_gbps = pre_bytes / L / (score_evict_ms * 1e-3) / 1e9
    rec = {
        "workload": w.name, "steps": steps, "warmup": warmup, "decode_steps": n_dec,
        "value": value, "unit": "GB/s",
        "pct_of_hbm_peak": {"measured": 100.0 * value / world / peak, "nominal_8000": 100.0 * value / world / 8000.0},
        "decode_tokens_per_s": tokens_per_s, "ms_per_step": float(step_ms.mean()),
        "roofline": roofline,
        "score_evict_ms_per_layer": score_evict_ms,
        "score_evict_roofline": {"bound": "hbm", "algorithmic_bytes_per_layer": pre_bytes / L, "achieved_GBps": se_gbps,
                                 "frac_of_measured": se_gbps / peak, "frac_of_nominal_8000": se_gbps / 8000.0},
        "phases_ms": {"score": float(phase[:, 0].mean()), "solver_and_page_table": float(phase[:, 1].mean()),
                      "select_compact": float(phase[:, 2].mean()), "decode": float(phase[:, 3].mean())},
        "solver_host_ms": sess.last_solver_ms,
        "budgets": {"min": int(min(budgets)), "max": int(max(budgets)), "sum": int(sum(int(x) for x in budgets)),
                    "r_avg": sess.r_avg},
        "query_rows_per_kv_head": M,
        "timed_region_ms": region_ms_max, "gpu_launches": int(launches), "clocks": clocks,
    }
    if M >= 128:
        # Scoring forms G*W logits per key in each of its two passes and every one of them goes through an
        # exponential: on this part that pipe (16 results per clock per SM) is slower than HBM for such shapes.
        n_exp = sum(Hkv * M * (t + P) for P, t in zip(prefix, lengths))
        mhz = (clocks or {}).get("sm_mhz") or 1965.0
        xu_peak = 16.0 * ctx.sms * mhz * 1e6
        score_ms = float(phase[:, 0].mean() / L)
        rec["score_xu_roofline"] = {
            "bound": "xu", "unit": "Gexp/s", "exponentials_per_layer": n_exp, "peak": xu_peak / 1e9,
            "peak_derivation": f"16 ex2 per clock per SM x {ctx.sms} SMs x {mhz:.0f} MHz (median SM clock sampled)",
            "achieved": n_exp / (score_ms * 1e-3) / 1e9, "frac": n_exp / (score_ms * 1e-3) / xu_peak,
            "score_ms_per_layer": score_ms,
            "note": "time is the whole scoring phase per layer (logit passes, pooling, sort, curves)"}

    # ---------------------------------------------------------------- prefill attention and scoring from its normalisers
    # The step before the path (Alg. 2 step 1 takes W_attn from the layer's own attention): causal attention of every
    # layer's prompt, timed per layer, whose row normalisers then let the scoring read the keys once.  Outside the
    # timed region of the headline number; the queries are random with the window queries in their last rows.
    if world == 1 and not args.no_prefill_attn:
        T, Hq = sess.T, w.n_q_heads
        lse_all = torch.empty(L, Hq, T, dtype=torch.float32, device=dev)
        q_full = torch.empty(T, Hq, d, dtype=torch.bfloat16, device=dev)
        o_full = torch.empty_like(q_full)
        gen = torch.Generator(device=dev)
        pf = [(ev(), ev()) for _ in range(L)]
        for l in range(L):
            gen.manual_seed(w.seed * 7919 + l)
            q_full.normal_(generator=gen)
            for b, t in enumerate(lengths):
                n = min(W, t)
                lo = int(sess.cu_host[b])
                q_full[lo + t - n: lo + t] = q_win[l][b, :, W - n:].transpose(0, 1)
            pf[l][0].record()
            sess.prefill_attention(q_full, k[l], v[l], out=o_full, lse=lse_all[l])
            pf[l][1].record()
        torch.cuda.synchronize()
        if sess.device_status("prefill") != xkv.OK:
            raise SystemExit(f"{name}: prefill attention reported a device error")
        pf_ms = np.array([a.elapsed_time(b) for a, b in pf])
        flops = 4.0 * d * Hq * sum(t * (t + 1) / 2 for t in lengths)
        tf = flops / (float(np.median(pf_ms)) * 1e-3) / 1e12
        rec["prefill_attn"] = {
            "kernel": "prefill_attn_kernel (tcgen05, causal, bf16 in, fp32 accumulate)", "layers_measured": L,
            "ms_per_layer_median": float(np.median(pf_ms)), "flops_per_layer": flops, "achieved_TFLOPs": tf,
            "frac_of_measured_bf16_burst": tf / ctx.tf_burst, "frac_of_measured_bf16_sustained": tf / ctx.tf_sustained,
            "peak_source": ctx.tf_src,
            "note": "4*d*Hq*sum_b t_b(t_b+1)/2 flops; outside the timed step (the model's own attention)"}
        lse_list = [lse_all[l] for l in range(L)]
        time.sleep(1.0)      # as below: the scoring of the timed steps did not follow a long tensor-core phase either
        reps = 6
        for _ in range(2):
            sess.score_layers(q_win, k, lse=lse_list)
        a, b_ = ev(), ev()
        a.record()
        for _ in range(reps):
            sess.score_layers(q_win, k, lse=lse_list)
        b_.record()
        torch.cuda.synchronize()
        check_status("scoring from the prefill normalisers")
        score_lse_ms = a.elapsed_time(b_) / reps
        se_lse = (score_lse_ms + float(phase[:, 2].mean())) / L
        se_lse_gbps = pre_bytes / L / (se_lse * 1e-3) / 1e9
        rec["score_from_prefill_lse"] = {
            "score_ms": score_lse_ms, "score_evict_ms_per_layer": se_lse,
            "score_evict_roofline": {"bound": "hbm", "algorithmic_bytes_per_layer": pre_bytes / L,
                                     "achieved_GBps": se_lse_gbps, "frac_of_measured": se_lse_gbps / peak,
                                     "frac_of_nominal_8000": se_lse_gbps / 8000.0},
            "note": "xkv_score_lse: the window rows' normalisers come from xkv_prefill_attn, so scoring is one pass "
                    "over the keys; select+compact time is that of the timed steps"}
        if M >= 128:
            n_exp1 = sum(Hkv * M * P for P in prefix)
            mhz = (clocks or {}).get("sm_mhz") or 1965.0
            rec["score_from_prefill_lse"]["xu_frac"] = n_exp1 / (score_lse_ms / L * 1e-3) / (16.0 * ctx.sms * mhz * 1e6)
        del lse_all, q_full, o_full, lse_list
        torch.cuda.empty_cache()

    # ---------------------------------------------------------------- decode over caches stored in 8 bits
    # The same budgets, the kept rows stored as 8-bit integers with a scale per row (Sec. II-B: quantisation is compatible
    # with eviction): the second bandwidth lever.  Outside the timed region of the headline number.
    if world == 1 and not args.no_q8:
        time.sleep(1.0)      # the prefill leg leaves the GPU at its power cap; compare with the timed steps' launches at like clocks
        q8 = ctx.XkvSession(L, w.n_q_heads, Hkv, d, W, w.pool_kernel, lengths, pool_mode=w.pool_mode,
                            max_new_tokens=n_dec, max_budget=w.n_max or None, total_budget=N_total,
                            curve_len=w.n_max or None, device=dev, decode_chunk_rows=args.chunk_rows,
                            kv_format=xkv.KV_INT8)
        q8.scores, q8.sorted = sess.scores, sess.sorted            # the scores of the last scoring pass
        q8._layer_stride = sess._layer_stride
        q8.assign_pages(budgets)
        q8.select_layers(budgets, k, v)
        n_q8 = min(n_dec, 48)
        qs = [ev() for _ in range(n_q8)]
        qe = [ev() for _ in range(n_q8)]
        for e in qs + qe:
            e.record()
        for s_ in range(n_q8):
            q, kn, vn = dec[s_ % n_distinct]
            xkv.profile_events(qs[s_], qe[s_])
            q8.decode(q, kn, vn)
        xkv.profile_events(None, None)
        torch.cuda.synchronize()
        for which in ("select", "decode"):
            if q8.device_status(which) != xkv.OK:
                raise SystemExit(f"{name}: 8-bit cache {which} reported a device error")
        q8_ms = float(np.mean([a.elapsed_time(b) for a, b in zip(qs, qe)][2:]))
        rows = float(np.mean(dbytes[2:n_q8])) / (2 * d * 2)           # cached rows (all layers, sequences, KV heads) per step
        q8_bytes = rows * (2 * d + 8)                                   # K and V bytes plus two fp32 scales per row
        bf16_ms = float(kern_ms[:, 2:n_q8].mean())
        rec["quantized_cache_decode"] = {
            "format": "8-bit integers with one fp32 scale per cached row, K and V",
            "steps_measured": n_q8 - 2, "avg_launch_ms": q8_ms, "stored_bytes_per_launch": q8_bytes,
            "achieved_GBps_of_stored_bytes": q8_bytes / (q8_ms * 1e-3) / 1e9,
            "frac_of_measured_hbm": q8_bytes / (q8_ms * 1e-3) / 1e9 / peak,
            "bf16_launch_ms_same_steps": bf16_ms, "speedup_over_bf16_cache": bf16_ms / q8_ms}
        del q8
        torch.cuda.empty_cache()

    # ---------------------------------------------------------------- full-cache decode, for comparison only
    if world == 1 and not args.no_full_cache and (headline or name == "llama3_8b_long" or args.full_cache_all):
        per_layer = sum(-(-(t + n_dec + sess.page_size) // sess.page_size) * sess.page_size for t in lengths) \
            * Hkv * d * 2 * 2                                            # K and V pages of one uncompressed layer
        free_b, _ = torch.cuda.mem_get_info(dev)
        n_full = int(min(L, (free_b - (6 << 30)) // max(per_layer, 1)))
        if n_full >= 1:
            full = ctx.XkvSession(n_full, w.n_q_heads, Hkv, d, W, w.pool_kernel, lengths, pool_mode=w.pool_mode,
                                  max_new_tokens=n_dec, device=dev)
            keep_all = np.full(n_full, max(full.prefix), dtype=np.int32)
            full.assign_pages(keep_all)
            for l in range(n_full):
                full.select_layer(l, int(keep_all[l]), k[l], v[l])      # budget = prefix length: nothing is evicted
            full.join()
            f0, f1 = ev(), ev()
            n_warm, n_timed = 2, min(6, n_dec - 2)
            for s in range(n_warm + n_timed):
                if s == n_warm:
                    f0.record()
                q, kn, vn = dec[s % n_distinct]
                full.decode(q[:n_full], kn[:n_full], vn[:n_full])
            f1.record()
            torch.cuda.synchronize()
            if full.device_status("decode") != xkv.OK:
                raise SystemExit("full-cache decode reported a device error")
            f_ms = f0.elapsed_time(f1) / n_timed
            f_bytes = sum(t + n_warm + (n_timed + 1) / 2 for t in lengths) * n_full * Hkv * 2 * d * 2
            comp_ms = float(phase[:, 3].mean()) / n_dec
            rec["full_cache_decode"] = {
                "layers_measured": n_full, "ms_per_decode_step_all_layers": f_ms * L / n_full,
                "GBps": f_bytes / (f_ms * 1e-3) / 1e9, "compressed_ms_per_decode_step": comp_ms,
                "ratio_full_over_compressed": f_ms * L / n_full / comp_ms,
                "note": "same decode kernel over the uncompressed cache (budget = prefix length)" +
                        ("" if n_full == L else f"; {n_full} of {L} layers fit beside the inputs, time scaled by "
                                                f"{L}/{n_full}")}
            del full
            torch.cuda.empty_cache()

    if headline:
        rec["_extras"] = headline_extras(ctx, w, sess, lengths, tens, dec, prefill, decode_bytes, budgets, n_dec,
                                         n_distinct, N_total)
    del sess, tens, q_win, k, v, dec
    gc.collect()
    torch.cuda.empty_cache()
    return rec


def headline_extras(ctx: Ctx, w, sess, lengths, tens, dec, prefill, decode_bytes, budgets, n_dec, n_distinct, N_total):
    """The end-to-end leg from host buffers, the oracle's CPU baseline and the parity sample (rank-0 parts only on
    rank 0); all of it outside the timed region of the headline number."""
    np, torch, xkv, args = ctx.np, ctx.torch, ctx.xkv, ctx.args
    dev, rank, world = ctx.dev, ctx.rank, ctx.world
    L, B, Hkv, Hq, d, W, G = w.n_layers, w.batch, w.n_kv_heads, w.n_q_heads, w.head_dim, w.window, w.group
    ev = lambda: torch.cuda.Event(enable_timing=True)
    q_win = [t[0] for t in tens]
    k = [t[1] for t in tens]
    v = [t[2] for t in tens]
    out = {}

    # ---------------------------------------------------------------- end-to-end leg (host buffers)
    if not args.no_e2e:
        try:
            import psutil
            per_layer = sum(x.numel() * 2 for x in tens[0])
            avail = psutil.virtual_memory().available
            n_host = int(max(1, min(L, (avail - (16 << 30)) // max(per_layer, 1))))
            # host copies of the inputs (pageable); with less host memory than inputs the first n_host layers' buffers
            # are sent again for the later layers (same sizes, so the same traffic)
            host_layers = [tuple(x.cpu() for x in tens[l]) for l in range(n_host)]
            slots = [tuple(torch.empty(x.shape, dtype=x.dtype, pin_memory=True) for x in tens[0]) for _ in range(2)]
            host_dec = [tuple(x.cpu().pin_memory() for x in dec[s]) for s in range(n_distinct)]
            out_host = torch.empty(sess.out.shape, dtype=sess.out.dtype, pin_memory=True)
            out_dev = [sess.out, torch.empty_like(sess.out)]
            cs = torch.cuda.Stream()
            slot_free = [ev(), ev()]
            for e in slot_free:
                e.record()

            def upload():
                """Every layer's Q_win, K, V: host buffer -> one of two pinned staging buffers -> device; the staging
                copy of layer l+1 runs on the host while layer l crosses the bus."""
                main = torch.cuda.current_stream()
                cs.wait_stream(main)
                for l in range(L):
                    s = l & 1
                    slot_free[s].synchronize()
                    for dst, src in zip(slots[s], host_layers[l % n_host]):
                        dst.copy_(src)
                    with torch.cuda.stream(cs):
                        for dst, src in zip(tens[l], slots[s]):
                            dst.copy_(src, non_blocking=True)
                        slot_free[s].record(cs)
                main.wait_stream(cs)

            def e2e_step():
                e, b = prefill(host_upload=upload)
                main = torch.cuda.current_stream()
                h2d = [ev() for _ in range(n_dec)]
                done = [ev() for _ in range(n_dec)]
                d2h = [ev() for _ in range(n_dec)]
                stage = [tuple(torch.empty_like(x) for x in dec[0]) for _ in range(2)]

                def send(s):
                    with torch.cuda.stream(cs):
                        if s >= 2:
                            cs.wait_event(done[s - 2])           # the staging inputs of step s-2 have been consumed
                        for dst, src in zip(stage[s & 1], host_dec[s % n_distinct]):
                            dst.copy_(src, non_blocking=True)
                        h2d[s].record(cs)

                cs.wait_stream(main)
                send(0)
                for s in range(n_dec):
                    if s + 1 < n_dec:
                        send(s + 1)
                    main.wait_event(h2d[s])
                    if s >= 2:
                        main.wait_event(d2h[s - 2])              # the output buffer of step s-2 has been read back
                    sess.decode(*stage[s & 1], out=out_dev[s & 1])
                    done[s].record(main)
                    with torch.cuda.stream(cs):
                        cs.wait_event(done[s])
                        out_host.copy_(out_dev[s & 1], non_blocking=True)
                        d2h[s].record(cs)
                main.wait_stream(cs)
                e.append(ev())
                e[4].record()
                return e, b

            h2d_bytes = L * per_layer + n_dec * sum(x.numel() * 2 for x in dec[0])
            d2h_bytes = sess.out.numel() * 2 * n_dec + sess.layer_gains.numel() * 4
            t0 = time.perf_counter()
            e_recs = [e2e_step()]
            ctx.sync_all()
            first_s = time.perf_counter() - t0
            note_extra = ""
            if first_s < 25.0:                        # short enough to afford an untimed first pass
                e_recs = [e2e_step()]
                ctx.sync_all()
            else:
                note_extra = "; one pass only (it is also the first touch of the host buffers)"
            e_dec_ms = ctx.max_over_ranks(sum(e[3].elapsed_time(e[4]) for e, _ in e_recs))
            e_step_ms = ctx.max_over_ranks(sum(e[0].elapsed_time(e[4]) for e, _ in e_recs) / len(e_recs))
            e_bytes = ctx.sum_over_ranks(float(sum(decode_bytes(e_recs[-1][1]))) * len(e_recs))
            out["e2e"] = {
                "value": e_bytes / (e_dec_ms * 1e-3) / 1e9, "unit": "GB/s",
                "h2d_bytes_per_step": int(h2d_bytes), "d2h_bytes_per_step": int(d2h_bytes),
                "ms_per_step": e_step_ms, "host_layers_held": n_host,
                "note": "value: decode phase with q/k_new/v_new copied from pinned host memory and the output copied "
                        "back every decode step (copies on a second stream, overlapping the neighbouring steps' "
                        "compute); ms_per_step: the whole pass including the host-to-device copy of every layer's "
                        "Q_win, K and V through two pinned staging buffers of one layer each" + note_extra}
            del host_layers, slots, host_dec, out_host
        except (RuntimeError, MemoryError, ImportError) as err:          # e.g. pinned allocation refused
            out["e2e"] = {"value": None, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0,
                          "note": f"host leg failed: {str(err)[:160]}"}

    if rank != 0 or world != 1:
        return out

    # ---------------------------------------------------------------- oracle: CPU baseline + parity sample
    if not args.no_cpu_baseline:
        from oracle import xkv_oracle as O
        t0 = lengths[0]
        n_par = 3
        # a fresh pass of the CUDA path whose outputs are kept for the sample: (layer 0, sequence 0), every KV head
        _, b_gpu = prefill()
        sel = torch.full((B, Hkv, sess.max_seqlen), -1, dtype=torch.int32, device=dev)
        sess.select_layer(0, int(b_gpu[0]), k[0], v[0], sel=sel)
        sess.join()
        torch.cuda.synchronize()
        n_keep = min(int(b_gpu[0]), t0 - W) + W
        gpu_scores = sess.scores[0][:, : t0 - W].cpu().numpy().astype(np.float64)
        gpu_sel = sel[0, :, :n_keep].cpu().numpy()
        bt = sess.block_table[0, 0].cpu().numpy()
        slots_ = np.arange(n_keep)
        pages = torch.from_numpy(bt[slots_ // sess.page_size].astype(np.int64)).to(dev)
        off = torch.from_numpy(slots_ % sess.page_size).to(dev)
        gpu_rows = {g: (sess.k_pages[pages, g, off].view(torch.int16).cpu().numpy(),
                        sess.v_pages[pages, g, off].view(torch.int16).cpu().numpy()) for g in range(Hkv)}
        gpu_out = []
        for s in range(n_par):
            sess.decode(*dec[s])
            gpu_out.append(sess.out[0, 0].float().cpu().numpy().astype(np.float64))
        torch.cuda.synchronize()

        cpu_t = (tens[0][0][0:1].cpu(), tens[0][1][:t0].cpu(), tens[0][2][:t0].cpu())
        dec_cpu = [tuple(x[0, 0].cpu() for x in dec[s]) for s in range(min(n_distinct, 16))]
        r = oracle_sample(w, cpu_t, t0, int(b_gpu[0]), 12.0, dec_cpu, keep_outputs=n_par)
        sample = (f"layer 0, sequence 0 ({t0} tokens), all {Hkv} KV heads, budget {int(b_gpu[0])}: the oracle's own "
                  f"scoring, top-k and compaction, then decode steps over its own cache")
        out["cpu_baseline"] = {
            "value": r["bytes"] / r["decode_s"] / 1e9, "unit": "GB/s", "cores": r["cores"], "kind": "oracle",
            "sample": sample + f": {r['steps']} decode steps of fp64 numpy attention in {r['decode_s']:.1f} s",
            "score_seconds": r["score_s"], "select_compact_seconds": r["evict_s"],
            "score_evict_ms_per_layer_equivalent": 1e3 * (r["score_s"] + r["evict_s"]) * B,
            "note": "score/select seconds are for this one sequence; x batch gives the layer equivalent"}

        near, bad, byte_mis, score_rel = 0, 0, 0, 0.0
        k_bits = tens[0][1][:t0].view(torch.int16).cpu().numpy()
        v_bits = tens[0][2][:t0].view(torch.int16).cpu().numpy()
        for g in range(Hkv):
            wv = r["w_units"][(0, g)]
            big = wv > 1e-4 * wv.max()
            score_rel = max(score_rel, float((np.abs(gpu_scores[g] - wv)[big] / wv[big]).max()))
            if O.near_tie(wv, int(b_gpu[0])):
                near += 1
                thr = O.sort_descending(wv)[min(int(b_gpu[0]), len(wv)) - 1]
                diff = np.setxor1d(gpu_sel[g], r["kept"][g])
                if not np.all(np.abs(wv[diff] - thr) <= 1e-5 * thr):
                    bad += 1
            elif not np.array_equal(gpu_sel[g], r["kept"][g]):
                bad += 1
            byte_mis += int((gpu_rows[g][0] != O.evict_by_index(k_bits[:, g], gpu_sel[g])).sum())
            byte_mis += int((gpu_rows[g][1] != O.evict_by_index(v_bits[:, g], gpu_sel[g])).sum())
        abs_err, rel_excess, rel_l2 = 0.0, 0.0, 0.0
        for s in range(n_par):
            ref, got = r["outputs"][s], gpu_out[s]
            err = np.abs(got - ref)
            abs_err = max(abs_err, float(err.max()))
            rel_excess = max(rel_excess, float((err / (2e-2 + 1e-2 * np.abs(ref))).max()))
            rel_l2 = max(rel_l2, float((np.linalg.norm(got - ref, axis=-1) /
                                        np.maximum(np.linalg.norm(ref, axis=-1), 1e-30)).max()))
        out["parity"] = {
            "sample": f"layer 0, sequence 0 ({t0} tokens), all {Hkv} KV heads, {n_par} decode steps of its {Hq} query "
                      f"heads; computed by the fp64 oracle outside the timed region (the full-size tests cover every "
                      f"workload)",
            "heads": Hkv, "near_tie_heads": near, "mismatching_heads_outside_near_tie_band": bad,
            "score_max_rel_err": score_rel, "compaction_mismatching_elements": byte_mis,
            "attn_max_abs_err": abs_err, "attn_max_err_over_tolerance": rel_excess, "attn_max_rel_l2": rel_l2,
            "tolerance": "kept sets identical outside a 1e-5 relative near-tie band; cache rows bit-exact; attention "
                         "within 2e-2 + 1e-2 |ref|",
            "ok": bool(bad == 0 and byte_mis == 0 and rel_excess <= 1.0)}
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, help="the headline workload")
    ap.add_argument("--table", default=",".join(TABLE),
                    help="comma-separated workloads also measured into `workloads` (a few steps each), or 'none'")
    ap.add_argument("--table-steps", type=int, default=3)
    ap.add_argument("--impl", default="xkv", choices=["xkv", "reference"])
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle legs (CPU baseline and parity)")
    ap.add_argument("--decode-steps", type=int, default=None, help="override the workloads' decode steps")
    ap.add_argument("--no-prefill-attn", action="store_true",
                    help="skip the prefill attention and the scoring from its normalisers")
    ap.add_argument("--no-q8", action="store_true", help="skip the decode over caches stored in 8 bits")
    ap.add_argument("--no-full-cache", action="store_true", help="skip the uncompressed-cache decode comparison")
    ap.add_argument("--full-cache-all", action="store_true", help="uncompressed-cache comparison for every workload")
    ap.add_argument("--lanes", type=int, default=None, help="side streams of the scoring and eviction phases")
    ap.add_argument("--chunk-rows", type=int, default=0, help="decode chunk size (0 = chosen on the device)")
    ap.add_argument("--layers", type=int, default=None, help="override the number of layers (small profiling cases)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    ctx = Ctx(args)
    table = {}
    names = [] if args.table == "none" else [n for n in args.table.split(",") if n and n != args.workload]
    for n in names:
        table[n] = run_workload(ctx, n, args.table_steps, 3, headline=False)
    head = run_workload(ctx, args.workload, args.steps, args.warmup, headline=True)
    extras = head.pop("_extras", {})
    table[args.workload] = {kk: vv for kk, vv in head.items()}

    if ctx.rank != 0:
        if ctx.world > 1:
            ctx.dist.barrier()
            ctx.dist.destroy_process_group()
        return

    w = ctx.WL.CONFIGS[args.workload]
    order = [n for n in TABLE if n in table] + [n for n in table if n not in TABLE]
    line = {
        "metric": METRIC, "value": head["value"], "unit": "GB/s", "n_gpus": ctx.world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "layers": args.layers or w.n_layers, "q_heads": w.n_q_heads,
                   "kv_heads": w.n_kv_heads, "head_dim": w.head_dim, "batch_per_gpu": w.batch, "prompt": w.prompt,
                   "window": w.window, "pool_kernel": w.pool_kernel, "avg_budget": w.avg_budget,
                   "decode_steps": head["decode_steps"], "page_size": 16,
                   "parallelism": f"replicas x{ctx.world} (independent batches)",
                   "l2": "inputs larger than L2 (K/V per layer 268 MB+, compacted caches of all layers > 126 MB)",
                   "decode_inputs": f"{DEC_DISTINCT} distinct sets of step inputs, reused in turn",
                   "query_direction_reading": "window queries carry sqrt(d)*u so heavy hitters are heavy"},
        "pct_of_hbm_peak": head["pct_of_hbm_peak"],
        "decode_tokens_per_s": head["decode_tokens_per_s"],
        "score_evict_ms_per_layer": head["score_evict_ms_per_layer"],
        "score_evict_roofline": head["score_evict_roofline"],
        "phases_ms": head["phases_ms"], "solver_host_ms": head["solver_host_ms"], "budgets": head["budgets"],
        "timed_region_ms": head["timed_region_ms"],
        "full_cache_decode": head.get("full_cache_decode"),
        "prefill_attn": head.get("prefill_attn"), "score_from_prefill_lse": head.get("score_from_prefill_lse"),
        "quantized_cache_decode": head.get("quantized_cache_decode"),
        "roofline": head["roofline"], "cpu_baseline": extras.get("cpu_baseline"), "e2e": extras.get("e2e"),
        "parity": extras.get("parity"),
        "gpu_launches": head["gpu_launches"], "clocks": head["clocks"],
        "workloads": {n: table[n] for n in order},
        "paper_context": "paper reports end-to-end only (RTX A6000): 61.6% KV memory reduction, 2.1x compute "
                         "efficiency, up to 5.2x throughput; no kernel-level number exists",
    }
    if "score_xu_roofline" in head:
        line["score_xu_roofline"] = head["score_xu_roofline"]
    print(json.dumps(line))
    if ctx.world > 1:
        ctx.dist.barrier()
        ctx.dist.destroy_process_group()


if __name__ == "__main__":
    main()
