#!/usr/bin/env python3
"""Benchmark of the Top-K+phi decode step (128K-context, Llama-3.2-3B head geometry).

One "step" is one decode token through all layers of the workload: per layer one
call of ``tkphi_decode_step`` (score + select, exact branch, subtraction, residual
estimate, merge) on one stream.  The prefill summary build is timed separately
and reported under ``build``.

    python bench.py --gpus N --steps K --warmup W [--impl reference]

Prints ONE JSON line (rank 0).  With N > 1 (torchrun) every rank runs an
independent replica of the same workload on its own GPU: the path has no
exchange step, so there is no data-path collective; timing is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from workloads import CONFIGS, make_layer_inputs, make_mlp_phi_params, make_phi_params  # noqa: E402


def _peaks():
    """(HBM GB/s, bf16 TFLOP/s burst, bf16 TFLOP/s sustained, "measured" | "fallback")."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), float(d["bf16_tflops"]), float(d["bf16_tflops_sustained"]), "measured"
    return 6650.0, 1590.0, 1400.0, "fallback"


# DRAM bytes (read + write) of one launch of the scoring kernel, from an ncu capture of this kernel on the
# workload below; set to None when the kernel changes, until the counters have been taken again.
SCORE_KERNEL_NCU_TRAFFIC = {"config": "c3_3b_128k", "budget": 0.01, "bytes": 268231936 + 3233792}


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clock and throttle reasons every 100 ms while the timed region runs."""

    def __init__(self, index: int):
        self.index = index
        self.samples = []
        self.reasons = set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self._nvml = None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nvml = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._nvml = None
            return
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()

    def _run(self):
        nv = self._nvml
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4),
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h)
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            self._stop.wait(0.01)

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=2)
        med = statistics.median(self.samples) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# --------------------------------------------------------------------------- workload
def algorithmic_bytes(cfg, seq_lens, topk, n_layers):
    """Bytes the method itself must move per decode step (the score buffer is an
    implementation artefact and is not counted).  seq_lens, topk: per sequence."""
    d, r = cfg.head_dim, cfg.n_feat
    n_anchor = cfg.n_sink + cfg.n_tail
    key_stream = sum(cfg.n_kv_heads * max(0, n - n_anchor) * d * 2 for n in seq_lens)
    gather = sum(cfg.n_q_heads * (int(k) + min(n_anchor, n)) * 4 * d for n, k in zip(seq_lens, topk))
    su = len(seq_lens) * cfg.n_kv_heads * (d * r + r) * 4
    weights = (cfg.n_q_heads + cfg.n_kv_heads) * (r * d + r) * 4
    per_layer = key_stream + gather + su + weights
    return {"key_stream": key_stream * n_layers, "total": per_layer * n_layers,
            "key_stream_per_layer": key_stream}


def workload_string(cfg, n_layers, N, budget, tmax, seq_lens=None):
    """The same text in both arms, so that the two lines can be matched."""
    s = (f"{cfg.name}: {n_layers} layers x {cfg.n_q_heads}q/{cfg.n_kv_heads}kv heads, d={cfg.head_dim}, "
         f"r={cfg.n_feat}, N={N}, anchors {cfg.n_sink}+{cfg.n_tail}, budget {budget:g} (K<={tmax}), batch {cfg.batch}")
    if seq_lens is not None and len(set(seq_lens)) > 1:
        s += f", ragged lengths {min(seq_lens)}..{max(seq_lens)}"
    return s


def run_ours(args, rank, world, device):
    import paper_2604_05438_b200 as T
    from paper_2604_05438_b200.build import build_library
    build_library()
    T.load_library()
    cfg = CONFIGS[args.config]
    n_layers = args.layers or cfg.n_layers
    N = args.seq_len or cfg.seq_len
    seed = 0
    torch.cuda.set_device(device)
    layers, phis, Ss, us = [], [], [], []
    t_gen = time.time()
    for l in range(n_layers):
        inp = make_layer_inputs(cfg, seed, layer=l, device=device,
                                seq_lens=([N] * cfg.batch) if (args.seq_len or cfg.seq_len_min is None) else None, n_steps=1)
        kv = T.KVCache(inp.k, inp.v, inp.cu_seqlens, cfg.n_q_heads, cfg.n_feat, cfg.n_sink, cfg.n_tail)
        layers.append((inp, kv))
        cache = (torch.empty(cfg.n_kv_heads, int(inp.cu_seqlens[-1]), cfg.n_feat, device=device)
                 if (args.phi_cache or args.mlp_phi) else None)   # written by the build, read by the decode steps
        if args.mlp_phi:      # the ReZero-MLP maps: (query side, key side, cache)
            mq, mk = (make_mlp_phi_params(cfg, seed + l, side, device=device) for side in ("q", "k"))
            phis.append((T.MlpMaps(mq.w_s, mq.b_s, mq.w_1, mq.b_1, mq.w_2, mq.b_2, mq.alpha, mq.w_o, mq.b_o),
                         T.MlpMaps(mk.w_s, mk.b_s, mk.w_1, mk.b_1, mk.w_2, mk.b_2, mk.alpha, mk.w_o, mk.b_o), cache))
        else:
            phi = make_phi_params(cfg, seed + l, device=device)
            phis.append(T.PhiMaps(phi.w_q, phi.b_q, phi.w_k, phi.b_k, phi.gamma_q, phi.gamma_k, cache))
    torch.cuda.synchronize()
    t_gen = time.time() - t_gen
    topk = layers[0][0].topk(args.budget)
    tmax = int(topk.max())
    topk_dev = torch.from_numpy(topk).to(device)
    B, Hq, Hkv, d, r = cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_feat
    kv0 = layers[0][1]
    ws = torch.empty(T.workspace_bytes(kv0, topk, tmax, T.WS_DECODE_STEP), dtype=torch.uint8, device=device)
    wsb = torch.empty(T.workspace_bytes(kv0, None, 0, T.WS_BUILD), dtype=torch.uint8, device=device)

    # ---- prefill summary build (timed separately)
    for l in range(n_layers):
        Ss.append(torch.empty(B, Hkv, d, r, device=device))
        us.append(torch.empty(B, Hkv, r, device=device))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    mlp_ms = None
    if args.mlp_phi:      # key features of every cache row first (timed by itself), then the build from those rows
        wsm = torch.empty(T.workspace_bytes(kv0, None, 0, T.WS_MLP_KEY_FEATURES), dtype=torch.uint8, device=device)
        T.mlp_key_features(layers[0][1], phis[0][1], phis[0][2], wsm)    # warm-up
        torch.cuda.synchronize()
        e0.record()
        for l in range(n_layers):
            T.mlp_key_features(layers[l][1], phis[l][1], phis[l][2], wsm)
        e1.record()
        torch.cuda.synchronize()
        mlp_ms = e0.elapsed_time(e1)
        assert T.device_status(wsm) == 0, "a device-side wait timed out"
        del wsm
        build_one = lambda l: T.build_summaries_cached(layers[l][1], phis[l][2], Ss[l], us[l], wsb)
    else:
        build_one = lambda l: T.build_summaries(layers[l][1], phis[l], Ss[l], us[l], wsb)
    build_one(0)                                                     # warm-up
    torch.cuda.synchronize()

    def build_all():
        for l in range(n_layers):
            build_one(l)

    if args.graph:      # as for the decode steps: the calls captured once, the graph replayed
        cap_b = torch.cuda.Stream()
        graph_b = torch.cuda.CUDAGraph()
        prev_b = torch.cuda.current_stream()
        with torch.cuda.stream(cap_b):
            with torch.cuda.graph(graph_b, stream=cap_b):
                build_all()
        torch.cuda.set_stream(prev_b)
        build_all = graph_b.replay
        build_all()                                                  # warm-up of the replay
        torch.cuda.synchronize()
    e0.record()
    build_all()
    e1.record()
    torch.cuda.synchronize()
    build_ms = e0.elapsed_time(e1)

    # ---- decode queries: a fresh query per step, resident in HBM for the device-timed loop
    n_q_sets = 8
    g = torch.Generator(device=device)
    g.manual_seed(1234)
    topic_q = [layers[l][0].q[0] for l in range(n_layers)]          # [B,Hq,d] bf16 correlated with needles
    q_dev = []
    for s in range(n_q_sets):
        qs = torch.stack([(topic_q[l].float() + 0.5 * torch.randn(B, Hq, d, generator=g, device=device))
                          .to(torch.bfloat16) for l in range(n_layers)])
        q_dev.append(qs.contiguous())                                # [layers,B,Hq,d]
    y_dev = torch.empty(n_layers, B, Hq, d, device=device)

    def step(qs):
        for l in range(n_layers):
            if args.mlp_phi:
                T.decode_step_mlp(layers[l][1], phis[l][0], phis[l][2], qs[l], topk, topk_dev, tmax, Ss[l], us[l],
                                  None, y_dev[l], None, 0, ws)
            else:
                T.decode_step(layers[l][1], phis[l], qs[l], topk, topk_dev, tmax, Ss[l], us[l], None, y_dev[l],
                              None, 0, ws)

    if args.graph:      # the step's launches captured once into a CUDA graph; every step copies its queries in and replays
        q_graph = torch.empty_like(q_dev[0])
        step_eager = step
        step_eager(q_graph.copy_(q_dev[0]))
        torch.cuda.synchronize()
        cap = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        prev = torch.cuda.current_stream()
        with torch.cuda.stream(cap):
            with torch.cuda.graph(graph, stream=cap):
                step_eager(q_graph)
        torch.cuda.set_stream(prev)

        def step(qs):
            q_graph.copy_(qs, non_blocking=True)
            graph.replay()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    for w in range(args.warmup):
        step(q_dev[w % n_q_sets])
    barrier()
    sampler = ClockSampler(device.index or 0)
    sampler.start()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    ev[0].record()
    for s in range(args.steps):
        step(q_dev[s % n_q_sets])
        ev[s + 1].record()
    barrier()
    per_step = [ev[s].elapsed_time(ev[s + 1]) for s in range(args.steps)]
    total_ms = ev[0].elapsed_time(ev[args.steps])
    assert T.device_status(ws) == 0, "a device-side wait timed out"
    assert torch.isfinite(y_dev).all()

    # ---- per-kernel durations (second pass with the library's event hooks), for the roofline
    kt = None
    if hasattr(T, "kernel_timing"):
        timed_step = step_eager if args.graph else step      # the event hooks fire at launch time, not on a replay
        kt = T.kernel_timing(lambda: [timed_step(q_dev[s % n_q_sets]) for s in range(min(args.steps, 8))])

    # ---- the Top-K baseline path (tkphi_topk_decode: same scoring, selection and exact branch, no residual), timed beside
    def step_topk(qs):
        for l in range(n_layers):
            T.topk_decode(layers[l][1], qs[l], topk, topk_dev, tmax, None, y_dev[l], ws)
    n_tk = min(args.steps, 8)
    for w in range(2):
        step_topk(q_dev[w % n_q_sets])
    e0.record()
    for s in range(n_tk):
        step_topk(q_dev[s % n_q_sets])
    e1.record()
    torch.cuda.synchronize()
    topk_only_us = e0.elapsed_time(e1) * 1e3 / n_tk

    # ---- end to end: host buffers, H2D of the queries and D2H of the outputs inside the timed region
    q_host = [qs.cpu().pin_memory() for qs in q_dev]
    y_host = torch.empty(n_layers, B, Hq, d).pin_memory()
    q_stage = torch.empty_like(q_dev[0])

    def step_e2e(s):
        q_stage.copy_(q_host[s % n_q_sets], non_blocking=True)
        step(q_stage)
        y_host.copy_(y_dev, non_blocking=True)
        torch.cuda.current_stream().synchronize()     # the caller reads y before the next token

    for w in range(min(args.warmup, 3)):
        step_e2e(w)
    barrier()
    t0 = time.perf_counter()
    for s in range(args.steps):
        step_e2e(s)
    barrier()
    e2e_ms = (time.perf_counter() - t0) * 1e3 / args.steps
    clocks = sampler.stop()          # sampled over both timed regions (device-timed loop and end-to-end loop)

    ms, e2e_ms = max_over_ranks([total_ms / args.steps, e2e_ms], world, device)

    seq_lens = [layers[0][0].seq_len(b) for b in range(B)]
    ab = algorithmic_bytes(cfg, seq_lens, topk, n_layers)
    peak, tf_burst, tf_sust, peak_kind = _peaks()
    out = {
        "metric": "Top-K+phi decode-step latency (us), 128K ctx",
        "value": ms * 1e3, "unit": "us/step", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 K/V, f32 accumulate", "data": "synthetic",
        "config": {"workload": workload_string(cfg, n_layers, N, args.budget, tmax, seq_lens),
                   "l2": "inputs (K/V of all layers) exceed L2 by >100x; no flush needed",
                   "replicas": world, "seed": seed, "phi_k_cache": bool(args.phi_cache or args.mlp_phi), "cuda_graph": bool(args.graph),
                   "phi": "one-block ReZero MLP, d_emb 512" if args.mlp_phi else "exp(Wx + b - |x|^2/2)"},
        "step_us": {"median": statistics.median(per_step) * 1e3, "min": min(per_step) * 1e3,
                    "max": max(per_step) * 1e3},
        "achieved_gbs": ab["total"] / (ms * 1e-3) / 1e9,
        "hbm_frac_of_measured_peak": ab["total"] / (ms * 1e-3) / 1e9 / peak,
        "algorithmic_bytes_per_step": ab["total"],
        "steps_per_s_all_gpus": whole_job_steps_per_s(ms, world),
        "gpu_launches": args.steps * n_layers * (8 if args.mlp_phi else 4 if args.phi_cache else 3),
        "e2e": {"value": e2e_ms * 1e3, "unit": "us/step", "h2d_bytes_per_step": q_stage.numel() * 2,
                "d2h_bytes_per_step": y_host.numel() * 4},
        "build": build_info(build_ms, n_layers, Hkv, sum(max(0, n - cfg.n_sink - cfg.n_tail) for n in seq_lens), d, r,
                            peak, tf_burst, tf_sust),
        "topk_decode_us_per_step": topk_only_us,
        "clocks": clocks,
        "gen_s": t_gen,
    }
    if mlp_ms is not None:      # four GEMMs per token and KV head: d x E, E x E twice, E x r (E = hidden width 512)
        E = 512
        fl = 2.0 * n_layers * Hkv * sum(seq_lens) * (d * E + 2 * E * E + E * r)
        out["mlp_key_features"] = {"ms_all_layers": mlp_ms, "tflops_bf16": fl / (mlp_ms * 1e-3) / 1e12,
                                   "frac_of_bf16_sustained_peak": fl / (mlp_ms * 1e-3) / 1e12 / tf_sust}
    if kt is not None:
        dom = kt["score"]
        a = ab["key_stream_per_layer"] / (dom["avg_ms"] * 1e-3) / 1e9
        t = SCORE_KERNEL_NCU_TRAFFIC
        traffic = (t["bytes"] if t and t["config"] == args.config and abs(t["budget"] - args.budget) < 1e-9
                   and not args.seq_len else None)
        out["roofline"] = {"bound": "hbm", "kernel": "score_kernel", "scope": "score_kernel only (the whole step: "
                           "hbm_frac_of_measured_peak)", "achieved": a, "peak": peak,
                           "unit": "GB/s", "frac": a / peak, "traffic": traffic,
                           "peak_kind": peak_kind, "algorithmic_bytes_per_launch": ab["key_stream_per_layer"],
                           "avg_launch_us": dom["avg_ms"] * 1e3}
        out["kernels_us_per_launch"] = {k: v["avg_ms"] * 1e3 for k, v in kt.items()}
    return out, (cfg, layers, phis, Ss, us, topk)


def max_over_ranks(values, world, device=None):
    """Replicas run independently (the path has no exchange step); a multi-rank number is the
    slowest rank's.  Returns the element-wise maximum of `values` over all ranks."""
    if world <= 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), device=device or "cpu", dtype=torch.float64)
    torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return [float(v) for v in t]


def whole_job_steps_per_s(ms_per_step, world):
    """Weak scaling: every rank decodes its own replica, so the job does `world` steps per step time."""
    return world * 1e3 / ms_per_step


def build_info(build_ms, n_layers, Hkv, n_mid, d, r, hbm_peak, tf_burst, tf_sust):
    """Prefill summary build, timed separately: K and V of the mid-region are read once;
    the two contractions cost 2 * (2 n d r) flop per KV head, issued twice each (bf16 hi + lo)."""
    kv_bytes = 2 * n_layers * Hkv * n_mid * d * 2          # n_mid: mid-region tokens summed over sequences
    flops_alg = 4.0 * n_layers * Hkv * n_mid * d * r
    t = build_ms * 1e-3
    return {"ms_all_layers": build_ms, "bound": "tensor",
            "kv_bytes": kv_bytes, "achieved_gbs": kv_bytes / t / 1e9,
            "hbm_frac_of_measured_peak": kv_bytes / t / 1e9 / hbm_peak,
            "algorithmic_tflops": flops_alg / t / 1e12, "issued_tflops_bf16": 2 * flops_alg / t / 1e12,
            "issued_frac_of_bf16_burst_peak": 2 * flops_alg / t / 1e12 / tf_burst,
            "issued_frac_of_bf16_sustained_peak": 2 * flops_alg / t / 1e12 / tf_sust}


# --------------------------------------------------------------------------- oracle legs
class OracleSample:
    """The float64 oracle (as it stands) on `n_heads` query heads of one layer of the workload.
    Inputs and the prefill summaries are prepared once; `step(i)` times one decode query per
    sampled head and scales to a full step (all heads, all sequences, one layer)."""

    def __init__(self, cfg, N, budget, n_heads, n_queries, seed=0, fixed_len=True):
        from oracle import tkphi_oracle as O
        self.O, self.cfg = O, cfg
        try:
            from threadpoolctl import threadpool_info
            self.threads = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
        except Exception:
            self.threads = 1
        self.inp = make_layer_inputs(cfg, seed, layer=0, seq_lens=[N] * cfg.batch if fixed_len else None,
                                     n_steps=n_queries)
        self.phi = make_phi_params(cfg, seed)
        self.topk = int(self.inp.topk(budget)[0])
        G = cfg.group
        self.heads = list(range(0, cfg.n_q_heads, max(1, cfg.n_q_heads // n_heads)))[:n_heads]
        self.built = {}
        for hq in self.heads:       # summaries are prefill state: built outside the timed decode sample
            kvh = hq // G
            if kvh not in self.built:
                K = self.inp.k[kvh, :N].double().numpy()
                V = self.inp.v[kvh, :N].double().numpy()
                self.built[kvh] = (K, V) + O.build_summaries(K, V, self.phi.w_k[kvh].double().numpy(),
                                                             self.phi.b_k[kvh].double().numpy(), self.phi.gamma_k,
                                                             cfg.n_sink, cfg.n_tail)

    def step(self, i):
        """Seconds of oracle time for the sampled heads, and the estimate for one full layer step."""
        O, cfg, phi = self.O, self.cfg, self.phi
        qi = i % self.inp.q.shape[0]
        t0 = time.perf_counter()
        for hq in self.heads:
            kvh = hq // cfg.group
            K, V, S, u = self.built[kvh]
            O.topkphi_attention(self.inp.q[qi, 0, hq].double().numpy(), K, V, cfg.n_sink, cfg.n_tail, self.topk,
                                phi.w_q[hq].double().numpy(), phi.b_q[hq].double().numpy(), phi.gamma_q,
                                phi.w_k[kvh].double().numpy(), phi.b_k[kvh].double().numpy(), phi.gamma_k,
                                S=S, u=u)
        dt = time.perf_counter() - t0
        return dt, dt / len(self.heads) * cfg.n_q_heads * cfg.batch


def run_reference(args):
    cfg = CONFIGS[args.config]
    n_layers = args.layers or cfg.n_layers
    N = args.seq_len or cfg.seq_len
    n_heads = 2
    smp = OracleSample(cfg, N, args.budget, n_heads, n_queries=max(1, min(16, args.warmup + args.steps)),
                       fixed_len=bool(args.seq_len) or cfg.seq_len_min is None)
    vals = []
    for s in range(args.warmup + args.steps):
        dt, per_layer_s = smp.step(s)
        if s >= args.warmup:
            vals.append(per_layer_s * n_layers)
    us = statistics.mean(vals) * 1e6
    seq_lens = [smp.inp.seq_len(b) for b in range(smp.inp.batch)]
    tmax = int(smp.inp.topk(args.budget).max())
    scale = cfg.n_q_heads * cfg.batch * n_layers / n_heads
    sample = (f"{n_heads} of {cfg.n_q_heads} query heads of sequence 0 of one layer per step, full N={N}, "
              f"scaled by heads, {cfg.batch} sequence(s) and {n_layers} layers; summaries prebuilt")
    return {
        "impl": "reference", "metric": "Top-K+phi decode-step latency (us), 128K ctx", "value": us,
        "unit": "us/step", "n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "ms_per_step": us / 1e3,
        "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_string(cfg, n_layers, N, args.budget, tmax, seq_lens)},
        "extrapolated": True, "scale_factor": scale,
        "cpu_baseline": {"value": us, "unit": "us/step", "cores": smp.threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": us, "unit": "us/step", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=32)
    ap.add_argument("--warmup", type=int, default=4)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="c3_3b_128k", choices=sorted(CONFIGS))
    ap.add_argument("--budget", type=float, default=0.01)
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (profiling)")
    ap.add_argument("--seq-len", type=int, default=0, help="override the context length (profiling)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", dest="graph", action="store_false",
                    help="launch every layer call eagerly instead of replaying the step's launches from a CUDA graph "
                         "(captured once from the same library calls; the default)")
    ap.add_argument("--mlp-phi", action="store_true",
                    help="feature maps = the one-block ReZero MLP: key features by tkphi_mlp_key_features into a cache, "
                         "summaries built from the cache, decode steps through tkphi_decode_step_mlp")
    ap.add_argument("--phi-cache", action="store_true",
                    help="keep the key features the build computes and read them at decode time (Sec. 4.2, cached variant)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        if rank == 0:
            print(json.dumps(run_reference(args)), flush=True)
        return 0

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback); use --impl reference for the oracle")
    device = torch.device("cuda", local)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.distributed.init_process_group("nccl", device_id=device)
    out, _ = run_ours(args, rank, world, device)
    if rank == 0:
        if not args.no_cpu_baseline:
            cfg = CONFIGS[args.config]
            n_layers = args.layers or cfg.n_layers
            N = args.seq_len or cfg.seq_len
            smp = OracleSample(cfg, N, args.budget, 8, n_queries=16,
                               fixed_len=bool(args.seq_len) or cfg.seq_len_min is None)
            dts, ests = zip(*[smp.step(i) for i in range(16)])
            out["cpu_baseline"] = {
                "value": statistics.mean(ests) * n_layers * 1e6, "unit": "us/step", "cores": smp.threads,
                "kind": "oracle",
                "sample": f"{len(smp.heads)} of {cfg.n_q_heads} query heads of one layer at full N={N}, 16 decode "
                          f"queries each ({sum(dts):.1f} s of oracle time), scaled by heads and {n_layers} layers; "
                          f"summaries prebuilt"}
        print(json.dumps(out), flush=True)
    if world > 1:
        torch.distributed.barrier()
        torch.distributed.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
