#!/usr/bin/env python
"""Benchmark of the A/F decode-layer hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config C] [--depth M]

A "step" is one pass of the whole hot path -- aflex_layer_step: paged GQA decode attention,
the W_o boundary projection and the dense (or MoE) SwiGLU FFN -- over one decode batch of
seeded synthetic input.  The default workload is configuration 2 (Qwen3-32B-shaped layer,
batch 32, context lengths U[512,4096], page size 16, shuffled page table), microbatch depth 1.
Prints ONE JSON line:

  value        decode-layer tokens/s, inputs resident in HBM, CUDA events around K steps
  e2e          the same with q / page table / sequence lengths copied from pinned host memory
               and y copied back, every step, inside the timed region
  roofline     the dominant kernel's achieved HBM rate against the measured copy bandwidth
  kernels      the same figures for every kernel kind of the step
  cpu_baseline the fp64 oracle timed on this machine's host cores on a bounded sample

With --gpus N > 1 (under torchrun) every rank runs an independent replica of the step on its
own GPU (the path has no exchange step on one node); value = N * B / max-over-ranks time.
--impl reference times the CPU oracle instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2608_01891_b200 import inputs as IN  # noqa: E402

METRIC = "decode-layer tokens/s (Qwen3-32B shape); attn HBM GB/s & FFN TFLOPS % of peak"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "50", "-i", str(self.index)],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) >= 7:
                self.rows.append(parts)

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.12)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except ValueError:
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def max_over_ranks(ms: float, dist, device) -> float:
    """Slowest rank's time: the job is only as fast as its slowest replica."""
    if dist is None:
        return ms
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_s(world: int, batch_per_rank: int, ms_per_step: float) -> float:
    """Weak scaling over independent replicas: every rank decodes its own batch each step."""
    return world * batch_per_rank / (ms_per_step * 1e-3)


def algorithmic_bytes(cfg, lens, M):
    """Algorithmic HBM bytes per launch of each kernel kind (every K/V element and every weight read
    once; activations, partial results and outputs once each).  Per step, per microbatch launch."""
    B, Hq, D, H, I = cfg.batch, cfg.num_q_heads, cfg.head_dim, cfg.hidden, cfg.inter
    A = Hq * D
    kv = float(np.sum(lens.astype(np.int64)) * cfg.kv_bytes_per_token) + 2.0 * B * A * 2 + float(np.sum((lens + 15) // 16)) * 4
    out = {"attn_decode": kv / M}
    rows = B / M
    out["linear_gemm"] = H * A * 2 + rows * (A + H) * 2
    if cfg.num_experts == 0:
        out["gateup_gemm"] = 2.0 * I * H * 2 + rows * (H + I) * 2
        out["down_gemm"] = 1.0 * H * I * 2 + rows * (I + H) * 2
        # decode batches run gate/up and down (and, at depth 1, W_o in front of them) as phases of one kernel
        out["gemm_chain"] = out["gateup_gemm"] + out["down_gemm"] + (out["linear_gemm"] if M == 1 else 0.0)
    else:
        E, K = cfg.num_experts, cfg.top_k
        out["moe_gateup_gemm"] = 2.0 * E * I * H * 2 + rows * K * (H + I) * 2
        out["moe_down_gemm"] = 1.0 * E * H * I * 2 + rows * K * (I * 2 + H * 4)
    return out


def algorithmic_flops(cfg, M):
    B, Hq, D, H, I = cfg.batch, cfg.num_q_heads, cfg.head_dim, cfg.hidden, cfg.inter
    rows = B / M
    k = cfg.top_k if cfg.num_experts else 1
    return {"linear_gemm": 2.0 * rows * H * Hq * D, "gateup_gemm": 4.0 * rows * H * I, "down_gemm": 2.0 * rows * H * I,
            "gemm_chain": 6.0 * rows * H * I + (2.0 * rows * H * Hq * D if M == 1 else 0.0),
            "moe_gateup_gemm": 4.0 * rows * k * H * I, "moe_down_gemm": 2.0 * rows * k * H * I}


def measure_energy(step, barrier, gpu_index, tokens_per_step, ms_step):
    """Joules per token from nvmlDeviceGetTotalEnergyConsumption around a >= 2 s loop of the step, at the
    clocks the GPU is found at (GPU settings are never changed).  Returns a dict, or a reason string."""
    try:
        import pynvml
        pynvml.nvmlInit()
        # NVML enumerates physical GPUs; map through CUDA_VISIBLE_DEVICES when it is a plain index list
        vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
        idx = gpu_index
        if vis and all(v.strip().isdigit() for v in vis.split(",")):
            idx = int(vis.split(",")[gpu_index])
        h = pynvml.nvmlDeviceGetHandleByIndex(idx)
        steps = max(50, int(2000.0 / max(ms_step, 1e-3)))
        barrier()
        e0 = pynvml.nvmlDeviceGetTotalEnergyConsumption(h)
        t0 = time.perf_counter()
        for _ in range(steps):
            step()
        barrier()
        dt = time.perf_counter() - t0
        e1 = pynvml.nvmlDeviceGetTotalEnergyConsumption(h)
        joules = (e1 - e0) / 1000.0
        return {"joules_per_token": joules / (steps * tokens_per_step), "watts_avg": joules / dt, "seconds": round(dt, 2),
                "steps": steps, "clocks": "as found (locked-clock sweep: changing GPU settings is closed on this pool)"}
    except Exception as exc:   # no NVML, no permission, unsupported counter
        return {"unavailable": str(exc)[:200]}


def run_energy_ops(args, cfg, local_rank, device, peaks):
    """Per-operator time and energy per token at the clocks the GPU is found at (the per-operator side of the paper's
    Section 3.2 frequency-sensitivity study; the clock sweep itself would need GPU settings to be changed)."""
    from paper_2608_01891_b200 import aflex as AF
    wl = build_workload(cfg, device)
    ctx = AF.Context(local_rank, max(AF.workspace_bytes(wl["layer"], cfg.batch, wl["kvh"].max_pages_per_seq), 6 << 30))
    stream = torch.cuda.current_stream()
    dense = dataclasses_replace_dense(cfg)
    H = cfg.hidden
    desc = AF.attn_desc(cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim)
    a_out = torch.empty_like(wl["q"])
    ops = [("attn_decode", cfg.batch, lambda: ctx.attn_decode(desc, wl["q"], wl["kv"], a_out, None, stream))]
    if cfg.num_experts == 0:
        wg, wu, wd = wl["wg"], wl["wu"], wl["wd"]
    else:
        wg, wu, wd = IN.make_ffn_weights(dense, device=device)
    for T in (32, 2048):
        x = IN.make_x(dense, device=device, tokens=T)
        y = torch.empty(T, H, dtype=torch.bfloat16, device=device)
        ops.append((f"ffn_dense(T={T})", T, (lambda x=x, y=y: ctx.ffn_dense(x, wg, wu, wd, y, stream))))
    ops.append(("layer_step(M=1)", cfg.batch,
                lambda: ctx.layer_step(wl["layer"], wl["q"], wl["kv"], wl["y"], 1, None, wl["logits"], None, stream)))
    sampler = ClockSampler(local_rank)
    sampler.start()
    rows = []
    for name, tokens, fn in ops:
        for _ in range(5):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(20):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / 20
        en = measure_energy(fn, torch.cuda.synchronize, local_rank, tokens, ms)
        row = {"operator": name, "tokens": tokens, "us": round(ms * 1e3, 1)}
        if "joules_per_token" in en:
            row.update({"mj_per_token": round(en["joules_per_token"] * 1e3, 3), "watts_avg": round(en["watts_avg"], 1)})
        else:
            row.update(en)
        rows.append(row)
    assert ctx.device_status() == AF.OK
    line = {"metric": "per-operator time and energy per token at default clocks", "unit": "mJ/token", "dtype": "bf16",
            "data": "synthetic", "config": {"workload": f"config {cfg.cfg_id}: {cfg.name}, operators alone"},
            "clocks": sampler.stop(), "locked_clock_sweep": "closed on this pool (GPU settings are never changed)",
            "operators": rows}
    print(json.dumps(line), flush=True)
    ctx.close()


def run_ffn_sweep(args, cfg, local_rank, device, peaks):
    """Dense SwiGLU FFN at the configuration's (H, I) over a range of token counts: where the FFN stops being
    a weight-streaming kernel and becomes a tensor-core kernel (arithmetic intensity ~ T flop per weight byte)."""
    from paper_2608_01891_b200 import aflex as AF
    H, I = cfg.hidden, cfg.inter
    dense = dataclasses_replace_dense(cfg)
    wg, wu, wd = IN.make_ffn_weights(dense, device=device)
    ctx = AF.Context(local_rank, 6 << 30)
    stream = torch.cuda.current_stream()
    sampler = ClockSampler(local_rank)
    sampler.start()
    rows = []
    for T in ([args.ffn_tokens] if args.ffn_tokens > 0 else (32, 64, 128, 256, 512, 1024, 2048, 4096, 8192)):
        x = IN.make_x(dense, device=device, tokens=T)
        y = torch.empty(T, H, dtype=torch.bfloat16, device=device)
        for _ in range(max(3, args.warmup)):
            ctx.ffn_dense(x, wg, wu, wd, y, stream)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n = max(10, args.steps // 2)
        e0.record(stream)
        for _ in range(n):
            ctx.ffn_dense(x, wg, wu, wd, y, stream)
        e1.record(stream)
        torch.cuda.synchronize()
        us = 1e3 * e0.elapsed_time(e1) / n
        flops = 6.0 * T * H * I
        wbytes = 3.0 * H * I * 2 + 2.0 * T * H * 2 + 2.0 * T * I * 2
        rows.append({"T": T, "us": round(us, 1), "tflops": round(flops / us / 1e6, 1),
                     "frac_bf16_burst": round(flops / us / 1e6 / peaks["bf16_tflops"], 4),
                     "frac_bf16_sustained": round(flops / us / 1e6 / peaks["bf16_tflops_sustained"], 4),
                     "weight_stream_gbs": round(wbytes / us / 1e3, 1),
                     "frac_hbm": round(wbytes / us / 1e3 / peaks["hbm_gbs"], 4)})
        ctx.profile_enable(True)                       # per kernel under event pairs (serialised: no launch overlap)
        for _ in range(3):
            ctx.ffn_dense(x, wg, wu, wd, y, stream)
        rows[-1]["kernels_us"] = {k: round(1e3 * v[0] / v[1], 1) for k, v in ctx.profile_read().items()}
        ctx.profile_enable(False)
    assert ctx.device_status() == AF.OK
    line = {"metric": "dense FFN throughput vs tokens (Qwen3-32B FFN shape)" if cfg.cfg_id in (2, 3) else
            f"dense FFN throughput vs tokens (H={H}, I={I})", "unit": "TFLOP/s", "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"ffn token sweep, H={H}, I={I}", "l2": "weights (>= 786 MB) larger than L2, no flush"},
            "peaks": peaks, "clocks": sampler.stop(), "sweep": rows}
    print(json.dumps(line), flush=True)
    ctx.close()


def run_prefill(args, cfg, local_rank, device, peaks):
    """Prefill (causal) attention over the paged cache at the configuration's head shape: whole prompts of several
    lengths, a ragged batch and a chunk appended to a long cached prefix.  Compute-bound, so each row reports
    TFLOP/s of the causal flops (4 Hq D per visible query-key pair) against the measured dense bf16 peaks."""
    from paper_2608_01891_b200 import aflex as AF
    Hq, Hkv, D = cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim
    ctx = AF.Context(local_rank, 1 << 26)
    stream = torch.cuda.current_stream()
    desc = AF.attn_desc(Hq, Hkv, D)
    rng = np.random.default_rng(20260801)
    cases = [("whole prompts 8 x 1024", [1024] * 8, None), ("whole prompts 8 x 2048", [2048] * 8, None),
             ("whole prompts 4 x 4096", [4096] * 4, None), ("whole prompts 2 x 8192", [8192] * 2, None),
             ("whole prompt 1 x 16384", [16384], None),
             ("ragged prompts, 8 lengths in [512, 4096]", [int(v) for v in rng.integers(512, 4097, size=8)], None),
             ("chunk of 2048 onto 8192 cached, 2 sequences", [10240] * 2, [2048] * 2)]
    if args.prefill_case >= 0:
        cases = cases[args.prefill_case:args.prefill_case + 1]
    sampler = ClockSampler(local_rank)
    sampler.start()
    rows = []
    for name, cached, new in cases:
        new = cached if new is None else new
        B = len(cached)
        c = dataclasses.replace(cfg, batch=B)
        lens = np.asarray(cached, dtype=np.int32)
        kvh = IN.make_paged_kv(c, lens, device=device)
        kv = AF.make_kv(kvh.k_cache, kvh.v_cache, kvh.page_table.to(device), kvh.seq_lens.to(device), kvh.seq_lens)
        qo = torch.zeros(B + 1, dtype=torch.int32)
        qo[1:] = torch.cumsum(torch.tensor(new, dtype=torch.int32), 0)
        qod = qo.to(device)
        T = int(qo[-1])
        q = (torch.randn(T, Hq, D, device=device) * 1.0).to(torch.bfloat16)
        out = torch.empty_like(q)
        pairs = sum(m * (n - m) + m * (m + 1) // 2 for n, m in zip(cached, new))
        flops = 4.0 * Hq * D * pairs
        for _ in range(max(3, args.warmup)):
            ctx.attn_prefill(desc, q, kv, qod, qo, out, stream)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.steps):
            ctx.attn_prefill(desc, q, kv, qod, qo, out, stream)
        e1.record(stream)
        torch.cuda.synchronize()
        us = 1e3 * e0.elapsed_time(e1) / args.steps
        tf = flops / us / 1e6
        rows.append({"case": name, "query_tokens": T, "us": round(us, 1), "tflops": round(tf, 1),
                     "frac_bf16_burst": round(tf / peaks["bf16_tflops"], 4),
                     "frac_bf16_sustained": round(tf / peaks["bf16_tflops_sustained"], 4)})
        del kvh, kv, q, out
    assert ctx.device_status() == AF.OK
    line = {"metric": "prefill attention throughput (causal flops)", "unit": "TFLOP/s", "dtype": "bf16", "data": "synthetic",
            "steps": args.steps, "warmup": max(3, args.warmup),
            "config": {"workload": f"causal attention over the paged cache, Hq={Hq}, Hkv={Hkv}, D={D}",
                       "l2": "q, out and K/V of a case exceed L2 together; no flush between iterations"},
            "peaks": peaks, "clocks": sampler.stop(), "cases": rows}
    print(json.dumps(line), flush=True)
    ctx.close()


def run_moe_sweep(args, cfg, local_rank, device, peaks):
    """Top-k MoE FFN (router logits given) at the configuration's (H, I, E, K) over a range of token counts: from the
    decode regime (every expert's weights streamed for a handful of rows) to the prefill regime (hundreds to thousands
    of rows per expert, tensor-core bound)."""
    from paper_2608_01891_b200 import aflex as AF
    H, I, E, K = cfg.hidden, cfg.inter, cfg.num_experts, cfg.top_k
    wg, wu, wd = IN.make_ffn_weights(cfg, device=device)
    ctx = AF.Context(local_rank, 8 << 30)
    stream = torch.cuda.current_stream()
    sampler = ClockSampler(local_rank)
    sampler.start()
    rows = []
    for T in (64, 256, 512, 1024, 2048, 4096, 8192):
        x = IN.make_x(cfg, device=device, tokens=T)
        logits = IN.make_router_logits(cfg, tokens=T).to(device)
        y = torch.empty(T, H, dtype=torch.bfloat16, device=device)
        counts = torch.zeros(E, dtype=torch.int32, device=device)
        for _ in range(max(3, args.warmup)):
            ctx.ffn_moe(x, wg, wu, wd, K, y, router_logits=logits, expert_counts=counts, stream=stream)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n = max(10, args.steps // 2)
        e0.record(stream)
        for _ in range(n):
            ctx.ffn_moe(x, wg, wu, wd, K, y, router_logits=logits, expert_counts=counts, stream=stream)
        e1.record(stream)
        torch.cuda.synchronize()
        us = 1e3 * e0.elapsed_time(e1) / n
        flops = 6.0 * T * K * H * I
        wbytes = 3.0 * E * H * I * 2 + 2.0 * T * K * H * 2 + 2.0 * T * K * I * 2
        rows.append({"T": T, "rows_per_expert": counts.cpu().tolist(), "us": round(us, 1), "tflops": round(flops / us / 1e6, 1),
                     "frac_bf16_burst": round(flops / us / 1e6 / peaks["bf16_tflops"], 4),
                     "frac_bf16_sustained": round(flops / us / 1e6 / peaks["bf16_tflops_sustained"], 4),
                     "weight_stream_gbs": round(wbytes / us / 1e3, 1),
                     "frac_hbm": round(wbytes / us / 1e3 / peaks["hbm_gbs"], 4)})
    assert ctx.device_status() == AF.OK
    line = {"metric": f"MoE FFN throughput vs tokens (H={H}, I={I}, E={E}, top-{K})", "unit": "TFLOP/s", "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": f"moe ffn token sweep, config {cfg.cfg_id} routing, H={H}, I={I}, E={E}, K={K}",
                       "l2": "expert weights (2.8 GB) larger than L2, no flush"},
            "peaks": peaks, "clocks": sampler.stop(), "sweep": rows}
    print(json.dumps(line), flush=True)
    ctx.close()


def run_prefill_layers(args, cfg, local_rank, device, peaks):
    """Whole decoder layers over prompts (aflex_prefill_layers: the paper's PA and PF operators chained): L layers,
    each with its own weights and KV cache, over several prompt mixes.  One JSON line: time per layer, prompt
    tokens/s, TFLOP/s of the layer's algorithmic flops against the measured bf16 peaks, per-kernel times."""
    from paper_2608_01891_b200 import aflex as AF
    L = args.prefill_layers
    Hq, Hkv, D, H, I = cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, cfg.hidden, cfg.inter
    A, NQ = Hq * D, (Hq + 2 * Hkv) * D
    attn = AF.attn_desc(Hq, Hkv, D)
    weights = [IN.make_decoder_weights(cfg, l, device=device) for l in range(L)]
    cases = [("whole prompts 8 x 1024", [1024] * 8, None), ("whole prompts 4 x 4096", [4096] * 4, None),
             ("whole prompt 1 x 16384", [16384], None),
             ("chunk of 2048 onto 8192 cached, 2 sequences", [10240] * 2, [2048] * 2)]
    if args.prefill_case >= 0:
        cases = cases[args.prefill_case:args.prefill_case + 1]
    stream = torch.cuda.current_stream()
    sampler = ClockSampler(local_rank)
    sampler.start()
    rows, prof = [], {}
    for name, cached, new in cases:
        new = cached if new is None else new
        B = len(cached)
        c = dataclasses.replace(cfg, batch=B)
        kvh = IN.make_paged_kv(c, np.asarray(cached, dtype=np.int32), device=device)
        table, lens = kvh.page_table.to(device), kvh.seq_lens.to(device)
        descs, kvs, keep = [], [], []
        for l, w in enumerate(weights):
            layer = AF.layer_desc(attn, H, I, w.o, w.gate, w.up, w.down, cfg.num_experts, cfg.top_k, w.router)
            descs.append(AF.decoder_desc(layer, w.qkv, w.ln_attn, w.ln_ffn, w.q_norm, w.k_norm, cfg.rms_eps, cfg.rope_theta))
            kc, vc = (kvh.k_cache, kvh.v_cache) if l == 0 else (kvh.k_cache.clone(), kvh.v_cache.clone())
            kvs.append(AF.make_kv(kc, vc, table, lens, kvh.seq_lens))
            keep.append((kc, vc))
        qo = torch.zeros(B + 1, dtype=torch.int32)
        qo[1:] = torch.cumsum(torch.tensor(new, dtype=torch.int32), 0)
        qod = qo.to(device)
        T = int(qo[-1])
        x = IN.make_x(dataclasses.replace(cfg, num_experts=0), device=device, tokens=T)
        y = torch.empty_like(x)
        ctx = AF.Context(local_rank, max(AF.prefill_workspace_bytes(d, T) for d in descs))
        run = lambda: ctx.prefill_layers(descs, kvs, x, qod, qo, y, stream)
        for _ in range(max(3, args.warmup)):
            run()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.steps):
            run()
        e1.record(stream)
        torch.cuda.synchronize()
        us_layer = 1e3 * e0.elapsed_time(e1) / args.steps / L
        pairs = sum(m * (n - m) + m * (m + 1) // 2 for n, m in zip(cached, new))
        ffn_flops = 6.0 * T * H * I * (cfg.top_k if cfg.num_experts else 1)
        flops = 2.0 * T * H * NQ + 2.0 * T * A * H + ffn_flops + 4.0 * Hq * D * pairs
        tf = flops / us_layer / 1e6
        rows.append({"case": name, "prompt_tokens": T, "us_per_layer": round(us_layer, 1),
                     "tokens_per_s_per_layer": round(T / us_layer * 1e6), "tflops": round(tf, 1),
                     "frac_bf16_burst": round(tf / peaks["bf16_tflops"], 4),
                     "frac_bf16_sustained": round(tf / peaks["bf16_tflops_sustained"], 4)})
        ctx.profile_enable(True)
        for _ in range(3):
            run()
        pr = ctx.profile_read()
        ctx.profile_enable(False)
        prof[name] = {k: round(1e3 * v[0] / v[1], 1) for k, v in pr.items()}
        assert ctx.device_status() == AF.OK
        ctx.close()
        del kvh, kvs, keep, x, y
        torch.cuda.empty_cache()
    line = {"metric": "whole decoder layer over prompts (prefill): tokens/s per layer", "unit": "tokens/s", "dtype": "bf16",
            "data": "synthetic", "steps": args.steps, "warmup": max(3, args.warmup),
            "config": {"workload": f"config {cfg.cfg_id}: {cfg.name}, {L} chained layers over prompt tokens",
                       "l2": "per-layer weights and activations larger than L2, no flush"},
            "peaks": peaks, "clocks": sampler.stop(), "cases": rows, "kernel_us_event_pairs": prof}
    print(json.dumps(line), flush=True)


def run_decoder_chain(args, cfg, local_rank, device, peaks):
    """Whole decoder layers chained (aflex_decoder_layers): L layers, each with its own weights and KV cache,
    at every microbatch depth of the configuration.  One JSON line: time per layer, tokens/s, the share of the
    measured HBM bandwidth the layer's algorithmic bytes reach, and the per-kernel times of the M = 1 chain."""
    from paper_2608_01891_b200 import aflex as AF
    L = args.decoder_layers
    kvh = IN.make_paged_kv(cfg, device=device)
    table, lens = kvh.page_table.to(device), kvh.seq_lens.to(device)
    attn = AF.attn_desc(cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim)
    descs, kvs, keep = [], [], []
    for l in range(L):
        w = IN.make_decoder_weights(cfg, l, device=device)
        if args.af_pair and args.ffn_device >= 0 and args.ffn_device != local_rank:
            fdev = f"cuda:{args.ffn_device}"                 # role-specific weights: the FFN's live on the FFN GPU
            w.gate, w.up, w.down, w.ln_ffn = w.gate.to(fdev), w.up.to(fdev), w.down.to(fdev), w.ln_ffn.to(fdev)
            w.router = None if w.router is None else w.router.to(fdev)
        layer = AF.layer_desc(attn, cfg.hidden, cfg.inter, w.o, w.gate, w.up, w.down, cfg.num_experts, cfg.top_k, w.router)
        descs.append(AF.decoder_desc(layer, w.qkv, w.ln_attn, w.ln_ffn, w.q_norm, w.k_norm, cfg.rms_eps, cfg.rope_theta))
        kc, vc = (kvh.k_cache, kvh.v_cache) if l == 0 else (kvh.k_cache.clone(), kvh.v_cache.clone())
        kvs.append(AF.make_kv(kc, vc, table, lens, kvh.seq_lens))
        keep.append((w, kc, vc))
    x = IN.make_hidden(cfg, device=device)
    y = torch.empty_like(x)
    stream = torch.cuda.current_stream()
    if args.af_pair:
        # Attention side on this GPU, FFN side on --ffn-device (the same GPU by default: the hand-over copies are
        # then device-local and the two sides share one memory system)
        ctx = AF.Context(local_rank, max(AF.af_workspace_bytes(d, cfg.batch, False) for d in descs))
        ctx_f = AF.Context(args.ffn_device if args.ffn_device >= 0 else local_rank,
                           max(AF.af_workspace_bytes(d, cfg.batch, True) for d in descs))
        torch.cuda.set_device(local_rank)
        run = lambda M: AF.af_decoder_layers(ctx, ctx_f, descs, kvs, x, y, M, None, stream)
    else:
        ctx = AF.Context(local_rank, max(AF.decoder_workspace_bytes(d, cfg.batch) for d in descs))
        ctx_f = None
        run = lambda M: ctx.decoder_layers(descs, kvs, x, y, M, None, stream)
    n_qkv = (cfg.num_q_heads + 2 * cfg.num_kv_heads) * cfg.head_dim
    extra = 2.0 * n_qkv * cfg.hidden                      # W_qkv bytes on top of the hot path's
    sampler = ClockSampler(local_rank)
    sampler.start()
    rows = []
    for M in cfg.microbatch_depths:
        for _ in range(max(3, args.warmup)):
            run(M)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.steps):
            run(M)
        e1.record(stream)
        torch.cuda.synchronize()
        us_layer = 1e3 * e0.elapsed_time(e1) / args.steps / L
        byts = M * (sum(v for k, v in algorithmic_bytes(cfg, kvh.seq_lens.numpy(), M).items() if k != "gemm_chain") + extra)
        rows.append({"M": M, "us_per_layer": round(us_layer, 1), "tokens_per_s": round(cfg.batch / us_layer * 1e6),
                     "algorithmic_gbs": round(byts / us_layer / 1e3, 1),
                     "frac_hbm": round(byts / us_layer / 1e3 / peaks["hbm_gbs"], 4)})
    ctx.profile_enable(True)
    for _ in range(5):
        run(1)
    prof = ctx.profile_read()
    ctx.profile_enable(False)
    assert ctx.device_status() == AF.OK and (ctx_f is None or ctx_f.device_status() == AF.OK)
    line = {"metric": "whole decoder layer, chained: tokens/s per layer", "unit": "tokens/s", "dtype": "bf16",
            "data": "synthetic", "config": {"workload": f"config {cfg.cfg_id}: {cfg.name}, {L} chained decoder layers"
                                            + (f", A/F pair (attention GPU {local_rank}, FFN GPU "
                                               f"{args.ffn_device if args.ffn_device >= 0 else local_rank})" if args.af_pair else ""),
                                            "batch": cfg.batch, "l2": "per-layer weights + KV larger than L2, no flush"},
            "peaks": peaks, "clocks": sampler.stop(), "depths": rows,
            "kernel_us_event_pairs_M1": {k: round(1e3 * v[0] / v[1], 1) for k, v in prof.items()}}
    print(json.dumps(line), flush=True)
    ctx.close()
    if ctx_f is not None:
        ctx_f.close()


def run_targets(args, cfg, wl, ctx, local_rank, device, peaks, stream):
    """Figures for the stated targets that the timed configuration does not show by itself:
    dense FFN at the Qwen3-32B weight shape with 1024 and 2048 tokens (tensor-core bound: TFLOP/s against the
    measured burst and sustained bf16 peaks); decode attention at configuration 5's KV cache (5.4 GB: the
    steady-state streaming rate, against the measured copy bandwidth and the nominal 8 TB/s); the M = 1 layer
    step of configurations 3, 4 and 5 (time, tokens/s, algorithmic bytes per second against the measured copy
    bandwidth).  Every case: 3 warm-up calls, then CUDA events around n calls on the launching stream; all
    inputs of a case exceed L2."""
    from paper_2608_01891_b200 import aflex as AF

    def time_us(fn, n):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(n):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        return 1e3 * e0.elapsed_time(e1) / n

    out = {"ffn_dense_qwen3_32b_shape": [], "layer_step_m1": []}
    # (the memory-bound layer steps first: the dense FFN at 1 K - 2 K tokens drives the board into its power cap, and a
    #  step timed right behind it would be timed at the clocks it leaves)
    for cid in (3, 4, 5):
        c = IN.CONFIGS[cid]
        w = wl if cid == cfg.cfg_id else build_workload(c, device)
        lens = w["kvh"].seq_lens.numpy()
        cx = ctx if cid == cfg.cfg_id else AF.Context(local_rank, AF.workspace_bytes(w["layer"], c.batch, w["kvh"].max_pages_per_seq))
        cx.set_attn_q_final(True)
        us = time_us(lambda: cx.layer_step(w["layer"], w["q"], w["kv"], w["y"], 1, None, w["logits"], None, stream), 40)
        byts = sum(v for k, v in algorithmic_bytes(c, lens, 1).items() if k != "gemm_chain")
        out["layer_step_m1"].append({"config": cid, "batch": c.batch, "us": round(us, 1), "tokens_per_s": round(c.batch / us * 1e6),
                                     "algorithmic_gbs": round(byts / us / 1e3, 1),
                                     "frac_hbm_measured": round(byts / us / 1e3 / peaks["hbm_gbs"], 4)})
        if cid == 5:
            a_out = torch.empty_like(w["q"])
            us = time_us(lambda: cx.attn_decode(w["layer"].attn, w["q"], w["kv"], a_out, None, stream), 20)
            kvb = algorithmic_bytes(c, lens, 1)["attn_decode"]
            out["attn_decode_steady_state"] = {"config": 5, "kv_bytes": int(kvb), "us": round(us, 1), "gbs": round(kvb / us / 1e3, 1),
                                               "frac_hbm_measured": round(kvb / us / 1e3 / peaks["hbm_gbs"], 4),
                                               "frac_hbm_nominal_8tbs": round(kvb / us / 1e3 / 8000.0, 4)}
        assert cx.device_status() == AF.OK
        if cx is not ctx:
            cx.close()
            del w
            torch.cuda.empty_cache()
    dense = IN.CONFIGS[2]
    if cfg.cfg_id in (2, 3):
        wg, wu, wd = wl["wg"], wl["wu"], wl["wd"]
    else:
        wg, wu, wd = IN.make_ffn_weights(dense, device=device)
    big = AF.Context(local_rank, 6 << 30)
    H, I = dense.hidden, dense.inter
    for T in (1024, 2048):
        x = IN.make_x(dense, device=device, tokens=T)
        y = torch.empty(T, H, dtype=torch.bfloat16, device=device)
        us = time_us(lambda: big.ffn_dense(x, wg, wu, wd, y, stream), 10)
        tf = 6.0 * T * H * I / us / 1e6
        out["ffn_dense_qwen3_32b_shape"].append({"T": T, "us": round(us, 1), "tflops": round(tf, 1),
                                                 "frac_bf16_burst": round(tf / peaks["bf16_tflops"], 4),
                                                 "frac_bf16_sustained": round(tf / peaks["bf16_tflops_sustained"], 4)})
    assert big.device_status() == AF.OK
    big.close()
    del wg, wu, wd
    return out


def run_plan(args, cfg, local_rank, device, peaks):
    """The planner of Section 4.3 ("dynamic microbatch depth", "adaptive request batching") fed with stage-time curves
    MEASURED on this GPU, and its predictions set against measured chain times.

    1. t_F(rows): the FFN side alone (aflex_ffn_dense / aflex_ffn_moe, back to back) at several row counts.
    2. t_layer(sub-batch): aflex_decoder_layers at depth 1 on sub-batches (prefixes of the batch, its shortest and
       its longest sequences); t_A = t_layer - t_F(rows), fitted by least squares as a0 + a1 * context tokens +
       a2 * rows, which gives the model's two attention curves.
    3. aflex_pipeline_model with shared_memory_system = 1 (one GPU); for every depth of the configuration
       aflex_pipeline_makespan's prediction for the near-equal split next to the measured chain time.
    4. aflex_plan_microbatches: the depth / split it picks over all depths, and the best split at depth 2 alone;
       both run, and the equal split at depth 2 beside it."""
    from paper_2608_01891_b200 import aflex as AF
    L = max(2, args.decoder_layers or 4)
    B = cfg.batch
    kvh = IN.make_paged_kv(cfg, device=device)
    lens_all = kvh.seq_lens.numpy().astype(np.int64)
    table_d = kvh.page_table.to(device)
    attn = AF.attn_desc(cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim)
    descs, caches, keep = [], [], []
    for l in range(L):
        w = IN.make_decoder_weights(cfg, l, device=device)
        layer = AF.layer_desc(attn, cfg.hidden, cfg.inter, w.o, w.gate, w.up, w.down, cfg.num_experts, cfg.top_k, w.router)
        descs.append(AF.decoder_desc(layer, w.qkv, w.ln_attn, w.ln_ffn, w.q_norm, w.k_norm, cfg.rms_eps, cfg.rope_theta))
        caches.append((kvh.k_cache, kvh.v_cache) if l == 0 else (kvh.k_cache.clone(), kvh.v_cache.clone()))
        keep.append(w)
    ctx = AF.Context(local_rank, max(max(AF.decoder_workspace_bytes(d, B) for d in descs), 1 << 30))
    stream = torch.cuda.current_stream()
    x_all = IN.make_hidden(cfg, device=device)

    def time_us(fn, n):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(n):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        return 1e3 * e0.elapsed_time(e1) / n

    def chain_us(rows_idx, M, offsets=None):
        """Microseconds per layer of the chain over the sequences rows_idx (in that order)."""
        idx = torch.as_tensor(np.asarray(rows_idx, dtype=np.int64))
        tab = table_d.index_select(0, idx.to(device))
        ln_h = kvh.seq_lens.index_select(0, idx).contiguous()
        ln_d = ln_h.to(device)
        kvs = [AF.make_kv(kc, vc, tab, ln_d, ln_h) for kc, vc in caches]
        x = x_all.index_select(0, idx.to(device)).contiguous()
        y = torch.empty_like(x)
        us = time_us(lambda: ctx.decoder_layers(descs, kvs, x, y, M, offsets, stream), max(5, args.steps // 4))
        return us / L

    # ---- 1. FFN curve
    w0 = keep[0]
    f_rows = sorted({r for r in (8, 16, 32, 64, 128, 256, B // 4, B // 3, B // 2, B) if 1 <= r <= B})
    f_us = []
    for r in f_rows:
        x = x_all[:r].contiguous()
        y = torch.empty_like(x)
        if cfg.num_experts == 0:
            f_us.append(time_us(lambda: ctx.ffn_dense(x, w0.gate, w0.up, w0.down, y, stream), 20))
        else:
            f_us.append(time_us(lambda: ctx.ffn_moe(x, w0.gate, w0.up, w0.down, cfg.top_k, y, w_router=w0.router, stream=stream), 20))
    t_f = lambda r: float(np.interp(r, f_rows, f_us))

    # ---- 2. attention-side fit from depth-1 chain times on sub-batches
    order = np.argsort(lens_all)
    subs = []
    for r in sorted({max(1, B // 8), max(1, B // 4), max(1, B // 2), max(1, 3 * B // 4), B}):
        subs.append(list(range(r)))
        if r < B:
            subs.append(order[:r].tolist())
            subs.append(order[-r:].tolist())
    rows_fit, tok_fit, ta_fit, meas_fit = [], [], [], []
    for sub in subs:
        us = chain_us(sub, 1)
        rows_fit.append(len(sub)); tok_fit.append(int(lens_all[sub].sum())); meas_fit.append(us)
        ta_fit.append(us - t_f(len(sub)))
    A = np.stack([np.ones(len(subs)), np.asarray(tok_fit, float), np.asarray(rows_fit, float)], axis=1)
    coef, *_ = np.linalg.lstsq(A, np.asarray(ta_fit), rcond=None)
    a0, a1, a2 = (float(c) for c in coef)
    fit_err = float(np.max(np.abs(A @ coef - np.asarray(ta_fit)) / np.asarray(meas_fit)))
    tok_hi = float(lens_all.sum())
    model = AF.pipeline_model(([0.0, tok_hi], [a0, a0 + a1 * tok_hi]), ([0.0, float(B)], [0.0, a2 * B]),
                              ([float(r) for r in f_rows], f_us), 0.0, 0.0, True)

    # ---- 3. prediction against measurement, near-equal splits
    def equal_offsets(M):
        base, extra = divmod(B, M)
        o = [0]
        for i in range(M):
            o.append(o[-1] + base + (1 if i < extra else 0))
        return o

    lens_list = lens_all.tolist()
    depth_rows = []
    for M in sorted(set(cfg.microbatch_depths) | {1, 2, 3, 4}):
        if M > B:
            continue
        offs = equal_offsets(M)
        pred = AF.pipeline_makespan(model, lens_list, offs, L) / L
        meas = chain_us(list(range(B)), M, offs)
        depth_rows.append({"M": M, "offsets": offs, "predicted_us_per_layer": round(pred, 1), "measured_us_per_layer": round(meas, 1),
                           "error": round(pred / meas - 1.0, 4)})

    # ---- 4. what the planner picks
    gran = max(1, B // 16)
    M_best, offs_best, pred_best = AF.plan_microbatches(model, lens_list, L, [1, 2, 3, 4], gran)
    meas_best = chain_us(list(range(B)), M_best, offs_best)
    _, offs2, pred2 = AF.plan_microbatches(model, lens_list, L, [2], gran)
    meas2 = chain_us(list(range(B)), 2, offs2)
    meas2_eq = next(r["measured_us_per_layer"] for r in depth_rows if r["M"] == 2)
    assert ctx.device_status() == AF.OK
    line = {"metric": "planner prediction against measured chain time", "unit": "us per layer", "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"config {cfg.cfg_id}: {cfg.name}, {L} chained decoder layers, one GPU (shared memory system)",
                       "batch": B},
            "ffn_curve": {"rows": f_rows, "us": [round(v, 1) for v in f_us]},
            "attention_fit": {"a0_us": round(a0, 2), "us_per_1k_context_tokens": round(a1 * 1e3, 3), "us_per_row": round(a2, 3),
                              "sub_batches": len(subs), "max_fit_error_of_layer_time": round(fit_err, 4)},
            "depths": depth_rows,
            "plan_all_depths": {"M": M_best, "offsets": offs_best, "predicted_us_per_layer": round(pred_best / L, 1),
                                "measured_us_per_layer": round(meas_best, 1)},
            "plan_depth_2": {"offsets": offs2, "predicted_us_per_layer": round(pred2 / L, 1), "measured_us_per_layer": round(meas2, 1),
                             "equal_split_measured_us_per_layer": meas2_eq}}
    print(json.dumps(line), flush=True)
    ctx.close()


def af_pair_devices(world: int, rank: int, local_rank: int, device_count: int):
    """Which GPUs the A/F pair measurement uses in a multi-GPU run: rank 0 alone drives it, with the Attention side on
    its own GPU and the FFN side on the next local one; every other rank only waits.  Returns (attention device, FFN
    device) for the rank that runs it, None for the ranks that wait, and a reason string when nobody runs it."""
    if world < 2:
        return "one GPU: not run (the pair needs two devices; both sides on one GPU are covered by the tests)"
    if device_count < 2:
        return "fewer than two visible devices: not run"
    if rank != 0:
        return None
    return (local_rank, (local_rank + 1) % device_count)


def wait_for_rank0(dist, host_group):
    """Host-side rendezvous (gloo) behind the replica timing: the other ranks block here, off the GPU, while rank 0
    measures the A/F pair on its own GPU and its neighbour's."""
    dist.barrier(group=host_group)


def run_af_pair_record(cfg, dev_a: int, dev_f: int, L: int, steps: int):
    """One A/F pair inside a node (the paper's data plane, Section 4.3): Attention side on GPU dev_a, FFN side on GPU
    dev_f, hidden states handed over by peer copies.  Per microbatch depth: microseconds per layer, checked bit for bit
    against the same call with both contexts on dev_a; the measured time of one hand-over copy; Eq. 2's prediction
    with the measured per-side kernel times and that t_comm."""
    from paper_2608_01891_b200 import aflex as AF
    da, df = f"cuda:{dev_a}", f"cuda:{dev_f}"
    torch.cuda.set_device(dev_a)
    kvh = IN.make_paged_kv(cfg, device=da)
    table, lens = kvh.page_table.to(da), kvh.seq_lens.to(da)
    attn = AF.attn_desc(cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim)
    descs_pair, descs_one, kvs, keep = [], [], [], []
    for l in range(L):
        w = IN.make_decoder_weights(cfg, l, device=da)
        f_side = [w.gate, w.up, w.down, w.ln_ffn, w.router]
        f_far = [None if t is None else t.to(df) for t in f_side] if dev_f != dev_a else f_side
        one = AF.layer_desc(attn, cfg.hidden, cfg.inter, w.o, w.gate, w.up, w.down, cfg.num_experts, cfg.top_k, w.router)
        far = AF.layer_desc(attn, cfg.hidden, cfg.inter, w.o, f_far[0], f_far[1], f_far[2], cfg.num_experts, cfg.top_k, f_far[4])
        descs_one.append(AF.decoder_desc(one, w.qkv, w.ln_attn, w.ln_ffn, w.q_norm, w.k_norm, cfg.rms_eps, cfg.rope_theta))
        descs_pair.append(AF.decoder_desc(far, w.qkv, w.ln_attn, f_far[3], w.q_norm, w.k_norm, cfg.rms_eps, cfg.rope_theta))
        kc, vc = (kvh.k_cache, kvh.v_cache) if l == 0 else (kvh.k_cache.clone(), kvh.v_cache.clone())
        kvs.append(AF.make_kv(kc, vc, table, lens, kvh.seq_lens))
        keep.append((w, f_far, kc, vc))
    x = IN.make_hidden(cfg, device=da)
    y_pair, y_one = torch.empty_like(x), torch.empty_like(x)
    ctx_a = AF.Context(dev_a, max(AF.af_workspace_bytes(d, cfg.batch, False) for d in descs_pair))
    ctx_f = AF.Context(dev_f, max(AF.af_workspace_bytes(d, cfg.batch, True) for d in descs_pair))
    ctx_f1 = AF.Context(dev_a, max(AF.af_workspace_bytes(d, cfg.batch, True) for d in descs_one))
    torch.cuda.set_device(dev_a)
    stream = torch.cuda.current_stream()

    def time_us(fn, n):
        for _ in range(3):
            fn()
        torch.cuda.synchronize(dev_a); torch.cuda.synchronize(dev_f)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(n):
            fn()
        e1.record(stream)
        torch.cuda.synchronize(dev_a); torch.cuda.synchronize(dev_f)
        return 1e3 * e0.elapsed_time(e1) / n

    rows = []
    for M in (1, 2, 4):
        if M > cfg.batch:
            continue
        AF.af_decoder_layers(ctx_a, ctx_f1, descs_one, kvs, x, y_one, M, None, stream)      # both sides on dev_a
        torch.cuda.synchronize(dev_a)
        AF.af_decoder_layers(ctx_a, ctx_f, descs_pair, kvs, x, y_pair, M, None, stream)     # the pair
        torch.cuda.synchronize(dev_a); torch.cuda.synchronize(dev_f)
        same = bool(torch.equal(y_one.view(torch.int16), y_pair.view(torch.int16)))
        us = time_us(lambda: AF.af_decoder_layers(ctx_a, ctx_f, descs_pair, kvs, x, y_pair, M, None, stream), steps) / L
        # per-side kernel time of one layer (event pair around every launch; no overlap counted)
        ctx_a.profile_enable(True); ctx_f.profile_enable(True)
        AF.af_decoder_layers(ctx_a, ctx_f, descs_pair, kvs, x, y_pair, M, None, stream)
        torch.cuda.synchronize(dev_a); torch.cuda.synchronize(dev_f)
        t_a = 1e3 * sum(v[0] for v in ctx_a.profile_read().values()) / L
        torch.cuda.set_device(dev_f)
        t_f = 1e3 * sum(v[0] for v in ctx_f.profile_read().values()) / L
        torch.cuda.set_device(dev_a)
        ctx_a.profile_enable(False); ctx_f.profile_enable(False)
        # one hand-over: [rows of a microbatch][H] bf16 from the attention GPU into the FFN GPU's memory
        r = -(-cfg.batch // M)
        src = torch.empty(r, cfg.hidden, dtype=torch.bfloat16, device=da)
        dst = torch.empty(r, cfg.hidden, dtype=torch.bfloat16, device=df)
        # (20 copies captured into a CUDA graph, so that the device time of a copy is measured, not the host's issue rate)
        g = torch.cuda.CUDAGraph()
        cap = torch.cuda.Stream(device=da)
        cap.wait_stream(stream)
        with torch.cuda.graph(g, stream=cap):
            for _ in range(20):
                dst.copy_(src, non_blocking=True)
        stream.wait_stream(cap)
        t_copy = time_us(g.replay, 10) / 20
        t_comm = 2.0 * M * t_copy                          # Eq. 2's t_comm: the whole batch, both directions
        rows.append({"M": M, "us_per_layer": round(us, 1), "bit_identical_to_one_gpu_pair": same,
                     "t_a_us": round(t_a, 1), "t_f_us": round(t_f, 1), "copy_us_per_boundary": round(t_copy, 2),
                     "eq2_prediction_us": round(AF.eq2_layer_time(t_a, t_f, t_comm, M), 1)})
    ok = ctx_a.device_status() == AF.OK
    torch.cuda.set_device(dev_f)
    ok = ok and ctx_f.device_status() == AF.OK
    torch.cuda.set_device(dev_a)
    for c in (ctx_f1, ctx_f, ctx_a):
        c.close()
    return {"config": cfg.cfg_id, "layers": L, "attention_gpu": dev_a, "ffn_gpu": dev_f, "device_status_ok": ok,
            "transfer": "cudaMemcpyPeerAsync into the consumer's own memory; no kernel reads peer memory", "depths": rows}


def dataclasses_replace_dense(cfg):
    """The configuration's FFN shape as a dense FFN (MoE configurations: one expert's shape)."""
    import dataclasses
    return dataclasses.replace(cfg, num_experts=0, top_k=0)


def build_workload(cfg, device):
    """Everything resident in HBM before the timed region starts."""
    from paper_2608_01891_b200 import aflex as AF
    kvh = IN.make_paged_kv(cfg, device=device)
    q = IN.make_q(cfg, device=device)
    wo = IN.make_wo(cfg, device=device)
    wg, wu, wd = IN.make_ffn_weights(cfg, device=device)
    logits = IN.make_router_logits(cfg).to(device) if cfg.num_experts else None
    table = kvh.page_table.to(device)
    lens = kvh.seq_lens.to(device)
    kv = AF.make_kv(kvh.k_cache, kvh.v_cache, table, lens, kvh.seq_lens)
    layer = AF.layer_desc(AF.attn_desc(cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim), cfg.hidden, cfg.inter,
                          wo, wg, wu, wd, cfg.num_experts, cfg.top_k)
    y = torch.zeros(cfg.batch, cfg.hidden, dtype=torch.bfloat16, device=device)
    return dict(kvh=kvh, q=q, wo=wo, wg=wg, wu=wu, wd=wd, logits=logits, table=table, lens=lens, kv=kv,
                layer=layer, y=y)


def oracle_sample(cfg, wl, rows):
    """Time the fp64 oracle's layer step on the sampled batch rows.  Returns (seconds, threads)."""
    from oracle import oracle as O
    kvh = wl["kvh"]
    table, lens = kvh.page_table.numpy(), kvh.seq_lens.numpy()
    ids, new_rows, o = [], [], 0
    mp = max((int(lens[b]) + 15) // 16 for b in rows)
    for b in rows:
        n = (int(lens[b]) + 15) // 16
        ids.extend(table[b, :n].tolist())
        r = np.zeros(mp, dtype=np.int32); r[:n] = np.arange(o, o + n); new_rows.append(r); o += n
    sel = torch.as_tensor(np.asarray(ids, dtype=np.int64), device=kvh.k_cache.device)
    u16 = lambda t: IN.bf16_bits(t.detach().cpu().contiguous())
    k, v = u16(kvh.k_cache.index_select(0, sel)), u16(kvh.v_cache.index_select(0, sel))
    q = u16(wl["q"][list(rows)])
    wo, wg, wu, wd = u16(wl["wo"]), u16(wl["wg"]), u16(wl["wu"]), u16(wl["wd"])
    logits = wl["logits"][list(rows)].cpu().numpy() if cfg.num_experts else None
    t0 = time.perf_counter()
    O.layer_step(q, k, v, np.stack(new_rows), lens[list(rows)].astype(np.int32), wo, wg, wu, wd,
                 logits=logits, top_k=cfg.top_k)
    return time.perf_counter() - t0, O.num_threads()


def run_reference(args, cfg, rank, world):
    """The CPU oracle as the reference arm: each step is a bounded sample of the workload."""
    if rank != 0:
        return
    wl_cfg = cfg
    kvh = IN.make_paged_kv(wl_cfg)
    wl = dict(kvh=kvh, q=IN.make_q(wl_cfg), wo=IN.make_wo(wl_cfg), logits=IN.make_router_logits(wl_cfg) if wl_cfg.num_experts else None)
    wl["wg"], wl["wu"], wl["wd"] = IN.make_ffn_weights(wl_cfg)
    rows = list(range(min(args.ref_rows, cfg.batch)))
    times, threads = [], 1
    for i in range(args.warmup + args.steps):
        dt, threads = oracle_sample(cfg, wl, rows)
        if i >= args.warmup:
            times.append(dt)
    ms = 1e3 * float(np.mean(times))
    value = len(rows) / (ms * 1e-3)
    sample = f"layer step on batch rows {rows[0]}..{rows[-1]} of {cfg.batch} (rows are independent)"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"config {cfg.cfg_id}: {cfg.name}", "batch": cfg.batch, "microbatch_depth": 1,
                       "sampled_rows": len(rows)},
            "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, choices=[1, 2, 3, 4, 5])
    ap.add_argument("--depth", type=int, default=1, help="microbatch depth M")
    ap.add_argument("--attn-ctas", type=int, default=0, help="persistent attention CTAs (0 = two per SM)")
    ap.add_argument("--ref-rows", type=int, default=0,
                    help="batch rows per reference/cpu-baseline sample (0 = about 15e9 multiply-adds of oracle work)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--quick", action="store_true",
                    help="only the warm-up and the timed steps of the layer step, then a short JSON line (value, ms_per_step, "
                         "gpu_launches): a small run with few launches, for a profiler")
    ap.add_argument("--ffn-sweep", action="store_true",
                    help="instead of the layer step: dense FFN (aflex_ffn_dense) at the configuration's weight shape "
                         "for T = 32..8192 tokens, TFLOP/s against the measured bf16 peak; prints one JSON line")
    ap.add_argument("--ffn-tokens", type=int, default=0, help="with --ffn-sweep: only this token count")
    ap.add_argument("--decoder-layers", type=int, default=0,
                    help="instead of the layer step: chain this many whole decoder layers (aflex_decoder_layers) at "
                         "every microbatch depth of the configuration; prints one JSON line")
    ap.add_argument("--af-pair", action="store_true",
                    help="with --decoder-layers: run the Attention side and the FFN side as an A/F pair "
                         "(aflex_af_decoder_layers), hidden states handed over by peer copies")
    ap.add_argument("--ffn-device", type=int, default=-1,
                    help="with --af-pair: CUDA device of the FFN side (default: the same GPU as the attention side)")
    ap.add_argument("--energy-ops", action="store_true",
                    help="instead of the layer step: time and NVML energy per token of attention, the dense FFN at "
                         "T = 32 and T = 2048 and the layer step, each alone, at the clocks the GPU is found at")
    ap.add_argument("--af-pair-record", type=int, default=-1, metavar="FFN_GPU",
                    help="instead of the layer step: the A/F pair record of the multi-GPU run (configuration 3, 4 layers, "
                         "depths 1 / 2 / 4) with the attention side on this GPU and the FFN side on GPU FFN_GPU (the "
                         "same GPU is allowed); prints one JSON line")
    ap.add_argument("--plan", action="store_true",
                    help="instead of the layer step: measure the stage-time curves of the configuration on this GPU, feed "
                         "them to aflex_plan_microbatches / aflex_pipeline_makespan and set the predictions against "
                         "measured aflex_decoder_layers times at every depth; prints one JSON line")
    ap.add_argument("--prefill", action="store_true",
                    help="instead of the layer step: prefill (causal) attention at the configuration's head shape over "
                         "several prompt mixes, TFLOP/s against the measured bf16 peaks")
    ap.add_argument("--prefill-layers", type=int, default=0,
                    help="instead of the layer step: this many whole decoder layers chained over prompt tokens "
                         "(aflex_prefill_layers), several prompt mixes")
    ap.add_argument("--prefill-case", type=int, default=-1,
                    help="with --prefill / --prefill-layers: run only this case of the list (a small single-kernel run for a profiler)")
    ap.add_argument("--no-energy", action="store_true",
                    help="skip the NVML energy reading (joules per token around a >= 2 s loop of the step, at the clocks "
                         "the GPU is found at; read-only)")
    ap.add_argument("--no-targets", action="store_true",
                    help="skip the 'targets' sub-record (steady-state attention at configuration 5, the dense FFN at "
                         "1024 / 2048 tokens, the M = 1 step of configurations 3-5)")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3

    if args.ref_rows <= 0:
        c = IN.CONFIGS[args.config]
        macs_row = (c.num_q_heads * c.head_dim * (2 * (c.len_lo + c.len_hi) // 2 + c.hidden)
                    + 3 * c.hidden * c.inter * max(1, c.top_k))
        args.ref_rows = int(max(1, min(c.batch, 15e9 // macs_row)))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    cfg = IN.CONFIGS[args.config]

    if args.impl == "reference":
        run_reference(args, cfg, rank, world)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    from paper_2608_01891_b200 import aflex as AF
    torch.cuda.set_device(local_rank)
    device = f"cuda:{local_rank}"
    dist = None
    host_group = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(device))
        host_group = dist.new_group(backend="gloo")       # host-side rendezvous for the part only rank 0 runs

    peaks = load_peaks()
    if args.ffn_sweep:
        if rank == 0:
            (run_moe_sweep if cfg.num_experts > 0 else run_ffn_sweep)(args, cfg, local_rank, device, peaks)
        return
    if args.decoder_layers > 0 and not args.plan:
        if rank == 0:
            run_decoder_chain(args, cfg, local_rank, device, peaks)
        return
    if args.energy_ops:
        if rank == 0:
            run_energy_ops(args, cfg, local_rank, device, peaks)
        return
    if args.plan:
        if rank == 0:
            run_plan(args, cfg, local_rank, device, peaks)
        return
    if args.af_pair_record >= 0:
        if rank == 0:
            print(json.dumps({"metric": "A/F pair across GPUs: us per decoder layer", "unit": "us", "dtype": "bf16",
                              "data": "synthetic", "af_pair": run_af_pair_record(IN.CONFIGS[3 if args.config == 2 else args.config],
                                                                                  local_rank, args.af_pair_record, 4, args.steps // 5 or 5)}), flush=True)
        return
    if args.prefill:
        if rank == 0:
            run_prefill(args, cfg, local_rank, device, peaks)
        return
    if args.prefill_layers > 0:
        if rank == 0:
            run_prefill_layers(args, cfg, local_rank, device, peaks)
        return
    wl = build_workload(cfg, device)
    lens_np = wl["kvh"].seq_lens.numpy()
    M = args.depth
    ws = AF.workspace_bytes(wl["layer"], cfg.batch, wl["kvh"].max_pages_per_seq)
    ctx = AF.Context(local_rank, ws)
    # q is a resident tensor (value) or arrives by a host-to-device copy (e2e), never as the output of the library
    # kernel enqueued just before the step: the documented promise that lets attention read it with its other inputs
    ctx.set_attn_q_final(True)
    if args.attn_ctas:
        ctx.set_attn_ctas(args.attn_ctas)
    stream = torch.cuda.current_stream()

    def step():
        ctx.layer_step(wl["layer"], wl["q"], wl["kv"], wl["y"], M, None, wl["logits"], None, stream)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps):
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            fn()
        e1.record(stream)
        barrier()
        return max_over_ranks(e0.elapsed_time(e1), dist, device)

    # ---- device-resident timing (the headline value)
    for _ in range(args.warmup):
        step()
    launches0 = ctx.launch_count()
    sampler = ClockSampler(local_rank)
    sampler.start()
    ms_total = timed(step, args.steps)
    launches = ctx.launch_count() - launches0
    if args.quick:
        sampler.stop()
        torch.cuda.synchronize()
        assert ctx.device_status() == AF.OK, ctx.last_error()
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": whole_job_tokens_per_s(world, cfg.batch, ms_total / args.steps),
                              "unit": "tokens/s", "ms_per_step": ms_total / args.steps, "steps": args.steps, "warmup": args.warmup,
                              "gpu_launches": int(launches), "config": {"workload": f"config {cfg.cfg_id}: {cfg.name}", "quick": True}}),
                  flush=True)
        ctx.close()
        if dist is not None:
            dist.destroy_process_group()
        return
    # the timed region can be shorter than one nvidia-smi sampling period: keep the same load
    # running (untimed) until the sampler has seen it
    if ms_total < 500:
        timed(step, int(500 / max(ms_total / args.steps, 1e-3)) + 1)
    clocks = sampler.stop()
    ms_step = ms_total / args.steps
    value = whole_job_tokens_per_s(world, cfg.batch, ms_step)
    assert ctx.device_status() == AF.OK, ctx.last_error()

    # ---- per-kernel durations: the same K steps with an event pair around every launch
    psteps = max(1, min(args.steps, 8192 // max(1, launches // args.steps)))
    ctx.profile_enable(True)
    timed(step, psteps)
    prof = ctx.profile_read()
    ctx.profile_enable(False)
    abytes = algorithmic_bytes(cfg, lens_np, M)
    aflops = algorithmic_flops(cfg, M)
    kernels = {}
    for name, (ms, n) in prof.items():
        avg_us = 1e3 * ms / n
        k = {"launches_per_step": n // psteps, "avg_us": round(avg_us, 2)}
        if name in abytes:
            k["gbs"] = round(abytes[name] / (avg_us * 1e-6) / 1e9, 1)
            k["frac_hbm"] = round(k["gbs"] / peaks["hbm_gbs"], 4)
        if name in aflops:
            k["tflops"] = round(aflops[name] / (avg_us * 1e-6) / 1e12, 2)
        kernels[name] = k
    dom = max((n for n in kernels if "gbs" in kernels[n]), key=lambda n: kernels[n]["avg_us"] * kernels[n]["launches_per_step"])
    roofline = {"kernel": dom, "bound": "hbm", "achieved": kernels[dom]["gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": kernels[dom]["frac_hbm"], "traffic": None, "peak_source": peaks["source"],
                "algorithmic_bytes_per_launch": abytes[dom]}
    ncu_traffic = os.path.join(ROOT, "profiles", "traffic.json")
    if os.path.exists(ncu_traffic):
        tr = json.load(open(ncu_traffic))
        key = f"config{cfg.cfg_id}/{dom}"
        if key in tr:
            # one single-kernel, single-launch ncu capture of this kernel on this workload; the record says which
            # commit's kernels were captured and how
            roofline["traffic"] = tr[key]["bytes"]
            roofline["traffic_source"] = {k: tr[key][k] for k in ("kernels_at_commit", "capture", "summary")}

    # ---- the two operators on their own: back-to-back calls of the public entry points over TWO alternating buffer
    #      sets (two copies of the KV cache for attention, two copies of the FFN weights), so that no launch can find
    #      lines its predecessor left in the 126 MB L2.  With programmatic dependent launch a call's ramp overlaps
    #      its predecessor's tail, so these are the streaming rates the step is built from; "us_event_pair" is the
    #      same call bracketed by an event pair (no overlap with a neighbour), from the per-kernel pass above.
    operators = {}
    if True:      # every rank: timed() holds the ranks' barrier
        a_out = torch.empty_like(wl["q"])
        x_ffn = IN.make_x(cfg, device=device)
        y_ffn = torch.empty_like(x_ffn)
        kv_sets = [wl["kv"], AF.make_kv(wl["kvh"].k_cache.clone(), wl["kvh"].v_cache.clone(), wl["table"], wl["lens"],
                                        wl["kvh"].seq_lens)]
        w_sets = [(wl["wg"], wl["wu"], wl["wd"]), (wl["wg"].clone(), wl["wu"].clone(), wl["wd"].clone())]
        keep_alive = kv_sets, w_sets
        turn = [0, 0]

        def attn_alone():
            turn[0] ^= 1
            ctx.attn_decode(wl["layer"].attn, wl["q"], kv_sets[turn[0]], a_out, None, stream)

        def ffn_alone():
            turn[1] ^= 1
            wg, wu, wd = w_sets[turn[1]]
            if cfg.num_experts == 0:
                ctx.ffn_dense(x_ffn, wg, wu, wd, y_ffn, stream)
            else:
                ctx.ffn_moe(x_ffn, wg, wu, wd, cfg.top_k, y_ffn, router_logits=wl["logits"], stream=stream)

        for name, fn in (("attn_decode", attn_alone), ("ffn", ffn_alone)):
            for _ in range(4):
                fn()
            us = 1e3 * timed(fn, args.steps) / args.steps
            ab1, fl1 = algorithmic_bytes(cfg, lens_np, 1), algorithmic_flops(cfg, 1)     # these calls take the whole batch at once
            if name == "attn_decode":
                byts = ab1["attn_decode"]
                operators[name] = {"us": round(us, 2), "gbs": round(byts / us / 1e3, 1),
                                   "frac_hbm_measured": round(byts / us / 1e3 / peaks["hbm_gbs"], 4),
                                   "frac_hbm_nominal_8tbs": round(byts / us / 1e3 / 8000.0, 4),
                                   "buffers": "two KV caches, alternating (each larger than L2)"}
                if M == 1 and "attn_decode" in kernels:
                    ep = kernels["attn_decode"]["avg_us"]
                    operators[name]["us_event_pair_in_step"] = ep
                    operators[name]["frac_hbm_nominal_8tbs_event_pair"] = round(byts / ep / 1e3 / 8000.0, 4)
            else:
                g, d = ("gateup_gemm", "down_gemm") if cfg.num_experts == 0 else ("moe_gateup_gemm", "moe_down_gemm")
                byts, fl = ab1[g] + ab1[d], fl1[g] + fl1[d]
                operators[name] = {"us": round(us, 2), "weight_stream_gbs": round(byts / us / 1e3, 1),
                                   "frac_hbm_measured": round(byts / us / 1e3 / peaks["hbm_gbs"], 4),
                                   "tflops": round(fl / us / 1e6, 1), "frac_bf16_burst": round(fl / us / 1e6 / peaks["bf16_tflops"], 4),
                                   "buffers": "two weight sets, alternating (each larger than L2)"}
        del kv_sets, w_sets, keep_alive
        torch.cuda.empty_cache()

    # ---- end to end: per-step inputs come from pinned host memory, the result goes back.
    # The per-step inputs (q, page table, sequence lengths, router logits) are packed into one pinned
    # staging buffer and travel in ONE host-to-device copy into one device buffer the tensors are views of.
    def carve(total_specs):
        off, out = 0, []
        for shape, dtype in total_specs:
            n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
            out.append((off, n, shape, dtype))
            off = (off + n + 255) & ~255
        return off, out
    specs = [(tuple(wl["q"].shape), torch.bfloat16), (tuple(wl["kvh"].page_table.shape), torch.int32),
             (tuple(wl["kvh"].seq_lens.shape), torch.int32)]
    if wl["logits"] is not None:
        specs.append((tuple(wl["logits"].shape), torch.float32))
    nbytes, layout = carve(specs)
    host_blob = torch.empty(nbytes, dtype=torch.uint8).pin_memory()
    dev_blob = torch.empty(nbytes, dtype=torch.uint8, device=device)
    views_h = [host_blob[o:o + n].view(dt).view(sh) for o, n, sh, dt in layout]
    views_d = [dev_blob[o:o + n].view(dt).view(sh) for o, n, sh, dt in layout]
    views_h[0].copy_(wl["q"].cpu()); views_h[1].copy_(wl["kvh"].page_table); views_h[2].copy_(wl["kvh"].seq_lens)
    if wl["logits"] is not None:
        views_h[3].copy_(wl["logits"].cpu())
    dq, dtab, dlens = views_d[0], views_d[1], views_d[2]
    dlog = views_d[3] if wl["logits"] is not None else None
    kv_e2e = AF.make_kv(wl["kvh"].k_cache, wl["kvh"].v_cache, dtab, dlens, wl["kvh"].seq_lens)
    hy = torch.empty(cfg.batch, cfg.hidden, dtype=torch.bfloat16).pin_memory()
    h2d = sum(n for _, n, _, _ in layout)
    d2h = hy.numel() * 2

    def step_e2e():
        dev_blob.copy_(host_blob, non_blocking=True)
        ctx.layer_step(wl["layer"], dq, kv_e2e, wl["y"], M, None, dlog, None, stream)
        hy.copy_(wl["y"], non_blocking=True)
        stream.synchronize()          # the caller consumes y before the next decode step

    for _ in range(3):
        step_e2e()
    ms_eager = timed(step_e2e, args.steps) / args.steps
    # The same operations captured once into a CUDA graph and replayed: one host call per step instead of a Python /
    # ctypes round per operation.  Every replay is followed by a stream synchronise (the caller consumes y before the
    # next decode step), inside the timed region.  Two forms: y copied to pinned host memory by a copy node, and y
    # written there by the step's own stores (the y pointer handed to aflex_layer_step is the pinned, device-mapped
    # host buffer: the result crosses PCIe as the last GEMM phase produces it, no separate copy).
    # A third form also leaves q where it is: the attention kernel's producer fetches each piece's queries (2 KB) from
    # the pinned, device-mapped host buffer itself, under the KV stream, and only the page table and the lengths
    # (the first thing the kernel needs) are copied ahead.  q sits at the front of the packed buffer, so the copied
    # part is its tail.
    q_bytes = layout[0][1]
    small_off = layout[1][0]

    def capture(direct_out: bool, direct_q: bool = False):
        graph = torch.cuda.CUDAGraph()
        cap = torch.cuda.Stream()
        cap.wait_stream(stream)
        with torch.cuda.graph(graph, stream=cap):
            if direct_q:
                dev_blob[small_off:].copy_(host_blob[small_off:], non_blocking=True)
            else:
                dev_blob.copy_(host_blob, non_blocking=True)
            ctx.layer_step(wl["layer"], views_h[0] if direct_q else dq, kv_e2e, hy if direct_out else wl["y"], M, None, dlog, None,
                           torch.cuda.current_stream())
            if not direct_out:
                hy.copy_(wl["y"], non_blocking=True)
        stream.wait_stream(cap)
        return graph

    ms_graph = {}
    y_ref = wl["y"].cpu()
    for direct_out in (False, True, "q"):
        graph = capture(direct_out is not False, direct_out == "q")

        def step_graph():
            graph.replay()
            stream.synchronize()

        hy.zero_()
        for _ in range(3):
            step_graph()
        assert torch.equal(hy, y_ref), "graph replay did not deliver y"
        ms_graph[direct_out] = timed(step_graph, args.steps) / args.steps
    ms_e2e = min(ms_graph.values())
    e2e = {"value": whole_job_tokens_per_s(world, cfg.batch, ms_e2e), "unit": "tokens/s", "ms_per_step": ms_e2e,
           "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
           "how": "replayed CUDA graph, synchronised every step: " + {
               False: "H2D copy of q / page table / lengths from pinned memory, aflex_layer_step, D2H copy of y",
               True: "H2D copy of q / page table / lengths from pinned memory, aflex_layer_step with y in pinned device-mapped host memory",
               "q": "H2D copy of page table / lengths, aflex_layer_step with q and y in pinned device-mapped host memory "
                    "(the kernels move them across PCIe themselves)"}[min(ms_graph, key=ms_graph.get)],
           "ms_per_step_graph_q_and_y_in_host_memory": ms_graph["q"],
           "ms_per_step_graph_y_stored_to_host": ms_graph[True], "ms_per_step_graph_y_copied_to_host": ms_graph[False],
           "ms_per_step_without_graph": ms_eager}

    # ---- energy per token at default clocks (read-only NVML; the paper's metric, Section 6.1)
    energy = None
    if not args.no_energy and rank == 0:
        energy = measure_energy(step, barrier, local_rank, cfg.batch, ms_step)

    # ---- the stated targets beyond this configuration (one GPU, rank 0 at N = 1 only: nobody waits at a barrier)
    targets = None
    if rank == 0 and world == 1 and not args.no_targets:
        targets = run_targets(args, cfg, wl, ctx, local_rank, device, peaks, stream)

    # ---- CPU baseline: the oracle on a bounded sample, rank 0 at N = 1 only
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        rows = list(range(min(args.ref_rows, cfg.batch)))
        dt, threads = oracle_sample(cfg, wl, rows)
        cpu = {"value": len(rows) / dt, "unit": "tokens/s", "cores": threads, "kind": "oracle", "seconds": round(dt, 2),
               "host_cpus": os.cpu_count(),
               "sample": f"fp64 oracle layer step on batch rows {rows[0]}..{rows[-1]} of {cfg.batch} (rows are independent)"}
        if cfg.cfg_id == 1:
            # the tiny configuration also gets a single-thread figure
            from oracle import oracle as O
            O.set_num_threads(1)
            dt1, _ = oracle_sample(cfg, wl, rows)
            O.set_num_threads(threads)
            cpu["value_1_thread"] = len(rows) / dt1

    # ---- the A/F pair across two GPUs (N >= 2 only): rank 0 drives its own GPU and the next one, the others wait on the host
    af_pair = af_pair_devices(world, rank, local_rank, torch.cuda.device_count())
    if world > 1:
        barrier()                                          # every rank has finished its replica work
        if isinstance(af_pair, tuple):
            del wl
            torch.cuda.empty_cache()
            try:
                af_pair = run_af_pair_record(IN.CONFIGS[3], af_pair[0], af_pair[1], 4, 10)
            except Exception as exc:                       # never lose the headline line to the extra record
                af_pair = {"failed": str(exc)[:300]}
            torch.cuda.set_device(local_rank)
        wait_for_rank0(dist, host_group)

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": {"workload": f"config {cfg.cfg_id}: {cfg.name}", "batch": cfg.batch, "microbatch_depth": M,
                           "hq_hkv_d": [cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim], "hidden": cfg.hidden,
                           "inter": cfg.inter, "experts": cfg.num_experts, "top_k": cfg.top_k,
                           "context_tokens": int(lens_np.sum()), "page_size": 16,
                           "l2": "inputs larger than L2 (KV + weights >> 126 MB), no flush",
                           "parallelism": "replicas only" if world > 1 else "1 GPU"},
                "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline, "kernels": kernels, "operators_alone": operators,
                "cpu_baseline": cpu}
        if energy is not None:
            line["energy"] = energy
        if targets is not None:
            line["targets"] = targets
        line["af_pair"] = af_pair
        print(json.dumps(line), flush=True)
    ctx.close()
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
