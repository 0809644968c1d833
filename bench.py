#!/usr/bin/env python
"""Benchmark of the Q4 KV-cache hot path on B200.

Default workload: the Llama-3.1-8B-shaped batched decode step (32 layers, 5 agents x 4096 cached
tokens, Q4 group-64 K and V in 256-token blocks): per layer, quantize-append one new K/V token per
agent, then decode attention of one query per agent over the whole Q4 cache.  One "step" is all
layers.  The metric is the achieved HBM bandwidth over the algorithmic bytes of the step (each
needed Q4 row read once + q + out + new rows); agent-steps/s rides along.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 1|2|3|4|5|6|7] [--impl reference]

N > 1 (under torchrun) runs independent replicas, one per GPU: the path has no collective.
`--impl reference` times the CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import math
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2603_04428_b200 import synth  # noqa: E402


# ------------------------------------------------------------------------------------------------
# workload arithmetic (bytes / flops the roofline is quoted on)
# ------------------------------------------------------------------------------------------------
def row_bytes(w: synth.Workload) -> int:
    """Bytes of one token's K and V rows over all KV heads."""
    k = w.d_qk // 2 + 4 * (w.d_qk // 64)
    v = 0 if w.v_aliases_k else w.d_v // 2 + 4 * (w.d_v // 64)
    return w.n_kv_heads * (k + v)


def decode_layer_bytes(w: synth.Workload, layer: int) -> int:
    win = w.layer_window(layer)
    toks = sum(min(n + w.new_tokens, win) if win else n + w.new_tokens for n in w.lens)
    cache = toks * row_bytes(w)
    q = w.n_agents * w.n_q_heads * w.d_qk * 2
    out = w.n_agents * w.n_q_heads * w.d_v * 4
    new_in = w.n_agents * w.new_tokens * w.n_kv_heads * (w.d_qk + (0 if w.v_aliases_k else w.d_v)) * 2
    new_out = w.n_agents * w.new_tokens * row_bytes(w)
    return cache + q + out + new_in + new_out


def prefill_layer_flops(w: synth.Workload) -> float:
    """4 * D * Hq * sum_i (P + i + 1) per agent (QK^T and PV, causal pairs only; D = d_qk = d_v)."""
    fl = 0.0
    for P in w.lens:
        C = w.new_tokens
        pairs = C * P + C * (C + 1) / 2
        fl += 2.0 * w.n_q_heads * pairs * (w.d_qk + w.d_v)
    return fl


def workload_name(w: synth.Workload) -> str:
    return w.name


# ------------------------------------------------------------------------------------------------
# clocks sampling
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None

    def start(self):
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                       "-lms", "100", "-i", str(self.gpu)], stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self) -> dict:
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f:
            c = [x.strip() for x in line.split(",")]
            if len(c) < 9:
                continue
            try:
                sm.append(float(c[1]))
                mx.append(float(c[2]))
            except ValueError:
                continue
            for name, val in zip(names, c[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.f.close()
        os.unlink(self.f.name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------------
# device-side workload
# ------------------------------------------------------------------------------------------------
class DeviceWorkload:
    """All state of one workload resident on the GPU: the Q4 pool (filled by the library's own quantizer
    from seeded on-device N(0,1) bf16 values), block tables, per-layer q / new K,V, outputs."""

    def __init__(self, w: synth.Workload, device_index: int, two_calls: bool = False, exact_products: bool = False,
                 sb_dtype: int = 0):
        import torch
        from paper_2603_04428_b200 import binding as B, harness as H
        self.torch, self.B, self.w = torch, B, w
        torch.cuda.set_device(device_index)
        A, L = w.n_agents, w.n_layers
        self.n_blocks = w.blocks_needed() + 4
        tabs = synth.block_tables(w.seed, 99, w.lens, self.n_blocks, extra_tokens=w.new_tokens)
        self.dc = H.DeviceCache(L, w.n_q_heads, w.n_kv_heads, w.d_qk, w.d_v, w.v_aliases_k, self.n_blocks, tabs,
                                fill_byte=None, exact_products=exact_products, sb_dtype=sb_dtype)
        dc = self.dc
        g = torch.Generator(device="cuda")
        g.manual_seed(w.seed)
        self.lens0 = H.dev(np.asarray(w.lens, dtype=np.int32))
        self.lens1 = H.dev(np.asarray([n + w.new_tokens for n in w.lens], dtype=np.int32))
        self.max_kv = max(w.lens) + w.new_tokens
        # ---- fill the cache: per layer, per agent (bounded temporaries) ----
        zero = H.dev(np.zeros(1, dtype=np.int32))
        for l in range(L):
            ko = vo = None
            if w.outlier_frac > 0:
                ko = torch.from_numpy(synth.outlier_channels(w.seed, 100 + l, w.n_kv_heads, w.d_qk, w.outlier_frac)).cuda()
                vo = torch.from_numpy(synth.outlier_channels(w.seed, 200 + l, w.n_kv_heads, w.d_v, w.outlier_frac)).cuda()
            for a, n in enumerate(w.lens):
                t, bt = dc.sub_batch(a, a + 1)
                for c0 in range(0, n, 8192):
                    c = min(8192, n - c0)
                    k = torch.randn((c, w.n_kv_heads * w.d_qk), generator=g, device="cuda", dtype=torch.float32)
                    if ko is not None:
                        k[:, ko] *= 8.0
                    k = k.to(torch.bfloat16).view(c, w.n_kv_heads, w.d_qk)
                    v = None
                    if not w.v_aliases_k:
                        v = torch.randn((c, w.n_kv_heads * w.d_v), generator=g, device="cuda", dtype=torch.float32)
                        if vo is not None:
                            v[:, vo] *= 8.0
                        v = v.to(torch.bfloat16).view(c, w.n_kv_heads, w.d_v)
                    offs = H.dev(np.asarray([0, c], dtype=np.int32))
                    pos = H.dev(np.asarray([c0], dtype=np.int32))
                    dc.append(l, pos, offs, k, v, bt=bt)
        # ---- per-step inputs and outputs ----
        nq = A if w.kind == "decode" else A * w.new_tokens
        self.q = torch.randn((L, nq, w.n_q_heads, w.d_qk), generator=g, device="cuda").to(torch.bfloat16)
        self.k_new = torch.randn((L, A * w.new_tokens, w.n_kv_heads, w.d_qk), generator=g, device="cuda").to(torch.bfloat16)
        self.v_new = None if w.v_aliases_k else torch.randn(
            (L, A * w.new_tokens, w.n_kv_heads, w.d_v), generator=g, device="cuda").to(torch.bfloat16)
        self.out = torch.empty((L, nq, w.n_q_heads, w.d_v), dtype=torch.float32, device="cuda")
        self.new_offs = H.dev(np.arange(A + 1, dtype=np.int32) * w.new_tokens)
        self.q_offs = self.new_offs
        self.ws = torch.zeros(max(B.q4kv_workspace_bytes(dc.spec, A, self.max_kv, 0),
                                  B.q4kv_workspace_bytes(dc.spec, A, self.max_kv, nq)), dtype=torch.uint8, device="cuda")
        torch.cuda.synchronize()
        assert dc.read_flags() == 0
        self.fused = fused_update_and_fetch(w) and not two_calls

    # one layer of the step ----------------------------------------------------------------------
    def append_layer(self, l):
        w, dc, B = self.w, self.dc, self.B
        B.q4kv_quantize_append(dc.spec, dc.pool, dc.n_blocks, l, dc.bt, self.lens0, self.new_offs,
                               w.n_agents * w.new_tokens, self.k_new[l], None if self.v_new is None else self.v_new[l],
                               dc.flags)

    def attend_layer(self, l):
        w, dc, B = self.w, self.dc, self.B
        if w.kind == "decode":
            B.q4kv_decode_attention(dc.spec, dc.pool, dc.n_blocks, l, dc.bt, self.lens1, self.max_kv,
                                    w.layer_window(l), self.q[l], w.softmax_scale, self.out[l], B.OUT_F32, None,
                                    self.ws, dc.flags)
        else:
            B.q4kv_prefill_attention(dc.spec, dc.pool, dc.n_blocks, l, dc.bt, self.lens1, self.q_offs,
                                     w.n_agents * w.new_tokens, w.new_tokens, self.max_kv, w.layer_window(l),
                                     self.q[l], w.softmax_scale, self.out[l], B.OUT_F32, None, self.ws, dc.flags)

    def fused_layer(self, l):
        """Update-and-fetch in one launch: the new token is quantized by the warp that attends its chunk."""
        w, dc, B = self.w, self.dc, self.B
        B.q4kv_append_decode_attention(dc.spec, dc.pool, dc.n_blocks, l, dc.bt, self.lens1, self.max_kv,
                                       w.layer_window(l), self.k_new[l], None if self.v_new is None else self.v_new[l],
                                       self.q[l], w.softmax_scale,
                                       self.out[l], B.OUT_F32, None, self.ws, dc.flags)

    def layers_supported(self):
        w = self.w
        return fused_update_and_fetch(w) and not w.v_aliases_k and w.n_layers <= 64

    def layers_step(self):
        """The whole step as ONE launch: update-and-fetch of all layers (for callers that hold every layer's rows)."""
        w, dc, B = self.w, self.dc, self.B
        if not hasattr(self, "ws_layers"):
            self.ws_layers = self.torch.zeros(B.q4kv_workspace_bytes_layers(dc.spec, w.n_agents, self.max_kv, w.n_layers),
                                              dtype=self.torch.uint8, device="cuda")
        B.q4kv_decode_attention_layers(dc.spec, dc.pool, dc.n_blocks, 0, w.n_layers, dc.bt, self.lens1, self.max_kv,
                                       [w.layer_window(l) for l in range(w.n_layers)], self.k_new, self.v_new, self.q,
                                       w.softmax_scale, self.out, B.OUT_F32, None, self.ws_layers, dc.flags)

    def step(self, l0=0, l1=None):
        for l in range(l0, self.w.n_layers if l1 is None else l1):
            if self.fused:
                self.fused_layer(l)
            else:
                self.append_layer(l)
                self.attend_layer(l)


def slowest_rank(torch, dist, seconds, device):
    """Replicas only: every rank times the same work on its own GPU; the job's time is the slowest rank's (element-wise
    maximum over the ranks), and the job's throughput is world_size x units / that time."""
    if dist is None:
        return [float(x) for x in seconds]
    tt = torch.tensor(seconds, device=device, dtype=torch.float64)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    return [float(x) for x in tt]


def time_region(torch, fn, iters):
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / 1e3


def timed_batches(torch, fn, k, min_total_s=0.5, max_batches=400):
    """Batches of exactly k calls of fn, back to back on the current stream, an event between consecutive batches and
    one synchronize at the end; enough batches that the timed region lasts at least min_total_s.  Returns the batch
    times in seconds (their median is what the line reports)."""
    t1 = time_region(torch, fn, k)                         # sizes the region (not reported)
    n = int(min(max_batches, max(3, math.ceil(min_total_s / max(t1, 1e-9)))))
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(n + 1)]
    torch.cuda.synchronize()
    ev[0].record()
    for i in range(n):
        for _ in range(k):
            fn()
        ev[i + 1].record()
    torch.cuda.synchronize()
    return [ev[i].elapsed_time(ev[i + 1]) / 1e3 for i in range(n)]


# ------------------------------------------------------------------------------------------------
# CPU oracle leg
# ------------------------------------------------------------------------------------------------
def oracle_sample(w: synth.Workload, budget_s: float = 12.0):
    """Time the oracle on ONE layer of the workload restricted to a sample of agents: quantize-append of the
    new tokens plus attention.  Returns (seconds per sample-step, bytes or flops covered, description, threads)."""
    from oracle import q4kv_oracle as O
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        threads = 1
    f32 = synth.bf16_bits_to_f32
    spec = O.Spec(1, w.n_q_heads, w.n_kv_heads, w.d_qk, w.d_v, w.v_aliases_k)
    if w.kind == "decode":
        # sample: the first agents until at least 12000 cached tokens
        agents, tot = [], 0
        for a, n in enumerate(w.lens):
            agents.append(a)
            tot += n
            if tot >= 12000:
                break
        lens = [w.lens[a] for a in agents]
    else:
        agents, lens = [0], [w.lens[0]]
    n_blocks = sum(-(-(n + w.new_tokens) // 256) for n in lens)
    tabs = synth.block_tables(w.seed, 99, lens, n_blocks, extra_tokens=w.new_tokens)
    pool = O.Pool(spec, n_blocks)
    for i, n in enumerate(lens):
        k = f32(synth.kv_bf16(w.seed, 10 * i + 1, n, w.n_kv_heads, w.d_qk))
        v = None if w.v_aliases_k else f32(synth.kv_bf16(w.seed, 10 * i + 2, n, w.n_kv_heads, w.d_v))
        O.quantize_append(pool, 0, tabs[i:i + 1], [0], [0, n], k, v)
    A = len(lens)
    kn = f32(synth.kv_bf16(w.seed, 501, A * w.new_tokens, w.n_kv_heads, w.d_qk))
    vn = None if w.v_aliases_k else f32(synth.kv_bf16(w.seed, 502, A * w.new_tokens, w.n_kv_heads, w.d_v))
    offs = [i * w.new_tokens for i in range(A + 1)]
    lens1 = [n + w.new_tokens for n in lens]
    if w.kind == "decode":
        q = f32(synth.normal_bf16(w.seed, 7, (A, w.n_q_heads, w.d_qk)))
        win = w.layer_window(w.n_layers - 1)          # a global layer when the model has them

        def one():
            O.quantize_append(pool, 0, tabs, lens, offs, kn, vn)
            O.decode_attention(pool, 0, tabs, lens1, win, q, w.softmax_scale)
        units = sum(lens1) * row_bytes(w)
        desc = f"1 layer, agents {agents} of {w.n_agents} ({sum(lens1)} cached tokens), append + decode attention"
    else:
        rows = list(range(0, w.new_tokens, max(1, w.new_tokens // 16)))[:16]
        q = f32(synth.normal_bf16(w.seed, 7, (w.new_tokens, w.n_q_heads, w.d_qk)))

        def one():
            O.quantize_append(pool, 0, tabs, lens, offs, kn, vn)
            O.prefill_attention(pool, 0, tabs, lens1, offs, 0, q, w.softmax_scale, rows=rows)
        units = sum(2.0 * w.n_q_heads * (lens[0] + r + 1) * (w.d_qk + w.d_v) for r in rows)
        desc = f"1 layer, agent 0, append {w.new_tokens} tokens + {len(rows)} of {w.new_tokens} query rows"
    t0 = time.perf_counter()
    one()
    dt = time.perf_counter() - t0
    reps = 1
    while (time.perf_counter() - t0) < budget_s and reps < 1000:
        one()
        reps += 1
    dt = (time.perf_counter() - t0) / reps
    desc += (f"; {reps} repetitions, {dt * reps:.1f} s of CPU work; the oracle's loops over agents and heads are "
             "single-threaded Python, 'cores' is the size of the BLAS thread pool its matrix products may use")
    return dt, units, desc, threads


def metric_of(w):
    if w.kind == "decode":
        return "q4_decode_step_hbm_gbps", "GB/s", 1e9
    return "q4_prefix_chunked_prefill_tflops", "TFLOP/s", 1e12


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    metric, unit, div = metric_of(w)
    times = []
    desc, threads, units = "", 1, 0
    for i in range(args.warmup + args.steps):
        dt, units, desc, threads = oracle_sample(w, budget_s=0.0)
        if i >= args.warmup:
            times.append(dt)
    t = float(np.mean(times))
    val = units / t / div
    line = {"impl": "reference", "metric": metric, "value": val, "unit": unit, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": workload_name(w), "sample": desc},
            "cpu_baseline": {"value": val, "unit": unit, "cores": threads, "kind": "oracle", "sample": desc},
            "e2e": {"value": val, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return d.get("hbm_gbs", 6650.0), d.get("bf16_tflops", 1590.0), d.get("bf16_tflops_sustained", 1400.0), "measured"
    return 6650.0, 1590.0, 1400.0, "fallback"


NOMINAL_BF16_TFLOPS = 2250.0

# DRAM bytes (read + write) of one launch of each workload's dominant kernel, from one profiler capture of that
# kernel; None where no capture of the current kernel exists.  The decode and prefill captures ran the workload with
# fewer layers (the launch itself is the full-size one, so nothing is scaled); the config-3 figure is a global layer's
# launch, the MLA figure the attention kernel without its merge launch (4.88 MB more when its records miss L2).
NCU_TRAFFIC_BYTES = {"llama31_8b_decode": 23_991_723, "gemma3_12b_ragged_decode": 365_462_784,
                     "dsv2lite_mla_decode": 21_440_512, "dsv2lite_mla_decode_exact_products": 21_446_656,
                     "llama31_8b_chunked_prefill": 241_124_480,
                     "dsv2lite_perhead_mla_decode": 191_148_800, "gemma3_12b_shaped_global_prefill": 151_449_472,
                     "dsv2lite_perhead_mla_prefill": 146_757_504,
                     "pack": 254_257_000, "unpack": 251_510_000, "append_8x1024": 33_606_912}


def measure(w, args, local, dist=None, full=True):
    """One workload on this rank's GPU: the L-layer step as a CUDA graph, timed in batches of args.steps replays over a
    region of at least half a second (median batch), the per-launch time of the attention kernel from a graph of the L
    attention calls, clocks sampled meanwhile; with full=True also the end-to-end step through host buffers."""
    import torch
    dw = DeviceWorkload(w, local, two_calls=args.two_calls, exact_products=args.exact_products,
                        sb_dtype=1 if args.sb_bf16 else 0)
    L = w.n_layers
    use_graph = not args.no_graph
    stream = torch.cuda.Stream()
    res = {}
    with torch.cuda.stream(stream):
        for _ in range(2):
            dw.step()
        stream.synchronize()
        graph = None
        if use_graph:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                dw.step()
        run = graph.replay if graph is not None else dw.step
        for _ in range(args.warmup):
            run()
        stream.synchronize()
        if dist is not None:
            dist.barrier()
        sampler = ClockSampler(local)
        sampler.start()
        torch.cuda.synchronize()
        k = args.steps if full or time_region(torch, run, 1) * args.steps < args.min_seconds / 2 else 1
        batches = timed_batches(torch, run, k, min_total_s=args.min_seconds)
        t_step = float(np.median(batches)) / k

        # per-launch durations: the L attention calls of a step (one per layer, each over its own layer's cache, so
        # every launch streams from HBM) replayed back to back from a graph of their own; likewise the L append calls
        def per_launch_s(layer_fn):
            for l in range(L):
                layer_fn(l)
            stream.synchronize()
            if use_graph:
                g2 = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g2, stream=stream):
                    for l in range(L):
                        layer_fn(l)
                fn = g2.replay
            else:
                def fn():
                    for l in range(L):
                        layer_fn(l)
            for _ in range(3):
                fn()
            return float(np.median(timed_batches(torch, fn, 1, min_total_s=args.min_seconds / 2))) / L
        att_s = per_launch_s(dw.fused_layer if dw.fused else dw.attend_layer)
        app_s = per_launch_s(dw.append_layer)
        gl_s = None
        if w.window:
            gl_layers = [l for l in range(L) if w.layer_window(l) == 0]
            gl_fn = dw.fused_layer if dw.fused else dw.attend_layer
            gl_s = per_launch_s(lambda i: gl_fn(gl_layers[i % len(gl_layers)]))
        lb_s = None
        if dw.layers_supported():
            for _ in range(3):
                dw.layers_step()
            lb_s = float(np.median(timed_batches(torch, dw.layers_step, 1, min_total_s=args.min_seconds / 2)))
        clocks = sampler.stop()
        res.update(lb_s=lb_s)
        res.update(t_step=t_step, k=k, n_batches=len(batches), region_s=float(np.sum(batches)), att_s=att_s, app_s=app_s,
                   gl_s=gl_s, clocks=clocks, graph=graph is not None, fused=dw.fused)
        if full:
            # ---- end to end through the C ABI with host buffers ----
            hq = dw.q.cpu().pin_memory()
            hk = dw.k_new.cpu().pin_memory()
            hv = None if dw.v_new is None else dw.v_new.cpu().pin_memory()
            hout = torch.empty(dw.out.shape, dtype=dw.out.dtype).pin_memory()

            # The step in four runs of layers, so that a run's inputs travel while the runs before it compute and its
            # results travel while the runs after it compute: one CUDA graph over two streams (every input and every
            # result still crosses the host link inside the step).
            side = torch.cuda.Stream()
            n_seg = 4 if L >= 8 else (2 if L >= 2 else 1)
            cuts = [L * i // n_seg for i in range(n_seg + 1)]
            e2e_graph = None
            if use_graph and n_seg >= 2:
                def run_in(a, b):
                    dw.q[a:b].copy_(hq[a:b], non_blocking=True)
                    dw.k_new[a:b].copy_(hk[a:b], non_blocking=True)
                    if hv is not None:
                        dw.v_new[a:b].copy_(hv[a:b], non_blocking=True)
                e2e_graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(e2e_graph, stream=stream):
                    run_in(cuts[0], cuts[1])
                    side.wait_stream(stream)                   # fork
                    arrived = [None]
                    with torch.cuda.stream(side):
                        for i in range(1, n_seg):
                            run_in(cuts[i], cuts[i + 1])
                            ev = torch.cuda.Event(); ev.record(side)
                            arrived.append(ev)
                    for i in range(n_seg):
                        if arrived[i] is not None:
                            stream.wait_event(arrived[i])
                        dw.step(cuts[i], cuts[i + 1])
                        if i + 1 < n_seg:
                            done = torch.cuda.Event(); done.record(stream)
                            with torch.cuda.stream(side):
                                side.wait_event(done)
                                hout[cuts[i]:cuts[i + 1]].copy_(dw.out[cuts[i]:cuts[i + 1]], non_blocking=True)
                        else:
                            hout[cuts[i]:cuts[i + 1]].copy_(dw.out[cuts[i]:cuts[i + 1]], non_blocking=True)
                    stream.wait_stream(side)                   # join

            def e2e_step():
                if e2e_graph is not None:
                    e2e_graph.replay()
                else:
                    dw.q.copy_(hq, non_blocking=True)
                    dw.k_new.copy_(hk, non_blocking=True)
                    if hv is not None:
                        dw.v_new.copy_(hv, non_blocking=True)
                    run()
                    hout.copy_(dw.out, non_blocking=True)
                stream.synchronize()
            for _ in range(2):
                e2e_step()
            e2e_iters = max(3, min(args.steps, 10))
            res["t_e2e"] = time_region(torch, e2e_step, e2e_iters) / e2e_iters
            res["h2d"] = hq.numel() * 2 + hk.numel() * 2 + (0 if hv is None else hv.numel() * 2)
            res["d2h"] = hout.numel() * 4
    assert dw.dc.read_flags() == 0, "device status flags set during the benchmark"
    del dw
    torch.cuda.empty_cache()
    return res


def roofline_of(w, res):
    hbm_peak, tf_burst, tf_sust, peak_kind = peaks()
    L = w.n_layers
    att_s = res["att_s"]
    if w.kind == "decode":
        step_units = float(sum(decode_layer_bytes(w, l) for l in range(L)))
        launch_units = step_units / L
        call = "q4kv_append_decode_attention" if res["fused"] else "q4kv_decode_attention"
        roof = {"bound": "hbm", "kernel": call + " (one call per layer, L calls replayed back to back)",
                "achieved": launch_units / att_s / 1e9, "peak": hbm_peak, "unit": "GB/s", "peak_kind": peak_kind}
        if w.window:
            # window and global layers differ by ~9x in bytes: quote the global layers, which dominate the step
            gl = [l for l in range(L) if w.layer_window(l) == 0]
            att_s = res["gl_s"]
            roof["achieved"] = float(np.mean([decode_layer_bytes(w, l) for l in gl])) / att_s / 1e9
            roof["kernel"] += ", global layers only"
        roof["frac"] = roof["achieved"] / roof["peak"]
    else:
        step_units = prefill_layer_flops(w) * L
        launch_units = step_units / L
        ach = launch_units / att_s / 1e12
        roof = {"bound": "tensor", "kernel": "q4kv_prefill_attention (one call per layer)",
                "achieved": ach, "peak": tf_sust, "unit": "TFLOP/s", "peak_kind": peak_kind + " sustained bf16",
                "frac": ach / tf_sust, "frac_of_burst": ach / tf_burst, "frac_of_nominal": ach / NOMINAL_BF16_TFLOPS}
    roof["traffic"] = NCU_TRAFFIC_BYTES.get(w.name)
    roof["avg_launch_us"] = att_s * 1e6
    if res.get("lb_s"):
        # the same step as one launch for all layers (q4kv_decode_attention_layers): the per-kernel rate at this
        # batch size when the caller has every layer's rows at hand; labelled, beside the per-layer number
        ach = step_units / res["lb_s"] / 1e9
        roof["layer_batched"] = {"kernel": "q4kv_decode_attention_layers (all layers in one launch)", "ms_per_step": res["lb_s"] * 1e3,
                                 "achieved": ach, "frac": ach / hbm_peak, "agent_steps_per_s": w.n_agents / res["lb_s"]}
    return step_units, roof


def config_of(w, res):
    L = w.n_layers
    return {"workload": workload_name(w), "layers": L, "agents": w.n_agents,
            "kv_lens": w.lens if len(set(w.lens)) > 1 else w.lens[0],
            "q_heads": w.n_q_heads, "kv_heads": w.n_kv_heads, "d_qk": w.d_qk, "d_v": w.d_v,
            "new_tokens_per_agent": w.new_tokens, "window": w.window,
            "l2": "inputs larger than L2: every step streams the whole multi-layer cache",
            "launch": "cuda graph replay of the L-layer step" if res["graph"] else "eager",
            "timing": f"median of {res['n_batches']} back-to-back batches of {res['k']} steps "
                      f"({res['region_s']:.2f} s timed)",
            "update_and_fetch": "one call per layer" if res["fused"]
            else "quantize-append launch + attention launch per layer",
            "multi_gpu": "replicas only"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", type=int, default=None,
                    help="index into the five configurations (0-based).  Default: configuration 1 as the headline, "
                         "with the other configurations and the copy-like kernels under all_configs")
    ap.add_argument("--impl", default="q4kv", choices=["q4kv", "reference"])
    ap.add_argument("--no-graph", action="store_true", help="launch eagerly instead of replaying a CUDA graph")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-all-configs", action="store_true", help="headline workload only")
    ap.add_argument("--two-calls", action="store_true",
                    help="decode step as a quantize-append launch plus an attention launch per layer instead of the "
                         "one-launch update-and-fetch")
    ap.add_argument("--min-seconds", type=float, default=0.5, help="least duration of each timed region")
    ap.add_argument("--sb-bf16", action="store_true",
                    help="bfloat16 scales and biases in the cache (q4kv_spec.sb_dtype = 1) instead of binary16")
    ap.add_argument("--exact-products", action="store_true",
                    help="set q4kv_spec.exact_products: every call takes the kernels that multiply the 4-bit codes exactly")
    ap.add_argument("--op", default="step", choices=["step", "pack", "unpack"],
                    help="step: the append + attention step of --workload; pack: q4kv_pack / q4kv_unpack / bulk append")
    ap.add_argument("--agents", type=int, default=0,
                    help="scaled variant of a uniform-length configuration: this many agents (named so in config.workload)")
    ap.add_argument("--layers", type=int, default=0, help="scaled variant: this many layers")
    args = ap.parse_args()
    if args.op in ("pack", "unpack"):
        print(json.dumps(run_pack(args)))
        return
    args.warmup = max(args.warmup, 3) if args.impl == "q4kv" else args.warmup
    default_run = (args.workload is None and args.agents == 0 and args.layers == 0 and not args.exact_products
                   and not args.sb_bf16)
    w = synth.workload(1 if args.workload is None else args.workload)
    if args.agents > 0 or args.layers > 0:
        # not one of the five configurations any more: the name says so, and no stored counter applies to it
        if args.agents > 0 and len(set(w.lens)) != 1:
            raise SystemExit("--agents scales configurations whose agents have one common length")
        lens = [w.lens[0]] * args.agents if args.agents > 0 else w.lens
        layers = args.layers if args.layers > 0 else w.n_layers
        w = dataclasses.replace(w, lens=lens, n_layers=layers, name=f"{w.name}_scaled_{len(lens)}agents_{layers}layers")
    if args.exact_products:
        w = dataclasses.replace(w, name=w.name + "_exact_products")       # other kernels: no stored counter applies
    if args.sb_bf16:
        w = dataclasses.replace(w, name=w.name + "_bf16_scale_bias")
    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    metric, unit, div = metric_of(w)
    res = measure(w, args, local, dist, full=True)
    t_step, t_e2e = slowest_rank(torch, dist, [res["t_step"], res["t_e2e"]], "cuda")
    step_units, roof = roofline_of(w, res)
    value = world * step_units / t_step / div
    e2e_val = world * step_units / t_e2e / div
    clocks = res["clocks"]
    line = {
        "metric": metric, "value": value, "unit": unit, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": t_step * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f16 tensor-core products on u4 codes, f32 accumulate", "data": "synthetic",
        "config": config_of(w, res),
        "agent_steps_per_s": world * w.n_agents / t_step,
        "step_bytes" if w.kind == "decode" else "step_flops": step_units,
        "append_avg_us": res["app_s"] * 1e6,
        "roofline": roof,
        "e2e": {"value": e2e_val, "unit": unit, "h2d_bytes_per_step": res["h2d"], "d2h_bytes_per_step": res["d2h"],
                "ms_per_step": t_e2e * 1e3},
        "gpu_launches": dw_launches(w, args.two_calls) * args.steps,
        "clocks": clocks,
        "ms_per_step_x_sm_mhz": None if not clocks.get("sm_mhz") else t_step * 1e3 * clocks["sm_mhz"],
    }
    if rank == 0 and world == 1 and default_run and not args.no_all_configs:
        allc = {}

        def entry(wi, ai):
            ri = measure(wi, ai, local, None, full=False)
            units_i, roof_i = roofline_of(wi, ri)
            mi, ui, di = metric_of(wi)
            allc[wi.name] = {"metric": mi, "value": units_i / ri["t_step"] / di, "unit": ui,
                             "ms_per_step": ri["t_step"] * 1e3, "agent_steps_per_s": wi.n_agents / ri["t_step"],
                             "append_avg_us": ri["app_s"] * 1e6, "roofline": roof_i, "config": config_of(wi, ri),
                             "gpu_launches_per_step": dw_launches(wi, ai.two_calls), "clocks": ri["clocks"]}

        for idx in (2, 3, 4, 5, 6, 7):
            entry(synth.workload(idx), args)
        # the MLA-latent decode again with q4kv_spec.exact_products set: the kernel that multiplies the codes (also the
        # route of bfloat16 caches and sharp softmax scales)
        w3 = synth.workload(3)
        entry(dataclasses.replace(w3, name=w3.name + "_exact_products"),
              argparse.Namespace(**{**vars(args), "exact_products": True}))
        # caches with bfloat16 scales and biases (q4kv_spec.sb_dtype = 1) on the two binary16-tile routes
        for idx in (3, 4):
            wi = synth.workload(idx)
            entry(dataclasses.replace(wi, name=wi.name + "_bf16_scale_bias"),
                  argparse.Namespace(**{**vars(args), "sb_bf16": True}))
        pk = run_pack(args)
        for name in ("pack", "unpack", "restore", "append_8x1024"):
            allc[name] = pk["kernels"][name]
        line["all_configs"] = allc
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        dt_o, units_o, desc, threads = oracle_sample(w)
        line["cpu_baseline"] = {"value": units_o / dt_o / div, "unit": unit, "cores": threads, "kind": "oracle",
                                "sample": desc, "seconds_per_sample": dt_o}
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def run_pack(args):
    """Persist / restore one Llama-3.1-8B-shaped agent (4096 tokens, 32 layers: 151 MB packed) and append a
    1024-token phase for 8 agents: the copy-like kernels of the path, each against the measured copy rate."""
    import torch
    from paper_2603_04428_b200 import binding as B, harness as H
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    hbm_peak, _, _, peak_kind = peaks()
    L, Hq, Hkv, D, n = 32, 32, 8, 128, 4096
    nb = n // 256 + 2
    dc = H.DeviceCache(L, Hq, Hkv, D, D, False, nb, synth.block_tables(synth.BASE_SEED, 99, [n], nb), fill_byte=7)
    nbytes = B.q4kv_packed_bytes(dc.spec, n)
    dst = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    min_s = getattr(args, "min_seconds", 0.5) / 2

    def timed(fn):
        for _ in range(max(3, args.warmup)):
            fn()
        return float(np.median(timed_batches(torch, fn, 1, min_total_s=min_s, max_batches=2000)))

    def timed_graph(fn):
        """fn's launches captured once in a CUDA graph and replayed: the kernels back to back, no host launch cost
        between them (a 20 us kernel launched from Python is otherwise timed at the host's launch rate)."""
        side = torch.cuda.Stream()
        with torch.cuda.stream(side):
            fn()
            side.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                fn()
            t = timed(g.replay)
            side.synchronize()
        return t
    if args.op == "unpack":
        # q4kv_unpack alone (pack and unpack are the same kernel by name: this is how a profiler tells them apart)
        B.q4kv_pack(dc.spec, dc.pool, dc.n_blocks, dc.tables[0], n, dst, dc.flags)
        t_unpack = timed_graph(lambda: B.q4kv_unpack(dc.spec, dst, n, dc.pool, dc.n_blocks, dc.tables[0], dc.flags))
        ach = 2 * nbytes / t_unpack / 1e9
        return {"metric": "q4_unpack_hbm_gbps", "value": ach, "unit": "GB/s", "n_gpus": 1, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": t_unpack * 1e3, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "u8", "data": "synthetic",
                "config": {"workload": "unpack_llama31_8b_agent", "packed_bytes": nbytes},
                "roofline": {"bound": "hbm", "kernel": "q4kv_unpack", "achieved": ach, "peak": hbm_peak, "unit": "GB/s",
                             "frac": ach / hbm_peak, "peak_kind": peak_kind, "avg_launch_us": t_unpack * 1e6,
                             "traffic": NCU_TRAFFIC_BYTES.get("unpack")}, "gpu_launches": args.steps}
    t_pack = timed_graph(lambda: B.q4kv_pack(dc.spec, dc.pool, dc.n_blocks, dc.tables[0], n, dst, dc.flags))
    t_unpack = timed_graph(lambda: B.q4kv_unpack(dc.spec, dst, n, dc.pool, dc.n_blocks, dc.tables[0], dc.flags))
    # ---- warm restore: pinned host image -> chunked copies overlapping q4kv_unpack (Table "TTFT", warm rows) ----
    image = torch.empty(nbytes, dtype=torch.uint8).pin_memory()
    image.copy_(dst)
    stage = torch.empty(8 * (nbytes // L), dtype=torch.uint8, device="cuda")
    copy_stream = torch.cuda.Stream()

    def restore():
        cur = torch.cuda.current_stream()
        copy_stream.wait_stream(cur)
        B.q4kv_restore(dc.spec, image, n, dc.pool, dc.n_blocks, dc.tables[0], stage, dc.flags, copy_stream=copy_stream,
                       unpack_stream=cur)
    t_restore = timed(restore)
    t_h2d = timed(lambda: dst.copy_(image, non_blocking=True))       # the plain pinned copy of the same bytes: the bound
    A, new = 8, 1024
    lens = [8192] * A
    nb2 = sum(-(-(x + new) // 256) for x in lens) + 2
    # 32 layers' worth of new rows (1.07 GB), so that consecutive launches do not find their inputs in L2
    LA = 32
    dc2 = H.DeviceCache(LA, Hq, Hkv, D, D, False, nb2, synth.block_tables(synth.BASE_SEED, 98, lens, nb2, extra_tokens=new),
                        fill_byte=None)
    k = torch.randn((LA, A * new, Hkv, D), device="cuda").to(torch.bfloat16)
    v = torch.randn((LA, A * new, Hkv, D), device="cuda").to(torch.bfloat16)
    pos = H.dev(np.asarray(lens, dtype=np.int32))
    offs = H.dev(np.arange(A + 1, dtype=np.int32) * new)

    def append_all():
        for l in range(LA):
            B.q4kv_quantize_append(dc2.spec, dc2.pool, dc2.n_blocks, l, dc2.bt, pos, offs, A * new, k[l], v[l], dc2.flags)
    t_app = timed_graph(append_all) / LA
    app_bytes = A * new * Hkv * D * 2 * 2 + A * new * Hkv * 144
    assert dc.read_flags() == 0 and dc2.read_flags() == 0

    def entry(kernel, nbytes_moved, t, note):
        ach = nbytes_moved / t / 1e9
        return {"metric": "hbm_gbps", "value": ach, "unit": "GB/s", "ms_per_step": t * 1e3,
                "roofline": {"bound": "hbm", "kernel": kernel, "achieved": ach, "peak": hbm_peak, "unit": "GB/s",
                             "frac": ach / hbm_peak, "peak_kind": peak_kind, "avg_launch_us": t * 1e6,
                             "traffic": NCU_TRAFFIC_BYTES.get(note)},
                "bytes": nbytes_moved}
    h2d_rate = nbytes / t_h2d / 1e9
    restore_entry = {"metric": "restore_gbps", "value": nbytes / t_restore / 1e9, "unit": "GB/s", "ms_per_step": t_restore * 1e3,
                     "roofline": {"bound": "h2d", "kernel": "q4kv_restore (pinned host image -> pool, 4096 tokens x 32 layers)",
                                  "achieved": nbytes / t_restore / 1e9, "peak": h2d_rate, "unit": "GB/s",
                                  "frac": t_h2d / t_restore, "peak_kind": "plain pinned host-to-device copy of the same bytes, "
                                  "measured in this run", "avg_launch_us": t_restore * 1e6, "traffic": None},
                     "bytes": nbytes}
    kernels = {"pack": entry("q4kv_pack", 2 * nbytes, t_pack, "pack"),
               "unpack": entry("q4kv_unpack", 2 * nbytes, t_unpack, "unpack"),
               "restore": restore_entry,
               "append_8x1024": entry("q4kv_quantize_append (8 agents x 1024 new tokens, one layer per launch)", app_bytes,
                                      t_app, "append_8x1024")}
    line = {"metric": "q4_pack_hbm_gbps", "value": kernels["pack"]["value"], "unit": "GB/s", "n_gpus": 1,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": t_pack * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
            "config": {"workload": "pack_unpack_append_llama31_8b_agent", "packed_bytes": nbytes,
                       "l2": "packed buffer + pool (302 MB) larger than L2; append: 32 layers of new rows (1.07 GB)"},
            "roofline": kernels["pack"]["roofline"], "kernels": kernels, "gpu_launches": args.steps}
    del dc, dc2, k, v, dst, image, stage
    torch.cuda.empty_cache()
    return line


def fused_update_and_fetch(w):
    """Decode shapes that q4kv_append_decode_attention covers (one launch per layer for append + attention)."""
    if w.kind != "decode":
        return False
    if w.v_aliases_k:      # the MLA-latent cache
        return (w.d_qk, w.d_v, w.n_kv_heads) == (576, 512, 1) and w.n_q_heads <= 16
    n_rep = w.n_q_heads // w.n_kv_heads
    return n_rep <= 4 and ((w.d_qk == w.d_v and w.d_qk in (128, 256)) or (w.d_qk, w.d_v) == (192, 128))


def dw_launches(w, two_calls=False):
    """Kernels of this library launched per step.  GQA decode: one update-and-fetch kernel per layer.  MLA-latent
    decode: the key-split update-and-fetch kernel and its merge kernel.  Prefill: one quantize-append and one
    attention kernel per layer.  As two calls, decode launches the quantize-append kernel as well."""
    mla = w.kind == "decode" and w.v_aliases_k
    if fused_update_and_fetch(w) and not two_calls:
        return (2 if mla else 1) * w.n_layers
    return (3 if mla else 2) * w.n_layers


if __name__ == "__main__":
    main()
