#!/usr/bin/env python
"""Benchmark of the MaskKV compress-and-attend path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One step = one transformer layer of the 32k LLaDA-shaped workload (N=32768 prompt keys, M=256 mask
queries, 32 heads, d=128, bf16, adaptive budgets) through the whole path:
maskkv_score -> maskkv_budget -> maskkv_select -> maskkv_compact -> maskkv_attend.
`value` is prompt tokens scored+compacted (and attended once) per second per layer, inputs resident
in HBM; `e2e` is the same with the layer's inputs in pinned host memory and both copies timed.
With N > 1 ranks (torchrun) each rank runs its own layers (no data-path collective): weak scaling.
`--impl reference` times the CPU oracle on a bounded sample of the same workload (rank 0 only).
Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import socket
import statistics
import subprocess

import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch

from paper_2510_09309_b200 import synth

METRIC = "prompt tokens scored+compacted/s per layer at 32k"
UNIT = "tokens/s"
RESIDENT_LAYERS = (0, 1, 15, 31)          # layers whose inputs stay resident and are cycled through
CALLS = ("score", "budget", "select", "compact", "attend")


# ----------------------------------------------------------------------------- multi-rank plumbing
def rank_world():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("LOCAL_RANK", "0"))


def shard_layers(n_layers: int, rank: int, world: int):
    """Layers this rank owns (round-robin): every layer belongs to exactly one rank."""
    return [l for l in range(n_layers) if l % world == rank]


def max_over_ranks(value: float, device=None) -> float:
    """The slowest rank's time; a no-op without a process group."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return value
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device=None) -> float:
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return value
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    """Reads SM clock, power and the clock-event reasons of one GPU every 10 ms through NVML (read-only queries) on a
    thread of its own.  mark() brackets the timed region; stop() reports the medians inside it."""

    def __init__(self, gpu_index: int):
        self.samples = []            # (time, sm_mhz, power_w, reasons bitmask)
        self.marks = {}
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            uuid = torch.cuda.get_device_properties(gpu_index).uuid      # CUDA_VISIBLE_DEVICES may renumber the GPUs
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + str(uuid)).encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(gpu_index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        except Exception:
            self._thread = None

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                mhz = float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                watts = nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0
                reasons = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                self.samples.append((time.perf_counter(), mhz, watts, reasons))
            except Exception:
                pass
            self._stop.wait(0.01)

    def mark(self, name: str):
        self.marks[name] = time.perf_counter()

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        if self._thread is None:
            return out
        self._stop.set()
        self._thread.join(timeout=2)
        nv = self.nv
        t0, t1 = self.marks.get("timed_start"), self.marks.get("timed_end")
        inside = [x for x in self.samples if t0 is not None and t1 is not None and t0 <= x[0] <= t1]
        region = "timed steps"
        if len(inside) < 3:
            inside, region = self.samples, "whole run"
        if not inside:
            return out
        bits = 0
        for x in inside:
            bits |= x[3]
        names = (("hw_slowdown", nv.nvmlClocksEventReasonHwSlowdown), ("hw_thermal_slowdown", nv.nvmlClocksEventReasonHwThermalSlowdown),
                 ("sw_thermal_slowdown", nv.nvmlClocksEventReasonSwThermalSlowdown), ("sw_power_cap", nv.nvmlClocksEventReasonSwPowerCap),
                 ("hw_power_brake", nv.nvmlClocksEventReasonHwPowerBrakeSlowdown))
        out.update(sm_mhz=statistics.median(x[1] for x in inside), power_w=round(statistics.median(x[2] for x in inside), 1),
                   samples=len(inside), region=region, reasons=[n for n, b in names if bits & b])
        return out



class LayerBuffers:
    """Device-side outputs and scratch shared by all layers of the workload (one layer in flight at a time)."""

    def __init__(self, ctx, B, wl, capacity, device):
        self.p = B.Problem(wl.torch_dtype, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.prompt_cu(), wl.live_cu(), device)
        R, Hkv, H, d = wl.n_requests, wl.n_kv_heads, wl.n_q_heads, wl.head_dim
        f32, i32 = torch.float32, torch.int32
        self.capacity = capacity
        self.scores = torch.empty((Hkv, self.p.sumN), dtype=f32, device=device)
        self.mass_p = torch.empty((R, Hkv), dtype=f32, device=device)
        self.mass_m = torch.empty((R, Hkv), dtype=f32, device=device)
        self.budgets = torch.empty((R, Hkv), dtype=i32, device=device)
        self.offsets = torch.zeros(R * Hkv + 1, dtype=i32, device=device)
        self.kept = torch.empty(capacity, dtype=i32, device=device)
        self.kc = torch.empty((capacity, d), dtype=wl.torch_dtype, device=device)
        self.vc = torch.empty((capacity, d), dtype=wl.torch_dtype, device=device)
        self.out = torch.empty((self.p.sumM, H, d), dtype=wl.torch_dtype, device=device)
        self.ws = torch.empty(max(ctx.maskkv_workspace_bytes(self.p), 256), dtype=torch.uint8, device=device)


def run_layer(ctx, buf, x, live, k_l, alpha, events=None):
    """The five calls of one layer on the current stream.  `events`: optional list of 6 CUDA events."""
    p = buf.p
    if events: events[0].record()
    ctx.maskkv_score(p, x["q_mask"], x["k_prompt"], x["k_mask"], buf.scores, buf.mass_p, buf.mass_m, buf.ws)
    if events: events[1].record()
    ctx.maskkv_budget(p, k_l, alpha, buf.mass_p, buf.mass_m, buf.capacity, buf.budgets, buf.offsets)
    if events: events[2].record()
    ctx.maskkv_select(p, buf.scores, buf.budgets, buf.offsets, buf.kept, buf.ws)
    if events: events[3].record()
    ctx.maskkv_compact(p, x["k_prompt"], x["v_prompt"], buf.kept, buf.offsets, buf.capacity, buf.kc, buf.vc)
    if events: events[4].record()
    ctx.maskkv_attend(p, live["q_live"], live["k_live"], live["v_live"], buf.kc, buf.vc, buf.offsets, buf.capacity, buf.out)
    if events: events[5].record()


# DRAM bytes (read + write) of one maskkv_score call at this workload.  bench.py cannot read DRAM counters itself: the
# figure is dram__bytes_read.sum + dram__bytes_write.sum of the call's two kernels from one ncu capture of this very
# command (sweep 1 279.5 MB + sweep 2 281.6 MB: the key tensor is read once per sweep); the JSON line names the source.
SCORE_DRAM_TRAFFIC_BYTES = 561.1e6
SCORE_DRAM_TRAFFIC_SOURCE = ("ncu --set full --clock-control none -k regex:score_(stats|colsum)_tc -s 3 -c 1 python bench.py --steps 4 "
                             "--warmup 3 --no-graph: dram__bytes_read.sum + dram__bytes_write.sum, sweep 1 279.5 MB + sweep 2 281.6 MB; "
                             "a constant of this file, not measured by this run")


def algorithmic_work(wl, mean_kept_per_head):
    """Per layer: flops of the one Q K^T product scoring needs, and the bytes each HBM-bound call must move."""
    N, M, H, Hkv, d = wl.prompt_lens[0], wl.n_mask, wl.n_q_heads, wl.n_kv_heads, wl.head_dim
    k = mean_kept_per_head
    return {
        "score_flops": 2.0 * M * (N + M) * d * H,                       # one Q K^T over prompt + mask keys
        "score_bytes": 2.0 * d * (N + M) * Hkv + 2.0 * d * M * H + 4.0 * N * Hkv,
        "select_bytes": 4.0 * N * Hkv + 4.0 * k * Hkv,                  # read every score once, write kept indices
        "compact_bytes": (4 * d * 2 + 4.0) * k * Hkv,                   # K and V row read + written, plus the index
        "attend_flops": 4.0 * M * (k + M) * d * H,
        "attend_bytes": 2.0 * (2 * M * H * d) + 2.0 * 2 * d * (k + M) * Hkv,
    }


def kv_cache_bytes(tokens_per_head: float, n_kv_heads: int, head_dim: int, elem_bytes: int = 2) -> float:
    """The paper's accounting of the KV cache of one layer (appendix, "Evaluation metrics"): 2 * L * H * d_head * s,
    keys and values of L tokens in each of H heads; for the compacted cache L is the mean number of kept tokens."""
    return 2.0 * tokens_per_head * n_kv_heads * head_dim * elem_bytes


def batched_calls(ctx, B, device):
    """maskkv_select / maskkv_compact / maskkv_attend on configs[4] (ragged serving: 8 requests of 1k-32k prompt tokens,
    256 segments, one layer, mean budget 256): per-call time warm (20 calls back to back) and cold (256 MB written
    between the calls, outside the timed region), with the algorithmic bytes each call must move."""
    wl = synth.config(5)
    x = synth.layer_inputs(wl, 1, device)
    live = synth.live_inputs(wl, 1, 0, device)
    buf = LayerBuffers(ctx, B, wl, wl.n_requests * wl.n_kv_heads * 2 * wl.mean_budget, device)
    run_layer(ctx, buf, x, live, wl.mean_budget, wl.alpha)
    torch.cuda.synchronize()
    p, d, M = buf.p, wl.head_dim, wl.n_mask
    S = wl.n_requests * wl.n_kv_heads
    kept = int(buf.offsets[-1].item())
    es = 2
    work = {
        "select": {"bytes": 4.0 * p.sumN * wl.n_kv_heads + 4.0 * kept},
        "compact": {"bytes": (4.0 * d * es + 4.0) * kept},
        "attend": {"bytes": 2.0 * es * p.sumM * wl.n_q_heads * d + 2.0 * es * d * (kept + p.sumM * wl.n_kv_heads),
                   "flops": 4.0 * M * d * (kept * wl.group + S * wl.group * M)},
    }
    calls = {
        "select": lambda: ctx.maskkv_select(p, buf.scores, buf.budgets, buf.offsets, buf.kept, buf.ws),
        "compact": lambda: ctx.maskkv_compact(p, x["k_prompt"], x["v_prompt"], buf.kept, buf.offsets, buf.capacity, buf.kc, buf.vc),
        "attend": lambda: ctx.maskkv_attend(p, live["q_live"], live["k_live"], live["v_live"], buf.kc, buf.vc, buf.offsets,
                                            buf.capacity, buf.out),
    }
    scratch = torch.empty(256 << 20, dtype=torch.uint8, device=device)
    hbm = load_peaks()["hbm_gbs"]
    out = {"workload": f"configs[4] ragged_serving, one layer: {wl.n_requests} requests, {p.sumN} prompt tokens, {S} segments, "
                       f"{kept} kept rows; events around single calls include the launch"}
    for name, call in calls.items():
        for _ in range(3):
            call()
        torch.cuda.synchronize()
        w0, w1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        w0.record()
        for _ in range(20):
            call()
        w1.record()
        torch.cuda.synchronize()
        warm_us = 1e3 * w0.elapsed_time(w1) / 20
        cold = []
        for i in range(10):
            scratch.fill_(i)                                           # evicts the call's inputs from L2
            c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            c0.record()
            call()
            c1.record()
            torch.cuda.synchronize()
            cold.append(1e3 * c0.elapsed_time(c1))
        cold_us = statistics.median(cold)
        row = {"warm_us": round(warm_us, 2), "cold_us": round(cold_us, 2), "bytes": work[name]["bytes"],
               "cold_GB/s": round(work[name]["bytes"] / (cold_us * 1e-6) / 1e9, 1),
               "cold_frac_of_hbm_peak": round(work[name]["bytes"] / (cold_us * 1e-6) / 1e9 / hbm, 3),
               "warm_GB/s": round(work[name]["bytes"] / (warm_us * 1e-6) / 1e9, 1)}
        if "flops" in work[name]:
            row["warm_TFLOP/s"] = round(work[name]["flops"] / (warm_us * 1e-6) / 1e12, 1)
        out[name] = row
    out["status_flags"] = ctx.maskkv_check_status()
    return out


def replayed_loop_us(call, n_graphs, reps, device):
    """Microseconds per call of `call(i)`, i = 0 .. n_graphs-1 (each i has its own pointers), when the whole sequence is
    captured into ONE CUDA graph (the overlapped launches between consecutive calls are kept inside a graph, not between
    graphs) and the graph is replayed, about `reps` calls in all timed with events.  None if capture is refused."""
    try:
        side = torch.cuda.Stream(device=device)
        side.wait_stream(torch.cuda.current_stream())
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                for j in range(n_graphs):
                    call(j)
        torch.cuda.current_stream().wait_stream(side)
        g.replay()
        torch.cuda.synchronize()
        rounds = max(1, reps // n_graphs)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(rounds):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        return 1e3 * e0.elapsed_time(e1) / (rounds * n_graphs)
    except Exception:
        torch.cuda.synchronize()
        return None


def timed_loop(call, reps, warm=3):
    """Average device time of `call(i)` over `reps` back-to-back invocations, in microseconds (CUDA events)."""
    for i in range(warm):
        call(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(reps):
        call(warm + i)
    e1.record()
    torch.cuda.synchronize()
    return 1e3 * e0.elapsed_time(e1) / reps


def dream_gqa_block(ctx, B, device, peaks, reps=200):
    """configs[3], one layer per call: 28 query heads on 4 KV heads, N=16384, M=512, d=128, bf16, uniform budget 512 per KV
    head.  maskkv_score and maskkv_attend alone, back to back, cycling through enough layers' inputs to exceed the L2;
    attention at these shapes is bound by the tensor cores (every K/V tile serves the 7 x 512 query rows of its group)."""
    wl = synth.config(4)
    N, M, H, Hkv, d, g = wl.prompt_lens[0], wl.n_mask, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.group
    n_sets = 10                                                     # 10 x (16.8 MB keys + 3.7 MB queries) > 126 MB L2
    xs, lives, caches = [], [], []
    buf = LayerBuffers(ctx, B, wl, Hkv * 512, device)
    for l in range(n_sets):
        x = synth.layer_inputs(wl, l, device)
        x.pop("planted", None); x.pop("v_mask", None)
        live = synth.live_inputs(wl, l, 0, device)
        run_layer(ctx, buf, x, live, 512, 1.0)
        caches.append((buf.kc.clone(), buf.vc.clone()))
        xs.append({"q_mask": x["q_mask"], "k_prompt": x["k_prompt"], "k_mask": x["k_mask"]})
        lives.append(live)
    torch.cuda.synchronize()
    p = buf.p
    outs = [torch.empty_like(buf.out) for _ in range(4)]            # 4 x 3.7 MB of output cycled as well

    def score(i):
        x = xs[i % n_sets]
        ctx.maskkv_score(p, x["q_mask"], x["k_prompt"], x["k_mask"], buf.scores, buf.mass_p, buf.mass_m, buf.ws)

    def attend(i):
        kc, vc = caches[i % n_sets]
        live = lives[i % n_sets]
        ctx.maskkv_attend(p, live["q_live"], live["k_live"], live["v_live"], kc, vc, buf.offsets, buf.capacity, outs[i % 4])

    score_us = timed_loop(score, reps)
    attend_us = timed_loop(attend, reps)
    k = 512
    score_flops = 2.0 * M * (N + M) * d * H
    attend_flops = 4.0 * M * (k + M) * d * H
    attend_bytes = 2.0 * (2 * M * H * d) + 2.0 * 2 * d * (k + M) * Hkv
    out = {"workload": f"configs[3] dream_gqa_16k, one layer per call: N={N} M={M} H={H} H_kv={Hkv} d={d}, budget {k} per KV head; "
                       f"{n_sets} layers' inputs cycled ({n_sets * (N * Hkv + M * H + M * Hkv) * d * 2 / 1e6:.0f} MB > L2), {reps} calls back to back",
           "score_us": round(score_us, 2), "attend_us": round(attend_us, 2)}
    for name, us, flops in (("score", score_us, score_flops), ("attend", attend_us, attend_flops)):
        tf = flops / (us * 1e-6) / 1e12
        out[name] = {"bound": "tensor", "achieved": round(tf, 1), "unit": "TFLOP/s", "flops": flops,
                     "frac_burst": round(tf / peaks["bf16_tflops"], 3), "frac_sustained": round(tf / peaks["bf16_tflops_sustained"], 3)}
    out["score"]["note"] = "one Q K^T counted; the two sweeps execute twice that"
    out["attend"]["flop_per_byte"] = round(attend_flops / attend_bytes, 1)
    out["status_flags"] = ctx.maskkv_check_status()
    return out


def kv_peak_bytes(n_layers, prompt_tokens, kept_per_head, n_kv_heads, head_dim, online, elem_bytes=2):
    """Peak bytes of prompt KV cache held during the first denoising step (paragraph after Eq. 13), with the paper's
    accounting 2 * tokens * heads * d_head * bytes per layer.  The model runs its layers in order; a layer's prompt K/V
    exist from the moment the layer has run.  Offline profile: layer l's budget is known beforehand, so the layer is
    compacted to kept_per_head[l] tokens per head before layer l + 1 runs - at most one uncompressed layer exists at
    a time.  Online: the budgets need the importance of every layer, i.e. the whole forward pass, so all layers are
    still uncompressed when the last one has run, and eviction only starts after that peak."""
    full = kv_cache_bytes(prompt_tokens, n_kv_heads, head_dim, elem_bytes)
    if online:
        return n_layers * full
    peak, held = 0.0, 0.0
    for l in range(n_layers):
        peak = max(peak, held + full)
        held += kv_cache_bytes(kept_per_head[l], n_kv_heads, head_dim, elem_bytes)
    return max(peak, held)


def stack_batched_block(ctx, B, device, peaks):
    """maskkv_select and maskkv_compact over ALL (layer, head) segments of configs[2] in one call each, with the layer as
    the request axis: 32 x 32 = 1024 segments of 32768 scores (134 MB) and about 261,000 kept rows (269 MB moved) - the
    launch in which the two calls have enough bytes for a bandwidth fraction to mean something.  Every layer's inputs
    are generated from the seed and scored on the device; its scores, masses, keys and values land in the stacked
    tensors.  The loop is the offline schedule of the paper (budgets known before the layer runs), so it also yields
    the kept rows per layer for the peak-memory comparison with the online schedule."""
    wl = synth.config(3)
    L, N, M, Hkv, H, d = wl.n_layers, wl.prompt_lens[0], wl.n_mask, wl.n_kv_heads, wl.n_q_heads, wl.head_dim
    k_layers = B.maskkv_layer_budgets(wl.total_budget(), wl.beta, wl.layer_importance())
    one = LayerBuffers(ctx, B, wl, Hkv * max(k_layers), device)
    pcu = [l * N for l in range(L + 1)]
    lcu = [l * M for l in range(L + 1)]
    p = B.Problem(wl.torch_dtype, H, Hkv, d, pcu, lcu, device)
    scores = torch.empty((Hkv, L * N), dtype=torch.float32, device=device)
    mass_p = torch.empty((L, Hkv), dtype=torch.float32, device=device)
    mass_m = torch.empty((L, Hkv), dtype=torch.float32, device=device)
    k_all = torch.empty((L * N, Hkv, d), dtype=wl.torch_dtype, device=device)
    v_all = torch.empty((L * N, Hkv, d), dtype=wl.torch_dtype, device=device)
    for l in range(L):
        x = synth.layer_inputs(wl, l, device)
        ctx.maskkv_score(one.p, x["q_mask"], x["k_prompt"], x["k_mask"], one.scores, one.mass_p, one.mass_m, one.ws)
        scores[:, l * N:(l + 1) * N] = one.scores
        mass_p[l] = one.mass_p[0]
        mass_m[l] = one.mass_m[0]
        k_all[l * N:(l + 1) * N] = x["k_prompt"]
        v_all[l * N:(l + 1) * N] = x["v_prompt"]
        del x
    capacity = Hkv * sum(k_layers)
    k_l_dev = torch.tensor(k_layers, dtype=torch.int32, device=device)
    budgets = torch.empty((L, Hkv), dtype=torch.int32, device=device)
    offsets = torch.zeros(L * Hkv + 1, dtype=torch.int32, device=device)
    kept = torch.empty(capacity, dtype=torch.int32, device=device)
    kc = torch.empty((capacity, d), dtype=wl.torch_dtype, device=device)
    vc = torch.empty_like(kc)
    ctx.maskkv_budget(p, 0, wl.alpha, mass_p, mass_m, capacity, budgets, offsets, k_l_dev)
    ctx.maskkv_select(p, scores, budgets, offsets, kept)
    ctx.maskkv_compact(p, k_all, v_all, kept, offsets, capacity, kc, vc)
    torch.cuda.synchronize()
    rows = int(offsets[-1].item())
    kept_per_layer = budgets.sum(1).cpu().tolist()
    work = {"select": 4.0 * L * N * Hkv + 4.0 * rows, "compact": (4.0 * d * 2 + 4.0) * rows}
    calls = {"select": lambda: ctx.maskkv_select(p, scores, budgets, offsets, kept),
             "compact": lambda: ctx.maskkv_compact(p, k_all, v_all, kept, offsets, capacity, kc, vc)}
    scratch = torch.empty(256 << 20, dtype=torch.uint8, device=device)
    hbm = peaks["hbm_gbs"]
    out = {"workload": f"configs[2] llada_stack_32k, all {L} layers in one call (layer = request axis): {L * Hkv} segments of {N} scores, "
                       f"{rows} kept rows; warm = 20 calls back to back (inputs of {work['select'] / 1e6:.0f} / {work['compact'] / 1e6:.0f} MB "
                       "exceed the L2 anyway), cold = 256 MB written before each call"}
    for name, call in calls.items():
        warm_us = timed_loop(lambda i: call(), 20)
        cold = []
        for i in range(10):
            scratch.fill_(i)
            c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            c0.record()
            call()
            c1.record()
            torch.cuda.synchronize()
            cold.append(1e3 * c0.elapsed_time(c1))
        cold_us = statistics.median(cold)
        out[name] = {"bound": "hbm", "bytes": work[name], "warm_us": round(warm_us, 2), "cold_us": round(cold_us, 2),
                     "warm_GB/s": round(work[name] / (warm_us * 1e-6) / 1e9, 1), "cold_GB/s": round(work[name] / (cold_us * 1e-6) / 1e9, 1),
                     "peak": hbm, "warm_frac_of_hbm_peak": round(work[name] / (warm_us * 1e-6) / 1e9 / hbm, 3),
                     "cold_frac_of_hbm_peak": round(work[name] / (cold_us * 1e-6) / 1e9 / hbm, 3)}
    out["status_flags"] = ctx.maskkv_check_status()
    # peak prompt-KV bytes of the first step under the two schedules of the paragraph after Eq. 13
    per_head = [r / Hkv for r in kept_per_layer]
    off_peak = kv_peak_bytes(L, N, per_head, Hkv, d, online=False)
    on_peak = kv_peak_bytes(L, N, per_head, Hkv, d, online=True)
    schedules = {"offline_profile_peak_bytes": off_peak, "online_peak_bytes": on_peak, "ratio": on_peak / off_peak,
                 "after_eviction_bytes": sum(kv_cache_bytes(k, Hkv, d) for k in per_head),
                 "kept_rows_per_layer": [int(r) for r in kept_per_layer],
                 "note": "prompt K/V of the 32-layer stack held during the first denoising step; offline = each layer compacted "
                         "before the next one runs (budgets from a precomputed importance profile), online = budgets need "
                         "every layer's importance, so nothing can be evicted before the whole stack is resident"}
    return out, schedules


def bench_ours(args):
    rank, world, local_rank = rank_world()
    import torch.distributed as dist
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the MaskKV path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    from paper_2510_09309_b200 import binding as B
    ctx = B.Context(local_rank)

    wl = synth.config(3)
    N = wl.prompt_lens[0]
    k_layers = B.maskkv_layer_budgets(wl.total_budget(), wl.beta, wl.layer_importance())
    my_layers = shard_layers(wl.n_layers, rank, world)
    # one rank keeps a boundary/middle mix resident; with several ranks each keeps four of its own layers
    resident = list(RESIDENT_LAYERS) if world == 1 else (my_layers * 4)[:4]
    capacity = wl.n_kv_heads * max(k_layers)                      # the host-side bound on rows per layer
    inputs = [synth.layer_inputs(wl, l, device) for l in resident]
    lives = [synth.live_inputs(wl, l, 0, device) for l in resident]
    for x in inputs:
        x.pop("planted", None); x.pop("v_mask", None)
    buf = LayerBuffers(ctx, B, wl, capacity, device)
    torch.cuda.synchronize()

    def step(i, events=None):
        j = i % len(resident)
        run_layer(ctx, buf, inputs[j], lives[j], k_layers[resident[j]], wl.alpha, events)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing
    sampler = ClockSampler(local_rank) if rank == 0 else None   # samples through warm-up, the timed region and the e2e leg
    for i in range(args.warmup):
        step(i)
    barrier()
    # The five calls of a layer allocate nothing and never synchronise, so a layer's step is captured once into a CUDA
    # graph (one per resident layer: the pointers differ) and the timed loop replays the graphs - what a serving loop
    # would do, and it removes the launch gaps between the six kernels.  --no-graph times plain calls instead.
    graphs, launches_per_step, graph_note = None, None, None
    if not args.no_graph:
        try:
            side = torch.cuda.Stream(device=device)
            side.wait_stream(torch.cuda.current_stream())
            graphs = []
            with torch.cuda.stream(side):
                for j in range(len(resident)):
                    before = ctx.maskkv_launch_count()
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g, stream=side):
                        step(j)
                    launches_per_step = ctx.maskkv_launch_count() - before
                    graphs.append(g)
            torch.cuda.current_stream().wait_stream(side)
            for j in range(len(resident)):                            # one replay each, untimed
                graphs[j].replay()
            barrier()
        except Exception as exc:                                       # capture refused: time plain calls and say so
            graphs, graph_note = None, f"graph capture failed ({str(exc)[:80]}); plain calls timed"
            torch.cuda.synchronize()

    def timed_step(i):
        if graphs is not None:
            graphs[i % len(resident)].replay()
        else:
            step(i)

    launches0 = ctx.maskkv_launch_count()
    barrier()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if sampler: sampler.mark("timed_start")
    t0.record()
    for i in range(args.steps):
        timed_step(args.warmup + i)
    t1.record()
    barrier()
    if sampler: sampler.mark("timed_end")
    launches = (launches_per_step * args.steps) if graphs is not None else (ctx.maskkv_launch_count() - launches0)
    elapsed_ms = max_over_ranks(t0.elapsed_time(t1), device)
    # the same steps as plain calls, for comparison (shorter run)
    eager_steps = min(args.steps, 300)
    barrier()
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    g0.record()
    for i in range(eager_steps):
        step(args.warmup + i)
    g1.record()
    barrier()
    eager_ms_per_step = max_over_ranks(g0.elapsed_time(g1), device) / eager_steps
    # Per-call breakdown from a separate pass: an event between every two calls costs a few microseconds of
    # serialisation per step, which does not belong in the headline number.
    per_call = [[torch.cuda.Event(enable_timing=True) for _ in range(6)] for _ in range(min(args.steps, 200))]
    for i, ev in enumerate(per_call):
        step(args.warmup + i, ev)
    barrier()
    mean_kept = float(buf.offsets[-1].item()) / wl.n_kv_heads
    call_us = {name: 1e3 * statistics.mean(ev[c].elapsed_time(ev[c + 1]) for ev in per_call) for c, name in enumerate(CALLS)}
    # ---- the later denoising steps: maskkv_attend alone, back to back, as the per-step loop of a layer would issue it.
    # The compacted cache is cloned until the copies exceed twice the L2, and the loop cycles through them.
    cache_bytes = 2 * buf.kc.numel() * buf.kc.element_size()
    n_copies = max(2, int(-(-2 * 126e6 // cache_bytes)))
    caches = [(buf.kc.clone(), buf.vc.clone()) for _ in range(n_copies)]
    p = buf.p

    def attend_step(i):
        kc, vc = caches[i % n_copies]
        live = lives[i % len(lives)]
        ctx.maskkv_attend(p, live["q_live"], live["k_live"], live["v_live"], kc, vc, buf.offsets, buf.capacity, buf.out)

    for i in range(5):
        attend_step(i)
    barrier()
    a_steps = min(max(args.steps, 50), 400)
    a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a0.record()
    for i in range(a_steps):
        attend_step(i)
    a1.record()
    barrier()
    attend_loop_us = 1e3 * max_over_ranks(a0.elapsed_time(a1), device) / a_steps
    attend_plain_us = attend_loop_us
    n_attend_graphs = n_copies                               # graph j: cache copy j, live set j % len(lives)
    if not args.no_graph and n_attend_graphs <= 64:
        replayed = replayed_loop_us(attend_step, n_attend_graphs, a_steps, device)
        if replayed is not None:
            attend_loop_us = max_over_ranks(replayed, device)
    # the same step with partial refresh: a quarter of the live rows have queries (maskkv_attend_rows)
    n_rows = max(1, wl.n_mask // 4)
    rows_cu = [r * n_rows for r in range(wl.n_requests + 1)]
    rows_cu_dev = torch.tensor(rows_cu, dtype=torch.int32, device=device)
    q_rows = [torch.cat([lv["q_live"][r * wl.n_mask:r * wl.n_mask + n_rows] for r in range(wl.n_requests)]).contiguous() for lv in lives]
    out_rows = torch.empty_like(q_rows[0])

    def attend_rows_step(i):
        kc, vc = caches[i % n_copies]
        live = lives[i % len(lives)]
        ctx.maskkv_attend_rows(p, q_rows[i % len(lives)], rows_cu, rows_cu_dev, live["k_live"], live["v_live"], kc, vc, buf.offsets,
                               buf.capacity, out_rows)

    for i in range(5):
        attend_rows_step(i)
    barrier()
    r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    r0.record()
    for i in range(a_steps):
        attend_rows_step(i)
    r1.record()
    barrier()
    attend_rows_us = 1e3 * max_over_ranks(r0.elapsed_time(r1), device) / a_steps
    if not args.no_graph and n_attend_graphs <= 64:
        replayed = replayed_loop_us(attend_rows_step, n_attend_graphs, a_steps, device)
        if replayed is not None:
            attend_rows_us = max_over_ranks(replayed, device)
    del caches
    # The loop above ran on the cache of the layer the last step left behind (a boundary layer, the larger budget at
    # one rank).  Most layers are middle layers with the smaller budget: compress one and time its step too.
    attend_mid = None
    mid = [j for j in range(len(resident)) if k_layers[resident[j]] == min(k_layers[l] for l in resident)]
    if mid and k_layers[resident[mid[0]]] != k_layers[resident[(args.warmup + len(per_call) - 1) % len(resident)]]:
        step(mid[0])
        barrier()
        mid_kept = float(buf.offsets[-1].item()) / wl.n_kv_heads
        caches = [(buf.kc.clone(), buf.vc.clone()) for _ in range(n_copies)]
        for i in range(5):
            attend_step(i)
        barrier()
        m0, m1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        m0.record()
        for i in range(a_steps):
            attend_step(i)
        m1.record()
        barrier()
        mid_plain = 1e3 * max_over_ranks(m0.elapsed_time(m1), device) / a_steps
        mid_us = mid_plain
        if not args.no_graph and n_attend_graphs <= 64:
            replayed = replayed_loop_us(attend_step, n_attend_graphs, a_steps, device)
            if replayed is not None:
                mid_us = max_over_ranks(replayed, device)
        attend_mid = {"us": round(mid_us, 2), "plain_calls_us": round(mid_plain, 2), "mean_kept_per_head": mid_kept,
                      "layer": resident[mid[0]]}
        del caches
        step(args.warmup + len(per_call) - 1)                          # leave the buffers as the later sections expect them
        barrier()
    # maskkv_score alone, launched the way the timed steps launch it (graph replays cycling the resident layers): the
    # duration the roofline objects use
    score_us = None
    if graphs is not None:
        side2 = torch.cuda.Stream(device=device)
        side2.wait_stream(torch.cuda.current_stream())
        sgraphs = []
        with torch.cuda.stream(side2):
            for j in range(len(resident)):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=side2):
                    ctx.maskkv_score(buf.p, inputs[j]["q_mask"], inputs[j]["k_prompt"], inputs[j]["k_mask"], buf.scores,
                                     buf.mass_p, buf.mass_m, buf.ws)
                sgraphs.append(g)
        torch.cuda.current_stream().wait_stream(side2)
        for g in sgraphs:
            g.replay()
        barrier()
        s_steps = min(args.steps, 400)
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s0.record()
        for i in range(s_steps):
            sgraphs[i % len(resident)].replay()
        s1.record()
        barrier()
        score_us = 1e3 * max_over_ranks(s0.elapsed_time(s1), device) / s_steps
        del sgraphs
    flags = ctx.maskkv_check_status()

    # ---- end to end: the layer's inputs start in pinned host memory, results end in host memory
    keys_in = ("q_mask", "k_prompt", "v_prompt", "k_mask")
    keys_live = ("q_live", "k_live", "v_live")
    host_x = {k: inputs[0][k].cpu().pin_memory() for k in keys_in}
    host_l = {k: lives[0][k].cpu().pin_memory() for k in keys_live}
    dev_x = {k: torch.empty_like(inputs[0][k]) for k in keys_in}
    dev_l = {k: torch.empty_like(lives[0][k]) for k in keys_live}
    host_out = torch.empty_like(buf.out, device="cpu").pin_memory()
    host_bud = torch.empty_like(buf.budgets, device="cpu").pin_memory()
    h2d = sum(t.numel() * t.element_size() for t in list(host_x.values()) + list(host_l.values()))
    d2h = host_out.numel() * host_out.element_size() + host_bud.numel() * host_bud.element_size()

    def e2e_step(i):
        for k in keys_in:
            dev_x[k].copy_(host_x[k], non_blocking=True)
        for k in keys_live:
            dev_l[k].copy_(host_l[k], non_blocking=True)
        run_layer(ctx, buf, dev_x, dev_l, k_layers[resident[0]], wl.alpha)
        host_out.copy_(buf.out, non_blocking=True)
        host_bud.copy_(buf.budgets, non_blocking=True)

    e2e_steps = max(3, min(args.steps, 50))
    for i in range(2):
        e2e_step(i)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(e2e_steps):
        e2e_step(i)
    e1.record()
    barrier()
    e2e_ms = max_over_ranks(e0.elapsed_time(e1), device)

    # ---- the same, with the prompt values left in pinned host memory: only the kept rows of V are ever needed on the
    # device (maskkv_compact is the one reader of v_prompt), so the gather reads them straight from host memory and the
    # evicted rows never cross the bus.  Reported next to the standard number, not instead of it.
    def e2e_lazy_step(i):
        for k in keys_in:
            if k != "v_prompt":
                dev_x[k].copy_(host_x[k], non_blocking=True)
        for k in keys_live:
            dev_l[k].copy_(host_l[k], non_blocking=True)
        p = buf.p
        ctx.maskkv_score(p, dev_x["q_mask"], dev_x["k_prompt"], dev_x["k_mask"], buf.scores, buf.mass_p, buf.mass_m, buf.ws)
        ctx.maskkv_budget(p, k_layers[resident[0]], wl.alpha, buf.mass_p, buf.mass_m, buf.capacity, buf.budgets, buf.offsets)
        ctx.maskkv_select(p, buf.scores, buf.budgets, buf.offsets, buf.kept, buf.ws)
        ctx.maskkv_compact(p, dev_x["k_prompt"], host_x["v_prompt"], buf.kept, buf.offsets, buf.capacity, buf.kc, buf.vc)
        ctx.maskkv_attend(p, dev_l["q_live"], dev_l["k_live"], dev_l["v_live"], buf.kc, buf.vc, buf.offsets, buf.capacity, buf.out)
        host_out.copy_(buf.out, non_blocking=True)
        host_bud.copy_(buf.budgets, non_blocking=True)

    e2e_lazy = None
    try:
        ref_out = buf.out.clone()
        for i in range(2):
            e2e_lazy_step(i)
        barrier()
        same = bool(torch.equal(ref_out, buf.out))
        z0, z1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        z0.record()
        for i in range(e2e_steps):
            e2e_lazy_step(i)
        z1.record()
        barrier()
        lazy_ms = max_over_ranks(z0.elapsed_time(z1), device)
        v_bytes = host_x["v_prompt"].numel() * host_x["v_prompt"].element_size()
        kept_v_bytes = int(buf.offsets[-1].item()) * wl.head_dim * host_x["v_prompt"].element_size()
        e2e_lazy = {"value": world * N / (lazy_ms / e2e_steps * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": h2d - v_bytes + kept_v_bytes, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
                    "same_output_as_copied_v": same,
                    "note": "v_prompt stays in pinned host memory; maskkv_compact reads the kept rows from there"}
    except Exception as exc:                                           # a platform without device access to pinned memory
        e2e_lazy = {"unavailable": str(exc)[:120]}
    clocks = sampler.stop() if sampler else {}

    # ---- select / compact / attend on a batch: at one layer they are launch- and latency-bound whatever the kernel does
    # (4-17 MB per call), so a fraction of the memory roof only shows when many segments go into one launch
    blocks = set(args.blocks.split(",")) if args.blocks else set()
    batched = batched_calls(ctx, B, device) if rank == 0 and "batched" in blocks else None
    dream = dream_gqa_block(ctx, B, device, load_peaks()) if rank == 0 and "dream" in blocks else None
    stack, schedules = stack_batched_block(ctx, B, device, load_peaks()) if rank == 0 and "stack" in blocks else (None, None)

    # ---- calibration step of the budget rule (Eq. 8), outside the timed step: a streaming reduction bound by HBM
    importance = None
    if rank == 0 and "extras" in blocks:
        n_tok, hidden = N + wl.n_mask, 4096                       # one LLaDA-8B-shaped layer: 541 MB read per call
        g = torch.Generator(device=device); g.manual_seed(synth.BASE_SEED + 8)
        h_in = torch.randn(n_tok, hidden, generator=g, device=device).bfloat16()
        h_out = (h_in.float() + 0.5 * torch.randn(n_tok, hidden, generator=g, device=device)).bfloat16()
        imp_out = torch.zeros(1, dtype=torch.float32, device=device)
        imp_ws = ctx.maskkv_layer_importance(h_in, h_out, imp_out)
        reps = 20
        for _ in range(3):
            ctx.maskkv_layer_importance(h_in, h_out, imp_out, imp_ws)
        torch.cuda.synchronize()
        i0, i1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        i0.record()
        for _ in range(reps):
            ctx.maskkv_layer_importance(h_in, h_out, imp_out, imp_ws)
        i1.record()
        torch.cuda.synchronize()
        imp_us = 1e3 * i0.elapsed_time(i1) / reps
        imp_bytes = 2.0 * n_tok * hidden * 2
        importance = {"workload": f"{n_tok} tokens x hidden {hidden}, bf16", "us": imp_us, "bytes": imp_bytes,
                      "value": float(imp_out.item())}
        # the response-token refresh test of the per-step loop: cos(V_t, V_t-1) < delta over the live rows of one
        # layer (256 x 4096: a latency-bound pair of launches) and over the same big tensors (HBM-bound)
        r_idx = torch.zeros(n_tok, dtype=torch.int32, device=device)
        r_cnt = torch.zeros(1, dtype=torch.int32, device=device)
        refresh = {}
        for name, rows, reps in (("one_layer_256_rows", wl.n_mask, 200), ("33k_rows", n_tok, 20)):
            a, b = h_in[:rows], h_out[:rows]
            for _ in range(3):
                ctx.maskkv_refresh_set(a, b, 0.9, r_idx, r_cnt)
            torch.cuda.synchronize()
            r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            r0.record()
            for _ in range(reps):
                ctx.maskkv_refresh_set(a, b, 0.9, r_idx, r_cnt)
            r1.record()
            torch.cuda.synchronize()
            us = 1e3 * r0.elapsed_time(r1) / reps
            gbs = 2.0 * rows * hidden * 2 / (us * 1e-6) / 1e9
            refresh[name] = {"us": round(us, 2), "GB/s": round(gbs, 1), "frac_of_hbm_peak": round(gbs / load_peaks()["hbm_gbs"], 3),
                             "refreshed": int(r_cnt.item())}
        importance["refresh_set"] = refresh
        del h_in, h_out
        # the mask-only vocabulary projection of the per-step loop: 256 masked rows x width 4096 x vocabulary 126,464
        # (LLaDA-8B's output embedding, 1.04 GB read once per call); a dense contraction on the tensor cores
        px = synth.project_inputs(n_tok, hidden, 126464, wl.n_mask, device, seed=1)
        p_ws = torch.empty(B.maskkv_mask_project_workspace_bytes(wl.n_mask, hidden), dtype=torch.uint8, device=device)
        project = {"workload": f"{wl.n_mask} masked rows of {n_tok} x width {hidden} x vocabulary 126464, bf16 operands"}
        p_flops = 2.0 * wl.n_mask * hidden * 126464
        for name, odt, osz in (("bf16_logits", torch.bfloat16, 2), ("fp32_logits", torch.float32, 4)):
            logits = torch.empty((wl.n_mask, 126464), dtype=odt, device=device)
            reps = 20
            for _ in range(3):
                ctx.maskkv_mask_project(px["hidden"], px["w_vocab"], logits, px["positions"], p_ws)
            torch.cuda.synchronize()
            p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            p0.record()
            for _ in range(reps):
                ctx.maskkv_mask_project(px["hidden"], px["w_vocab"], logits, px["positions"], p_ws)
            p1.record()
            torch.cuda.synchronize()
            us = 1e3 * p0.elapsed_time(p1) / reps
            p_bytes = 126464.0 * hidden * 2 + wl.n_mask * 126464.0 * osz + 2.0 * wl.n_mask * hidden * 2
            tf = p_flops / (us * 1e-6) / 1e12
            peak_tf = load_peaks()["bf16_tflops_sustained"]
            project[name] = {"us": round(us, 2),
                             "roofline": {"bound": "tensor", "achieved": round(tf, 1), "peak": peak_tf, "unit": "TFLOP/s",
                                          "frac": round(tf / peak_tf, 3), "frac_sustained": round(tf / peak_tf, 3),
                                          "frac_burst": round(tf / load_peaks()["bf16_tflops"], 3),
                                          "peak_source": "frac = of the sustained bf16 peak; 20 back-to-back calls (4.5 ms)"},
                             "hbm_GB/s": round(p_bytes / (us * 1e-6) / 1e9, 1),
                             "frac_of_hbm_peak": round(p_bytes / (us * 1e-6) / 1e9 / load_peaks()["hbm_gbs"], 3)}
            del logits
        importance["mask_project"] = project
        del px, p_ws

    if world > 1:
        dist.destroy_process_group()
    if rank != 0:
        return None

    ms_per_step = elapsed_ms / args.steps
    value = world * N / (ms_per_step * 1e-3)
    peaks = load_peaks()
    work = algorithmic_work(wl, mean_kept)
    score_s = (score_us if score_us is not None else call_us["score"]) * 1e-6
    achieved_tf = work["score_flops"] / score_s / 1e12
    peak_tf = peaks["bf16_tflops_sustained"]
    # the score-alone loop is a few hundred back-to-back calls (tens of milliseconds): the burst peak is the fairer
    # denominator for the default short runs, the sustained one for seconds-long loops; both are reported
    peak_burst_tf = peaks["bf16_tflops"]
    hbm = peaks["hbm_gbs"]
    other = {
        "score_hbm": {"bound": "hbm", "achieved": work["score_bytes"] / score_s / 1e9, "peak": hbm, "unit": "GB/s"},
        "select": {"bound": "hbm", "achieved": work["select_bytes"] / (call_us["select"] * 1e-6) / 1e9, "peak": hbm, "unit": "GB/s"},
        "compact": {"bound": "hbm", "achieved": work["compact_bytes"] / (call_us["compact"] * 1e-6) / 1e9, "peak": hbm, "unit": "GB/s"},
        "attend": {"bound": "hbm", "achieved": work["attend_bytes"] / (call_us["attend"] * 1e-6) / 1e9, "peak": hbm, "unit": "GB/s",
                   "tflops": work["attend_flops"] / (call_us["attend"] * 1e-6) / 1e12},
    }
    for v in other.values():
        v["frac"] = v["achieved"] / v["peak"]
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "configs[2] llada_stack_32k, one layer per step: N=32768 M=256 H=H_kv=32 d=128, "
                               "adaptive budgets (k_l 512/238, alpha=0.1)", "layers_resident": len(resident),
                   "l2": "inputs 545 MB per step > 126 MB L2; resident layers are cycled", "calls": list(CALLS),
                   "launch": "one CUDA graph per resident layer, replayed" if graphs is not None else (graph_note or "plain calls")},
        "ms_per_step_plain_calls": eager_ms_per_step,
        "call_us": {k: round(v, 2) for k, v in call_us.items()},
        "attend_step_us": round(attend_loop_us, 2),
        "attend_step": {"us": round(attend_loop_us, 2), "plain_calls_us": round(attend_plain_us, 2),
                        "launch": ("the steps over all cache copies captured in one CUDA graph, replayed" if attend_loop_us != attend_plain_us
                                   else "plain calls"),
                        "steps": a_steps, "mean_kept_per_head": mean_kept,
                        "l2": f"{n_copies} copies of the compacted cache ({cache_bytes * n_copies / 1e6:.0f} MB) cycled",
                        "partial_refresh_us": round(attend_rows_us, 2),
                        "partial_refresh": f"{n_rows} of {wl.n_mask} live rows have queries (maskkv_attend_rows)",
                        "middle_layer": attend_mid},
        "kv_cache": {"prompt_bytes_per_layer": kv_cache_bytes(N, wl.n_kv_heads, wl.head_dim),
                     "compacted_bytes_per_layer": kv_cache_bytes(mean_kept, wl.n_kv_heads, wl.head_dim),
                     "ratio": N / max(mean_kept, 1e-9), "formula": "2 * tokens * heads * d_head * 2 bytes per layer"},
        "compress_tokens_per_s": N / (1e-6 * (call_us["score"] + call_us["budget"] + call_us["select"] + call_us["compact"])),
        "e2e": {"value": world * N / (e2e_ms / e2e_steps * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": e2e_steps},
        "e2e_v_in_host_memory": e2e_lazy,
        "gpu_launches": int(launches),
        "clocks": clocks,
        "status_flags": flags,
        "roofline_tensor": {"kernel": "maskkv_score (its two kernels, replayed alone; one Q K^T product counted)", "bound": "tensor",
                     "achieved": achieved_tf, "peak": peak_tf, "unit": "TFLOP/s", "frac": achieved_tf / peak_tf,
                     "frac_sustained": achieved_tf / peak_tf, "frac_burst": achieved_tf / peak_burst_tf, "peak_burst": peak_burst_tf,
                     "peak_source": peaks["source"] + " (frac = of the sustained bf16 peak; frac_burst = of the burst peak)",
                     "traffic": SCORE_DRAM_TRAFFIC_BYTES, "traffic_source": SCORE_DRAM_TRAFFIC_SOURCE,
                     "algorithmic_bytes": work["score_bytes"], "executed_over_algorithmic_flops": 2.0},
        "roofline": dict(exp_roofline(wl, score_s * 1e6, clocks.get("sm_max_mhz") or 1965.0, measure_exp_rate(ctx, device)),
                         traffic=SCORE_DRAM_TRAFFIC_BYTES, traffic_source=SCORE_DRAM_TRAFFIC_SOURCE,
                         algorithmic_bytes=work["score_bytes"],
                         why=("the two sweeps of maskkv_score are bound by the special-function unit: every logit is "
                              "exponentiated once per sweep; with one MMA k-step of eight the call is 6 % faster, with the "
                              "exponentials removed 30 % (timing probes in csrc/score_tc.cu); the tensor-core view of the same "
                              "call is roofline_tensor")),
        "score_us": round(score_s * 1e6, 2),
        "roofline_other_calls": other,
        "mean_kept_per_head": mean_kept,
    }
    if batched is not None:
        line["batched_calls"] = batched
    if dream is not None:
        line["dream_gqa_16k"] = dream
    if stack is not None:
        line["stack_batched"] = stack
        line["kv_peak_first_step"] = schedules
    if importance is not None:
        gbs = importance["bytes"] / (importance["us"] * 1e-6) / 1e9
        line["refresh_set"] = importance.pop("refresh_set", None)
        line["mask_project"] = importance.pop("mask_project", None)
        line["layer_importance"] = {"workload": importance["workload"], "us": round(importance["us"], 2),
                                    "roofline": {"bound": "hbm", "achieved": gbs, "peak": hbm, "unit": "GB/s", "frac": gbs / hbm}}
    line["cpu_baseline"] = oracle_baseline(wl, budget_s=15.0)
    return line


def measure_exp_rate(ctx, device):
    """Exponentials per second of the special-function units, measured live: the library's stand-alone kernel (nothing
    but ex2.approx.ftz.f32 in eight independent chains per thread, two CTAs of 1024 threads per SM), about a millisecond
    per launch, best of five after a warm-up."""
    scratch = torch.zeros(4, dtype=torch.float32, device=device)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    best = 0.0
    for it in range(6):
        e0.record()
        n = ctx.maskkv_selftest_exp_rate(4000, scratch)
        e1.record()
        torch.cuda.synchronize()
        if it > 0:
            best = max(best, n / (e0.elapsed_time(e1) * 1e-3))
    return best


def exp_roofline(wl, score_us, sm_max_mhz, measured_rate=None):
    """The unit that actually bounds maskkv_score: every logit is exponentiated once per sweep (row statistics, then
    weights) on the special-function unit, 16 results per clock per SM on 148 SMs.  `peak` is the rate measured in this
    run by the stand-alone kernel when there is one, else the nominal count at the maximum SM clock."""
    N, M, H = wl.prompt_lens[0], wl.n_mask, wl.n_q_heads
    exps = 2.0 * M * (N + M) * H
    achieved = exps / (score_us * 1e-6) / 1e12
    nominal = 148 * 16 * sm_max_mhz * 1e6 / 1e12
    peak = measured_rate / 1e12 if measured_rate else nominal
    return {"kernel": "maskkv_score (its two kernels, replayed alone)", "bound": "alu", "achieved": achieved, "peak": peak, "unit": "Texp/s",
            "frac": achieved / peak, "peak_nominal": nominal, "frac_of_nominal": achieved / nominal,
            "peak_source": ("measured in this run: maskkv_selftest_exp_rate, a kernel of nothing but ex2.approx.ftz.f32"
                            if measured_rate else "148 SMs x 16 ex2 per clock x max SM clock (nominal unit count)")}


# ----------------------------------------------------------------------------- peaks and the CPU oracle
def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def oracle_threads() -> int:
    """Threads the oracle's numpy calls actually use: the size of the BLAS pool numpy is linked against (its matrix
    products are the only multi-threaded part); the host's core count if that cannot be read."""
    try:
        from threadpoolctl import threadpool_info
        import numpy  # noqa: F401  (the pools are listed once the library is loaded)
        pools = [int(i["num_threads"]) for i in threadpool_info() if i.get("user_api") == "blas"]
        if pools:
            return max(pools)
    except Exception:
        pass
    return os.cpu_count() or 1


def oracle_sample(wl, n_heads: int, layer: int = 0):
    """The workload restricted to its first `n_heads` heads (same per-head cost), generated on the CPU."""
    sub = synth.scaled(wl, wl.name + f"_first{n_heads}heads", n_q_heads=n_heads, n_kv_heads=n_heads, n_layers=wl.n_layers)
    x = synth.layer_inputs(sub, layer, "cpu")
    live = synth.live_inputs(sub, layer, 0, "cpu")
    return sub, x, live


def oracle_pass(sub, x, live, k_l):
    """One pass of the whole path in the CPU oracle (as it stands); returns seconds."""
    import numpy as np
    from oracle import maskkv_oracle as O
    t = time.perf_counter()
    pcu, lcu = sub.prompt_cu(), sub.live_cu()
    sc, mp, mm = O.score(x["q_mask"], x["k_prompt"], x["k_mask"], pcu, lcu)
    bud, off = O.head_budgets(mp.astype(np.float32), mm.astype(np.float32), k_l, sub.alpha, sub.prompt_lens)
    idx, _ = O.select(sc.astype(np.float32), bud, pcu)
    kc, vc = O.compact(x["k_prompt"], x["v_prompt"], idx, off, pcu)
    O.attend(live["q_live"], live["k_live"], live["v_live"], kc, vc, off, lcu, sub.n_kv_heads)
    return time.perf_counter() - t


def oracle_baseline(wl, budget_s: float):
    """Times the oracle on a bounded sample (a few heads of one layer) and scales to a whole layer."""
    N, H = wl.prompt_lens[0], wl.n_q_heads
    sub, x, live = oracle_sample(wl, 1)
    t1 = oracle_pass(sub, x, live, 238)
    n_heads = int(max(1, min(H, budget_s / max(t1, 1e-3))))
    if n_heads > 1:
        sub, x, live = oracle_sample(wl, n_heads)
        t = oracle_pass(sub, x, live, 238)
    else:
        t = t1
    return {"value": N / (t * H / n_heads), "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
            "sample": f"{n_heads} of {H} heads of one 32k layer through the whole path (fp64 numpy), {t:.2f} s; "
                      f"scaled to a full layer by {H}/{n_heads}", "host_cores": os.cpu_count()}


REFERENCE_BUDGET_S = 150.0     # host time the whole reference run may take (calibration pass included)


def bench_reference(args):
    """The oracle, as it stands, on the host cores.  A step is one head of one 32k layer through the whole path; when
    --steps is so large that whole heads would not fit the time budget, a step is one head over the first n_keys prompt
    keys (the oracle's cost is linear in the keys) and the result is scaled by N / n_keys as well."""
    rank, world, _ = rank_world()
    if rank != 0:
        return None
    wl = synth.config(3)
    N, H = wl.prompt_lens[0], wl.n_q_heads
    n_heads = 1
    sub, x, live = oracle_sample(wl, n_heads)
    oracle_pass(sub, x, live, 238)                                   # first call pays for page-ins and imports
    t_head = oracle_pass(sub, x, live, 238)                          # calibration, untimed
    target = REFERENCE_BUDGET_S / (args.steps + args.warmup + 2)
    n_keys = N
    if t_head > target:
        n_keys = max(1024, int(N * target / t_head) // 128 * 128)
        sub = synth.scaled(wl, wl.name + "_first_head_truncated", n_q_heads=1, n_kv_heads=1, n_layers=wl.n_layers,
                           prompt_lens=(n_keys,))
        x = synth.layer_inputs(sub, 0, "cpu")
        live = synth.live_inputs(sub, 0, 0, "cpu")
    k_l = min(238, n_keys)
    for _ in range(args.warmup):
        oracle_pass(sub, x, live, k_l)
    times = [oracle_pass(sub, x, live, k_l) for _ in range(args.steps)]
    t = sum(times) / len(times)
    scale = (H / n_heads) * (N / n_keys)
    value = N / (t * scale)
    sample = (f"each step = {n_heads} of {H} heads of one 32k layer, first {n_keys} of {N} prompt keys, through the whole path "
              f"(fp64 numpy oracle); scaled by {scale:g}")
    return {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * t * scale, "ms_per_step_is": f"extrapolated: measured {1e3 * t:.1f} ms per sampled step x {scale:g}",
        "ms_per_sampled_step": 1e3 * t, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "configs[2] llada_stack_32k, one layer per step (sampled)", "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }


def launcher_command(n_ranks: int, argv, port: int):
    """The command that starts `n_ranks` ranks of this script on one node, one per GPU (what a driver would type)."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_ranks}", "--master-addr", "127.0.0.1",
            "--master-port", str(port), os.path.abspath(__file__)] + list(argv)


def self_launch(n_ranks: int, argv) -> int:
    """`python bench.py --gpus N` with N > 1 outside a launcher: start the N ranks ourselves and hand back their exit
    code.  NCCL's communicator lines go to stderr (NCCL_DEBUG=INFO unless the caller chose otherwise), so that stdout
    still carries rank 0's one JSON line."""
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "INFO")
    env.setdefault("NCCL_DEBUG_FILE", "/dev/stderr")
    return subprocess.call(launcher_command(n_ranks, argv, port), env=env)


def bench_plumbing(args):
    """The multi-rank plumbing alone (rendezvous, layer sharding, reductions over ranks), on whatever backend the box
    has - gloo on a machine without GPUs: what the CPU tests run through the launcher."""
    import torch.distributed as dist
    rank, world, local_rank = rank_world()
    use_cuda = torch.cuda.is_available() and torch.cuda.device_count() >= world
    device = None
    if world > 1:
        if use_cuda:
            torch.cuda.set_device(local_rank)
            device = torch.device("cuda", local_rank)
            dist.init_process_group("nccl", device_id=device)
        else:
            dist.init_process_group("gloo")
    mine = shard_layers(synth.config(3).n_layers, rank, world)
    slowest = max_over_ranks(10.0 + 5.0 * rank, device)
    total = sum_over_ranks(float(len(mine)), device)
    gathered = [mine]
    if world > 1:
        gathered = [None] * world
        dist.all_gather_object(gathered, mine)
        dist.destroy_process_group()
    if rank != 0:
        return None
    return {"plumbing_only": True, "n_gpus": world, "backend": "nccl" if (use_cuda and world > 1) else ("gloo" if world > 1 else "none"),
            "layers_per_rank": gathered, "layers_total": total, "slowest_rank_time": slowest}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-graph", action="store_true", help="time plain calls instead of replaying CUDA graphs")
    ap.add_argument("--blocks", default="batched,dream,stack,extras",
                    help="side measurements to run after the timed steps (comma list; empty = none): batched = select / compact / "
                         "attend on the ragged serving batch, dream = the Dream-shaped layer, stack = select / compact over all "
                         "1024 segments of the 32-layer stack, extras = layer importance, refresh test, mask-only projection")
    ap.add_argument("--plumbing-only", action="store_true",
                    help="run the multi-rank plumbing (rendezvous, sharding, reductions) and nothing else; needs no GPU")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and "RANK" not in os.environ:
        raise SystemExit(self_launch(args.gpus, sys.argv[1:]))       # not under a launcher: start the ranks ourselves
    if args.plumbing_only:
        line = bench_plumbing(args)
        if line is not None:
            print(json.dumps(line), flush=True)
        return
    if args.impl == "reference":
        args.steps = 3 if args.steps is None else max(1, args.steps)
        args.warmup = 1 if args.warmup is None else max(0, args.warmup)
        line = bench_reference(args)
    else:
        args.steps = 2000 if args.steps is None else max(1, args.steps)
        args.warmup = 5 if args.warmup is None else max(3, args.warmup)
        line = bench_ours(args)
    if line is not None:
        print(json.dumps(line), flush=True)


if __name__ == "__main__":
    main()
