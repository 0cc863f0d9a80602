#!/usr/bin/env python
"""Benchmark of the step-attention hot path (RoPE-append -> split-KV attention -> combine).

A "step" is one pass of the whole path for one transformer layer on the 7B-class workload
(28 query / 4 kv heads, head_dim 128, L = 4096 cached tokens, n = 196 new tokens, bf16).
The run cycles over a ring of independent layer caches whose footprint exceeds the L2, the
way a 28-layer model revisits each layer's cache once per navigation step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

N > 1 (under torchrun) runs N independent replicas (the path has no exchange step); the
printed value is the max over ranks.  One JSON line goes to stdout on rank 0.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2512_10310_b200 import workloads as W
from paper_2512_10310_b200.replicas import aggregate_steps_per_s, max_over_ranks as _max_over_ranks

RING_LAYERS = 32            # independent layer caches cycled through (footprint > L2)
L2_BYTES = 126 * 2 ** 20
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.02):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.dev = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.dev, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.dev, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.dev)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.dev)
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def physical_gpu_index(local_index: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_index])
        except Exception:
            return local_index
    return local_index


# ------------------------------------------------------------------------------------------------
# our arm
# ------------------------------------------------------------------------------------------------

# DRAM bytes (read + write) of one attention launch at this workload, from the ncu capture that
# profiles/attn_pair_kernel_step_7b_L4096.md summarises.  The counters belong to the kernel sources
# as they were then: once one of them changes, the figure is withheld until it is taken again.
K2_DRAM_BYTES_PER_LAUNCH = 10_252_800
K2_SOURCES = ("attn_pair.cuh", "ptx_sm100.cuh", "common.cuh")
K2_SOURCES_SHA256 = "6f7c38c01567322f232d5812107eed20469ee785406c52cd6ea74afc6b542220"


def attention_dram_traffic():
    import hashlib
    h = hashlib.sha256()
    src = os.path.join(os.path.dirname(os.path.abspath(__file__)), "paper_2512_10310_b200", "csrc")
    try:
        for name in K2_SOURCES:
            with open(os.path.join(src, name), "rb") as fh:
                h.update(fh.read())
    except OSError:
        return None
    return K2_DRAM_BYTES_PER_LAUNCH if h.hexdigest() == K2_SOURCES_SHA256 else None


class LayerRing:
    """Device buffers of RING_LAYERS independent layers of the workload + pinned host copies."""

    def __init__(self, B, handle, cfg, dev, layers, random_device_inputs=False):
        self.B, self.h, self.cfg, self.dev = B, handle, cfg, dev
        L, n, Hq, Hkv, D = cfg.cache_len, cfg.num_new, cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim
        self.p = B.step_params(cfg.dtype, Hq, Hkv, D, L, n, L + n, cfg.rope_theta)
        qbytes = B.evlnStepQRotSize(handle, self.p)
        wbytes = B.evlnStepWorkspaceSize(handle, self.p)
        self.splits = B.evlnStepNumSplits(handle, self.p)
        self.layers = []
        dt = cfg.torch_dtype
        for l in range(layers):
            if random_device_inputs:
                # same distribution, drawn on the device (the cache-length sweep needs no host copies)
                gen = torch.Generator(device=dev).manual_seed(cfg.seed * 7919 + l)
                mk = lambda *sh: (torch.randn(*sh, generator=gen, device=dev, dtype=torch.float32) * cfg.input_scale).to(dt)
                self.layers.append(dict(
                    kc=mk(Hkv, L + n, D), vc=mk(Hkv, L + n, D), q=mk(n, Hq, D), k=mk(n, Hkv, D), v=mk(n, Hkv, D),
                    q_rot=torch.empty(qbytes, dtype=torch.uint8, device=dev),
                    ws=torch.empty(wbytes, dtype=torch.uint8, device=dev),
                    out=torch.empty((n, Hq, D), dtype=dt, device=dev)))
                kc = self.layers[-1]["kc"]
                continue
            x = W.make_step_inputs(dataclasses.replace(cfg, seed=cfg.seed * 7919 + l))
            kc = torch.zeros((Hkv, L + n, D), dtype=dt, device=dev)
            vc = torch.zeros((Hkv, L + n, D), dtype=dt, device=dev)
            kc[:, :L] = x["k_cache"].to(dev).permute(1, 0, 2)
            vc[:, :L] = x["v_cache"].to(dev).permute(1, 0, 2)
            # the new tokens arrive as one fused [n, Hq + 2 Hkv, D] buffer (what a QKV projection
            # leaves); the calls take its three strided views
            host_qkv = torch.cat([x["q_new"], x["k_new"], x["v_new"]], dim=1).contiguous().pin_memory()
            qkv = host_qkv.to(dev)
            host_in = [host_qkv]
            self.layers.append(dict(
                kc=kc, vc=vc, qkv=qkv, q=qkv[:, :Hq], k=qkv[:, Hq:Hq + Hkv], v=qkv[:, Hq + Hkv:],
                q_rot=torch.empty(qbytes, dtype=torch.uint8, device=dev),
                ws=torch.empty(wbytes, dtype=torch.uint8, device=dev),
                out=torch.empty((n, Hq, D), dtype=dt, device=dev),
                host_in=host_in,
                host_out=torch.empty((n, Hq, D), dtype=dt).pin_memory(),
            ))
        self.bytes_per_layer = 2 * kc.numel() * kc.element_size()

    def step(self, l):
        B, y = self.B, self.layers[l]
        B.evlnRopeAppend(self.h, self.p, y["q"], y["k"], y["v"], y["q_rot"], y["kc"], y["vc"])
        B.evlnStepAttention(self.h, self.p, y["q_rot"], y["kc"], y["vc"], y["ws"])
        B.evlnStepCombine(self.h, self.p, y["ws"], y["out"], None)

    def attention_only(self, l):
        y = self.layers[l]
        self.B.evlnStepAttention(self.h, self.p, y["q_rot"], y["kc"], y["vc"], y["ws"])

    def step_e2e(self, l, s_in=None, s_out=None):
        """Host buffers in, host buffer out.  With side streams the host-to-device copies, the
        kernels and the device-to-host copy of consecutive steps overlap (each step still waits for
        its own inputs and is followed by its own read-back)."""
        y = self.layers[l]
        cur = torch.cuda.current_stream()
        with torch.cuda.stream(s_in if s_in is not None else cur):
            y["qkv"].copy_(y["host_in"][0], non_blocking=True)
        if s_in is not None:
            cur.wait_stream(s_in)
        self.step(l)
        if s_out is not None:
            s_out.wait_stream(cur)
        with torch.cuda.stream(s_out if s_out is not None else cur):
            y["host_out"].copy_(y["out"], non_blocking=True)

    def capture_e2e(self):
        """One CUDA graph of a pass over the ring through the public calls with host buffers:
        copies in on one stream, kernels on the capture stream, copies out on a third."""
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            cur = torch.cuda.current_stream()
            s_in.wait_stream(cur)
            s_out.wait_stream(cur)
            for l in range(len(self.layers)):
                self.step_e2e(l, s_in, s_out)
            cur.wait_stream(s_in)
            cur.wait_stream(s_out)
        return g


def capture(fn, layers):
    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        for l in range(layers):
            fn(l)                                    # warm the path on the side stream
    torch.cuda.current_stream().wait_stream(s)
    torch.cuda.synchronize()
    with torch.cuda.graph(g):
        for l in range(layers):
            fn(l)
    return g


def timed(run_chunk, chunks, barrier):
    """Barrier + sync, CUDA events around `chunks` calls of run_chunk on the current stream."""
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    torch.cuda.synchronize()
    e0.record()
    for _ in range(chunks):
        run_chunk()
    e1.record()
    torch.cuda.synchronize()
    barrier()
    return e0.elapsed_time(e1)            # ms


def run_ours(args, rank, world, local_rank, dist):
    from paper_2512_10310_b200 import binding as B

    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    cfg = W.STEP_7B
    handle = B.evlnCreate(local_rank)
    ring = LayerRing(B, handle, cfg, dev, RING_LAYERS)
    for l in range(RING_LAYERS):
        ring.step(l)
    assert B.evlnGetDeviceStatus(handle) == 0

    def barrier():
        if dist is not None:
            dist.barrier()

    def max_over_ranks(x):
        return _max_over_ranks(x, dist, dev)

    steps = max(RING_LAYERS, (args.steps // RING_LAYERS) * RING_LAYERS)
    warm = max(3 * RING_LAYERS, -(-args.warmup // RING_LAYERS) * RING_LAYERS)
    g_step = capture(ring.step, RING_LAYERS)
    g_attn = capture(ring.attention_only, RING_LAYERS)

    for _ in range(warm // RING_LAYERS):
        g_step.replay()
    torch.cuda.synchronize()

    sampler = ClockSampler(physical_gpu_index(local_rank))
    sampler.start()
    ms = timed(g_step.replay, steps // RING_LAYERS, barrier)
    ms_attn = timed(g_attn.replay, steps // RING_LAYERS, barrier)
    clocks = sampler.stop()
    assert B.evlnGetDeviceStatus(handle) == 0, "a kernel gave up on a bounded wait"

    # end to end through the public calls with host buffers (eager launches + copies)
    e2e_steps = min(steps, 64 * RING_LAYERS)
    for l in range(RING_LAYERS):
        ring.step_e2e(l)
    torch.cuda.synchronize()

    g_e2e = ring.capture_e2e()
    for _ in range(3):
        g_e2e.replay()
    torch.cuda.synchronize()
    ms_e2e = timed(g_e2e.replay, e2e_steps // RING_LAYERS, barrier)

    us_step = max_over_ranks(ms * 1e3 / steps)
    us_attn = max_over_ranks(ms_attn * 1e3 / steps)
    us_e2e = max_over_ranks(ms_e2e * 1e3 / e2e_steps)

    # The metric is quoted against the cache length: the same layer-step at other L (7B-class shape),
    # a short measurement each, on rank 0 of a single-GPU run only.
    h2d = sum(t.numel() * t.element_size() for t in ring.layers[0]["host_in"])
    d2h = ring.layers[0]["host_out"].numel() * ring.layers[0]["host_out"].element_size()
    by_len, action_steps = [], []
    if world == 1 and not args.no_sweep:
        del g_step, g_attn
        ring.layers.clear()
        torch.cuda.empty_cache()
        peaks_s, _ = load_peaks()
        for L in (1024, 8192, 16384, 32768):
            c = dataclasses.replace(cfg, name=f"step_7b_L{L}", cache_len=L)
            kv_bytes = 2 * (L + c.num_new) * c.num_kv_heads * c.head_dim * 2
            layers = max(2, min(RING_LAYERS, int(2.2 * L2_BYTES / kv_bytes) + 1))
            r = LayerRing(B, handle, c, dev, layers, random_device_inputs=True)
            gs, ga = capture(r.step, layers), capture(r.attention_only, layers)
            reps = max(3, 640 // layers)
            for _ in range(3):
                gs.replay()
            t_s = timed(gs.replay, reps, barrier) * 1e3 / (reps * layers)
            t_a = timed(ga.replay, reps, barrier) * 1e3 / (reps * layers)
            roof = max(c.flops() / (peaks_s["bf16_tflops"] * 1e12), c.algorithmic_bytes() / (peaks_s["hbm_gbs"] * 1e9)) * 1e6
            by_len.append({"cache_len": L, "us_per_step": round(t_s, 2), "attention_us": round(t_a, 2),
                           "attention_tflops": round(c.flops() / t_a / 1e6, 1), "kv_splits": r.splits,
                           "step_roofline_frac": round(roof / t_s, 4)})
            del gs, ga, r
            torch.cuda.empty_cache()
        # The 8 action tokens that follow a frame in the streaming episode (same layer shape): a step
        # bound by streaming K and V once, quoted against the measured HBM bandwidth.
        for L in (4096, 20656):
            c = dataclasses.replace(cfg, name=f"action_7b_L{L}", cache_len=L, num_new=8)
            kv_bytes = 2 * (L + c.num_new) * c.num_kv_heads * c.head_dim * 2
            layers = max(2, min(RING_LAYERS, int(2.2 * L2_BYTES / kv_bytes) + 1))
            r = LayerRing(B, handle, c, dev, layers, random_device_inputs=True)
            gs = capture(r.step, layers)
            reps = max(3, 640 // layers)
            for _ in range(3):
                gs.replay()
            t_s = timed(gs.replay, reps, barrier) * 1e3 / (reps * layers)
            action_steps.append({"cache_len": L, "new_tokens": 8, "us_per_step": round(t_s, 2), "kv_splits": r.splits,
                                 "kv_gbs": round(kv_bytes / t_s / 1e3, 1),
                                 "hbm_frac": round(kv_bytes / t_s / 1e3 / peaks_s["hbm_gbs"], 4)})
            del gs, r
            torch.cuda.empty_cache()
        assert B.evlnGetDeviceStatus(handle) == 0, "a kernel gave up on a bounded wait"
    B.evlnDestroy(handle)
    if rank != 0:
        return None

    peaks, peaks_kind = load_peaks()
    flops = cfg.flops()
    abytes = cfg.algorithmic_bytes()
    t_flop_us = flops / (peaks["bf16_tflops"] * 1e12) * 1e6
    t_hbm_us = abytes / (peaks["hbm_gbs"] * 1e9) * 1e6
    achieved_tf = flops / (us_attn * 1e-6) / 1e12
    line = {
        "metric": "new-frame step-attention latency", "value": round(us_step, 3), "unit": "us/step",
        "n_gpus": world, "steps": steps, "warmup": warm, "ms_per_step": us_step / 1e3,
        "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {
            "workload": f"{cfg.name}: 28q/4kv heads, head_dim 128, L=4096, n=196, theta 1e6, bf16, one layer-step "
                        "= evlnRopeAppend + evlnStepAttention + evlnStepCombine",
            "kv_splits": ring.splits,
            "launch": f"CUDA graph of {RING_LAYERS} layer-steps, replayed",
            "l2": f"inputs larger than L2: ring of {RING_LAYERS} independent layer caches, "
                  f"{RING_LAYERS * ring.bytes_per_layer / 2**20:.0f} MiB of K/V revisited round-robin",
            "parallelism": "replicas only" if world > 1 else "single GPU",
        },
        "tflops": round(flops / (us_step * 1e-6) / 1e12 * world, 2),
        "gbs": round(abytes / (us_step * 1e-6) / 1e9 * world, 1),
        "steps_per_s": round(aggregate_steps_per_s(us_step, world), 1),
        "step_roofline_frac": round(max(t_flop_us, t_hbm_us) / us_step, 4),
        "roofline": {
            "kernel": "attn_pair_kernel (evlnStepAttention)", "bound": "tensor",
            "achieved": round(achieved_tf, 2), "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
            "frac": round(achieved_tf / peaks["bf16_tflops"], 4), "peak_kind": f"{peaks_kind} burst bf16",
            "traffic": attention_dram_traffic(), "us_per_launch": round(us_attn, 3),
            "timing": f"CUDA events around graph replays of {RING_LAYERS} back-to-back attention launches",
            "flops_per_launch": flops,
        },
        "e2e": {"value": round(us_e2e, 3), "unit": "us/step", "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": e2e_steps,
                "launch": f"CUDA graph of {RING_LAYERS} steps: pinned host-to-device copies, the three calls, "
                          "device-to-host copy; copies on side streams overlap the neighbouring steps' kernels"},
        "gpu_launches": 3 * steps,
        "clocks": clocks,
    }
    if by_len:
        line["by_cache_len"] = by_len
    if action_steps:
        line["action_token_step"] = action_steps
    return line


# ------------------------------------------------------------------------------------------------
# CPU oracle arms
# ------------------------------------------------------------------------------------------------

def oracle_sample_time(cfg, tokens_per_step, steps, warmup):
    """Times the oracle's step routine, as it stands, on a block of `tokens_per_step` consecutive
    new tokens (all heads) of the workload: rotate + append + attention for those tokens."""
    from oracle import step_oracle as so
    x = W.make_step_inputs(cfg)
    f64 = lambda t: np.ascontiguousarray(t.to(torch.float64).numpy())
    L, n = cfg.cache_len, cfg.num_new
    kc = np.zeros((L + n, cfg.num_kv_heads, cfg.head_dim))
    vc = np.zeros_like(kc)
    kc[:L], vc[:L] = f64(x["k_cache"]), f64(x["v_cache"])
    q, k, v = f64(x["q_new"]), f64(x["k_new"]), f64(x["v_new"])
    so.step(q, k, v, kc, vc, L, cfg.rope_theta, storage="bf16")     # fills slots L..L+n-1
    rng = np.random.default_rng(0)
    total = 0.0
    m = tokens_per_step
    for s in range(warmup + steps):
        i0 = int(rng.integers(0, n - m + 1))
        t0 = time.perf_counter()
        so.step(q[i0:i0 + m], k[i0:i0 + m], v[i0:i0 + m], kc, vc, L + i0, cfg.rope_theta, storage="bf16")
        if s >= warmup:
            total += time.perf_counter() - t0
    return total / steps, so.num_threads()


def cpu_baseline_full_step(cfg):
    """One full step of the oracle (all query rows), threads as the oracle uses them."""
    from oracle import step_oracle as so
    x = W.make_step_inputs(cfg)
    f64 = lambda t: np.ascontiguousarray(t.to(torch.float64).numpy())
    L, n = cfg.cache_len, cfg.num_new
    kc = np.zeros((L + n, cfg.num_kv_heads, cfg.head_dim))
    vc = np.zeros_like(kc)
    kc[:L], vc[:L] = f64(x["k_cache"]), f64(x["v_cache"])
    q, k, v = f64(x["q_new"]), f64(x["k_new"]), f64(x["v_new"])
    reps = 5
    t0 = time.perf_counter()
    for _ in range(reps):
        so.step(q, k, v, kc, vc, L, cfg.rope_theta, storage="bf16")
    dt = (time.perf_counter() - t0) / reps
    return dt, so.num_threads()


def run_reference(args, rank, world):
    if rank != 0:
        return None
    cfg = W.STEP_7B
    # one sample unit = one new token x all 28 query heads through the oracle's step routine
    probe, threads = oracle_sample_time(cfg, 1, 3, 1)
    budget_s = 120.0
    total_steps = args.steps + args.warmup
    per = max(1, min(cfg.num_new, int(budget_s / max(total_steps, 1) / max(probe, 1e-9))))
    if probe * total_steps > 2 * budget_s:
        steps = max(1, int(budget_s / probe) - args.warmup)
    else:
        steps = args.steps
    t_step, threads = oracle_sample_time(cfg, per, steps, min(args.warmup, 3))
    us_full = t_step / per * cfg.num_new * 1e6
    line = {
        "impl": "reference", "metric": "new-frame step-attention latency", "value": round(us_full, 1),
        "unit": "us/step", "n_gpus": world, "steps": steps, "warmup": min(args.warmup, 3),
        "ms_per_step": us_full / 1e3, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{cfg.name}: 28q/4kv heads, head_dim 128, L=4096, n=196, theta 1e6 "
                               "(fp64 CPU oracle of the same step)"},
        "cpu_baseline": {"value": round(us_full, 1), "unit": "us/step", "cores": threads, "kind": "oracle",
                         "sample": f"{per} consecutive of {cfg.num_new} new tokens (all 28 heads) per step, rotate + "
                                   f"append + attention; time scaled by {cfg.num_new}/{per}"},
        "e2e": {"value": round(us_full, 1), "unit": "us/step", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    if steps != args.steps:
        line["config"]["note"] = f"steps reduced from {args.steps} to {steps} to bound the CPU run"
    return line


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=65536)
    ap.add_argument("--warmup", type=int, default=3200)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true", help="skip the short cache-length sweep")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        line = run_reference(args, rank, world)
        if line is not None:
            print(json.dumps(line), flush=True)
        return

    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        torch.cuda.set_device(local_rank)
        dist_mod.init_process_group("nccl", device_id=torch.device(f"cuda:{local_rank}"))
        dist = dist_mod
    line = run_ours(args, rank, world, local_rank, dist)
    if line is not None:
        if world == 1 and not args.no_cpu_baseline:
            dt, threads = cpu_baseline_full_step(W.STEP_7B)
            line["cpu_baseline"] = {
                "value": round(dt * 1e6, 1), "unit": "us/step", "cores": threads, "kind": "oracle",
                "sample": "mean of 5 full steps of the same workload (all 196 tokens x 28 heads), rotate + append + attention",
            }
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
