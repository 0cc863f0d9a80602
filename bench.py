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
    """Samples SM clock and throttle reasons through NVML while timed regions run (`recording` set)."""

    def __init__(self, index: int, period_s: float = 0.004):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.recording = threading.Event()
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
            if not self.recording.is_set():
                time.sleep(self.period)
                continue
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

MIN_REPLAYS = 200           # every timed graph is replayed at least this often, whatever --steps says
K2_SOURCES = ("attn_pair.cuh", "ptx_sm100.cuh", "common.cuh")
K2_TRAFFIC_FILE = os.path.join(ROOT, "profiles", "attn_pair_kernel_step_7b_L4096.traffic.txt")


def attention_dram_traffic():
    """DRAM bytes (read + write) of one attention launch at the headline workload, as counted by the
    last ncu capture.  The figure belongs to the kernel sources as they were then (their SHA-256 is
    stored beside it): once one of them changes it is withheld until the counters are taken again."""
    import hashlib
    h = hashlib.sha256()
    src = os.path.join(ROOT, "paper_2512_10310_b200", "csrc")
    try:
        for name in K2_SOURCES:
            with open(os.path.join(src, name), "rb") as fh:
                h.update(fh.read())
        rec = dict(line.strip().split("=", 1) for line in open(K2_TRAFFIC_FILE) if "=" in line and not line.startswith("#"))
        return int(rec["dram_bytes_per_launch"]) if rec.get("sha256") == h.hexdigest() else None
    except (OSError, KeyError, ValueError):
        return None


class LayerRing:
    """Device buffers of independent layers of one workload (+ pinned host copies when asked for).
    One position table serves all layers, as in a model: it is made once per pass over the ring."""

    def __init__(self, B, handle, cfg, dev, layers, host_copies=False):
        self.B, self.h, self.cfg, self.dev = B, handle, cfg, dev
        L, n, Hq, Hkv, D = cfg.cache_len, cfg.num_new, cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim
        self.table = torch.empty(max(B.evlnRopeTableBytes(D, n), 16), dtype=torch.uint8, device=dev)
        self.p = B.step_params(cfg.dtype, Hq, Hkv, D, L, n, L + n, cfg.rope_theta, rope_table=self.table,
                               rope_table_first_pos=L, rope_table_count=n)
        qbytes = B.evlnStepQRotSize(handle, self.p)
        wbytes = B.evlnStepWorkspaceSize(handle, self.p)
        self.splits = B.evlnStepNumSplits(handle, self.p)
        self.layers = []
        dt = cfg.torch_dtype
        for l in range(layers):
            if not host_copies:
                # same distribution, drawn on the device
                gen = torch.Generator(device=dev).manual_seed(cfg.seed * 7919 + l)
                mk = lambda *sh: (torch.randn(*sh, generator=gen, device=dev, dtype=torch.float32) * cfg.input_scale).to(dt)
                self.layers.append(dict(
                    kc=mk(Hkv, L + n, D), vc=mk(Hkv, L + n, D), q=mk(n, Hq, D), k=mk(n, Hkv, D), v=mk(n, Hkv, D),
                    q_rot=torch.empty(qbytes, dtype=torch.uint8, device=dev),
                    ws=torch.empty(max(wbytes, 16), dtype=torch.uint8, device=dev),
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
            self.layers.append(dict(
                kc=kc, vc=vc, qkv=qkv, q=qkv[:, :Hq], k=qkv[:, Hq:Hq + Hkv], v=qkv[:, Hq + Hkv:],
                q_rot=torch.empty(qbytes, dtype=torch.uint8, device=dev),
                ws=torch.empty(max(wbytes, 16), dtype=torch.uint8, device=dev),
                out=torch.empty((n, Hq, D), dtype=dt, device=dev),
                host_in=[host_qkv],
                host_out=torch.empty((n, Hq, D), dtype=dt).pin_memory(),
            ))
        self.bytes_per_layer = 2 * kc.numel() * kc.element_size()
        self.make_table()
        torch.cuda.synchronize()

    def make_table(self):
        c = self.cfg
        self.B.evlnRopeTable(self.h, c.head_dim, c.rope_theta, c.cache_len, c.num_new, self.table)

    def step(self, l):
        B, y = self.B, self.layers[l]
        B.evlnRopeAppend(self.h, self.p, y["q"], y["k"], y["v"], y["q_rot"], y["kc"], y["vc"])
        B.evlnStepAttention(self.h, self.p, y["q_rot"], y["kc"], y["vc"], y["ws"])
        B.evlnStepCombine(self.h, self.p, y["ws"], y["out"], None)

    def append_only(self, l):
        y = self.layers[l]
        self.B.evlnRopeAppend(self.h, self.p, y["q"], y["k"], y["v"], y["q_rot"], y["kc"], y["vc"])

    def attention_only(self, l):
        y = self.layers[l]
        self.B.evlnStepAttention(self.h, self.p, y["q_rot"], y["kc"], y["vc"], y["ws"])

    def combine_only(self, l):
        y = self.layers[l]
        self.B.evlnStepCombine(self.h, self.p, y["ws"], y["out"], None)

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

    def capture_e2e(self, copy_streams=1):
        """One CUDA graph of a pass over the ring through the public calls with host buffers:
        copies in on side streams, kernels on the capture stream, copies out on further side
        streams.  With more than one stream per direction consecutive steps' copies are independent
        nodes of the graph, so a copy can be set up while the previous one still moves data."""
        s_ins = [torch.cuda.Stream() for _ in range(copy_streams)]
        s_outs = [torch.cuda.Stream() for _ in range(copy_streams)]
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            cur = torch.cuda.current_stream()
            for s in s_ins + s_outs:
                s.wait_stream(cur)
            self.make_table()
            for l in range(len(self.layers)):
                self.step_e2e(l, s_ins[l % copy_streams], s_outs[l % copy_streams])
            for s in s_ins + s_outs:
                cur.wait_stream(s)
        return g


class PagedBatch:
    """The batched-serving workload (16 episodes on a page pool) on the device, one or more
    independent layers (pools), as CUDA-graph-able calls."""

    def __init__(self, B, handle, cfg, x, dev, layers):
        self.B, self.h, self.cfg = B, handle, cfg
        Bn, P, Hq, Hkv, D = len(x["cache_lens"]), cfg.page_size, cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim
        self.lens, self.offs = x["cache_lens"], x["new_offsets"]
        max_pages = max(len(t) for t in x["page_table"])
        table = torch.zeros((Bn, max_pages), dtype=torch.int32)
        for b, t in enumerate(x["page_table"]):
            table[b, :len(t)] = torch.tensor(t, dtype=torch.int32)
        self.table = table.to(dev)
        # one position table for 0 .. the longest episode: made once, like a model's RoPE cache
        count = max(L + self.offs[b + 1] - self.offs[b] for b, L in enumerate(self.lens))
        self.rope_table = torch.empty(B.evlnRopeTableBytes(D, count), dtype=torch.uint8, device=dev)
        B.evlnRopeTable(handle, D, cfg.rope_theta, 0, count, self.rope_table)
        self.p = B.paged_params(Hq, Hkv, D, Bn, P, x["num_pages"], max_pages, cfg.rope_theta,
                                rope_table=self.rope_table, rope_table_first_pos=0, rope_table_count=count)
        total = self.offs[-1]
        wbytes = B.evlnPagedWorkspaceSize(handle, self.p, self.lens, self.offs)
        self.layers = []
        for l in range(layers):
            # layer 0 holds the seeded pools; further layers hold independent random pools of the same shape
            if l == 0:
                kp = x["k_pool"].to(dev).permute(0, 2, 1, 3).contiguous()
                vp = x["v_pool"].to(dev).permute(0, 2, 1, 3).contiguous()
            else:
                gen = torch.Generator(device=dev).manual_seed(cfg.seed * 7919 + l)
                mk = lambda *sh: (torch.randn(*sh, generator=gen, device=dev, dtype=torch.float32) * cfg.input_scale).to(torch.bfloat16)
                kp, vp = mk(x["num_pages"], Hkv, P, D), mk(x["num_pages"], Hkv, P, D)
            self.layers.append(dict(
                kp=kp, vp=vp, q=x["q_new"].to(dev), k=x["k_new"].to(dev), v=x["v_new"].to(dev),
                q_rot=torch.empty(total * Hq * D * 2 + 256, dtype=torch.uint8, device=dev),
                ws=torch.empty(wbytes, dtype=torch.uint8, device=dev),
                out=torch.empty((total, Hq, D), dtype=torch.bfloat16, device=dev)))
        self.kv_bytes = sum(2 * (L + (self.offs[b + 1] - self.offs[b])) * Hkv * D * 2 for b, L in enumerate(self.lens))
        G = Hq // Hkv
        self.flops = sum(4 * D * Hq * ((self.offs[b + 1] - self.offs[b]) * L
                                       + (self.offs[b + 1] - self.offs[b]) * (self.offs[b + 1] - self.offs[b] + 1) // 2)
                         for b, L in enumerate(self.lens))
        self.alg_bytes = self.kv_bytes + 2 * total * Hq * D * 2 + 4 * total * Hkv * D * 2

    def step(self, l):
        B, y = self.B, self.layers[l]
        B.evlnPagedRopeAppend(self.h, self.p, y["q"], y["k"], y["v"], self.lens, self.offs, self.table, y["q_rot"], y["kp"], y["vp"])
        B.evlnPagedStepAttention(self.h, self.p, y["q_rot"], y["kp"], y["vp"], self.lens, self.offs, self.table, y["ws"])
        B.evlnPagedStepCombine(self.h, self.p, y["ws"], self.lens, self.offs, y["out"], None)

    def attention_only(self, l):
        y = self.layers[l]
        self.B.evlnPagedStepAttention(self.h, self.p, y["q_rot"], y["kp"], y["vp"], self.lens, self.offs, self.table, y["ws"])


def capture(fn, layers, before=None):
    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        if before is not None:
            before()
        for l in range(layers):
            fn(l)                                    # warm the path on the side stream
    torch.cuda.current_stream().wait_stream(s)
    torch.cuda.synchronize()
    with torch.cuda.graph(g):
        if before is not None:
            before()
        for l in range(layers):
            fn(l)
    return g


CLOCKS = None               # the run's ClockSampler: records while a timed region is open


def timed_replays(graph, replays, per_replay, barrier, warm=3):
    """`warm` untimed replays, then barrier + sync, CUDA events around EACH of `replays` replays of the
    graph on the current stream.  Returns microseconds per unit (a replay holds `per_replay` units):
    mean over the whole timed region, median / p10 / p90 over the replays."""
    for _ in range(warm):
        graph.replay()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(replays + 1)]
    barrier()
    torch.cuda.synchronize()
    if CLOCKS is not None:
        CLOCKS.recording.set()
    ev[0].record()
    for r in range(replays):
        graph.replay()
        ev[r + 1].record()
    torch.cuda.synchronize()
    if CLOCKS is not None:
        CLOCKS.recording.clear()
    barrier()
    per = sorted(ev[r].elapsed_time(ev[r + 1]) * 1e3 / per_replay for r in range(replays))
    pick = lambda q: per[min(len(per) - 1, int(q * len(per)))]
    return {"mean": ev[0].elapsed_time(ev[replays]) * 1e3 / (replays * per_replay), "median": pick(0.5),
            "p10": pick(0.1), "p90": pick(0.9), "replays": replays}


def r3(x):
    return round(x, 3)


def ring_layers_for(kv_bytes):
    """Enough independent layers that the K/V revisited round-robin exceed the L2 more than twice."""
    return max(2, min(RING_LAYERS, int(2.2 * L2_BYTES / kv_bytes) + 1))


def graph_of(fn):
    """A CUDA graph of one call of fn() (warmed once on a side stream first)."""
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        fn()
    torch.cuda.current_stream().wait_stream(s)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        fn()
    return g


def measure_widening(B, handle, cfg, dev, barrier, peaks):
    """The workloads beyond the plain step (7B-class layer shape throughout):
    a packed sequence under the action-isolating mask, one call against the loop of 2N+1 steps;
    the un-rotated store re-indexed by a frame sampler (gather + rotate pass, then the step);
    reloads of frame segments from a pinned host store, alone and beside the attention of a step."""
    Hq, Hkv, D, theta = cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, cfg.rope_theta
    bf = torch.bfloat16
    gen = torch.Generator(device=dev).manual_seed(99)
    mk = lambda *sh: (torch.randn(*sh, generator=gen, device=dev, dtype=torch.float32) * cfg.input_scale).to(bf)
    res = {}

    # ---- packed sequence: instruction 256, 12 frames of 196 visual + 8 action tokens ----
    I, F, A, N = 256, 196, 8, 12
    T, n_vis = I + N * (F + A), I + N * F
    pp = B.packed_params(Hq, Hkv, D, I, F, A, N, n_vis, theta)
    reps = 8                      # independent copies cycled through, so that the caches do not sit in L2
    packs = [dict(q=mk(T, Hq, D), k=mk(T, Hkv, D), v=mk(T, Hkv, D), kc=torch.empty((Hkv, n_vis + A, D), dtype=bf, device=dev),
                  vc=torch.empty((Hkv, n_vis + A, D), dtype=bf, device=dev),
                  ws=torch.empty(B.evlnPackedWorkspaceSize(handle, pp), dtype=torch.uint8, device=dev),
                  out=torch.empty((T, Hq, D), dtype=bf, device=dev)) for _ in range(reps)]
    pp = B.packed_params(Hq, Hkv, D, I, F, A, N, n_vis + A, theta)

    def packed_all():
        for y in packs:
            B.evlnPackedForward(handle, pp, y["q"], y["k"], y["v"], y["kc"], y["vc"], y["ws"], y["out"])

    # the same rows through ordinary steps: the instruction, then frame step + action step per frame
    calls = [(0, I, 0)]
    for t in range(N):
        r0 = I + t * (F + A)
        calls += [(I + t * F, F, r0), (I + (t + 1) * F, A, r0 + F)]
    sp = [B.step_params("bf16", Hq, Hkv, D, L, n, n_vis + A, theta) for L, n, _ in calls]
    qr = torch.empty(max(B.evlnStepQRotSize(handle, p) for p in sp), dtype=torch.uint8, device=dev)
    wl = torch.empty(max(B.evlnStepWorkspaceSize(handle, p) for p in sp), dtype=torch.uint8, device=dev)

    def loop_all():
        for y in packs:
            for p, (L, n, r0) in zip(sp, calls):
                B.evlnStep(handle, p, y["q"][r0:r0 + n], y["k"][r0:r0 + n], y["v"][r0:r0 + n], qr, y["kc"], y["vc"], wl,
                           y["out"][r0:r0 + n])

    g1, g2 = graph_of(packed_all), graph_of(loop_all)
    t1 = timed_replays(g1, MIN_REPLAYS, reps, barrier)
    t2 = timed_replays(g2, MIN_REPLAYS, reps, barrier)
    kind_flops = 4 * D * Hq * (n_vis * (n_vis + 1) // 2 + sum(A * (I + (t + 1) * F) + A * (A + 1) // 2 for t in range(N)))
    res["packed_forward"] = {
        "workload": f"packed sequence: instruction {I}, {N} frames x ({F} visual + {A} action tokens), {T} tokens",
        "one_call_us": r3(t1["median"]), "one_call_p10": r3(t1["p10"]), "one_call_p90": r3(t1["p90"]), "launches_one_call": 6,
        "step_loop_us": r3(t2["median"]), "launches_step_loop": 3 * len(calls), "speedup": round(t2["median"] / t1["median"], 2),
        "tflops_one_call": round(kind_flops / t1["median"] / 1e6, 1)}
    del g1, g2, packs
    torch.cuda.empty_cache()

    # ---- un-rotated store + frame sampler: 16 kept frames of 196 tokens + instruction 256 -> 3392 kept tokens ----
    kept_frames, store_frames = 16, 64
    kept = I + kept_frames * F
    store_cap = I + store_frames * F
    layers = ring_layers_for(2 * kept * Hkv * D * 2)
    tbl = torch.empty(B.evlnRopeTableBytes(D, kept + F), dtype=torch.uint8, device=dev)
    B.evlnRopeTable(handle, D, theta, 0, kept + F, tbl)
    gp = B.gather_params("bf16", Hkv, D, store_cap, kept + F, theta, rope_table=tbl, rope_table_first_pos=0,
                         rope_table_count=kept + F)
    frames = B.evlnSampleFrames(B.EVLN_SAMPLE_UNIFORM, store_frames, kept_frames)
    seg_src = [0] + [I + f * F for f in frames]
    seg_len = [I] + [F] * kept_frames
    st_p = B.step_params("bf16", Hq, Hkv, D, kept, F, kept + F, theta, rope_table=tbl, rope_table_first_pos=0,
                         rope_table_count=kept + F)
    lay = [dict(ks=mk(Hkv, store_cap, D), vs=mk(Hkv, store_cap, D), kw=torch.empty((Hkv, kept + F, D), dtype=bf, device=dev),
                vw=torch.empty((Hkv, kept + F, D), dtype=bf, device=dev), q=mk(F, Hq, D), k=mk(F, Hkv, D), v=mk(F, Hkv, D),
                qr=torch.empty(B.evlnStepQRotSize(handle, st_p), dtype=torch.uint8, device=dev),
                ws=torch.empty(B.evlnStepWorkspaceSize(handle, st_p), dtype=torch.uint8, device=dev),
                out=torch.empty((F, Hq, D), dtype=bf, device=dev)) for _ in range(layers)]

    def gather_all():
        for y in lay:
            B.evlnGatherRope(handle, gp, seg_src, seg_len, y["ks"], y["vs"], y["kw"], y["vw"])

    def step_all():
        for y in lay:
            B.evlnStep(handle, st_p, y["q"], y["k"], y["v"], y["qr"], y["kw"], y["vw"], y["ws"], y["out"])

    def both_all():
        for y in lay:
            B.evlnGatherRope(handle, gp, seg_src, seg_len, y["ks"], y["vs"], y["kw"], y["vw"])
            B.evlnStep(handle, st_p, y["q"], y["k"], y["v"], y["qr"], y["kw"], y["vw"], y["ws"], y["out"])

    tg = timed_replays(graph_of(gather_all), MIN_REPLAYS, layers, barrier)
    ts = timed_replays(graph_of(step_all), MIN_REPLAYS, layers, barrier)
    tb = timed_replays(graph_of(both_all), MIN_REPLAYS, layers, barrier)
    moved = 2 * 2 * kept * Hkv * D * 2          # K and V of every kept token, read + written
    res["reindexed_store"] = {
        "workload": f"un-rotated store of {store_frames} frames, uniform sampler keeps {kept_frames}: {kept} kept tokens + {F} new",
        "gather_rope_us": r3(tg["median"]), "gather_bytes": moved,
        "gather_gbs": round(moved / tg["median"] / 1e3, 1), "gather_hbm_frac": round(moved / tg["median"] / 1e3 / peaks["hbm_gbs"], 4),
        "step_us": r3(ts["median"]), "gather_plus_step_us": r3(tb["median"]), "ring_layers": layers}
    del lay
    torch.cuda.empty_cache()

    # ---- host-resident store: reload of 1 and of 8 (= half of a budget of 16) frame segments for all 28
    #      layers on a side stream, alone and beside the attention steps of those layers ----
    L28 = 28
    host_frames = 17
    hk = [torch.empty((Hkv, host_frames * F, D), dtype=bf).pin_memory() for _ in range(2)]     # K and V host stores of one layer
    ring = LayerRing(B, handle, cfg, dev, L28)
    gpl = B.gather_params("bf16", Hkv, D, 16 * F, 16 * F, theta)
    stores = [(torch.empty((Hkv, 16 * F, D), dtype=bf, device=dev), torch.empty((Hkv, 16 * F, D), dtype=bf, device=dev))
              for _ in range(L28)]
    side = torch.cuda.Stream()

    def fetch(nseg):
        for ks, vs in stores:
            for sgi in range(nseg):
                B.evlnStoreFetch(handle, gpl, hk[0], hk[1], sgi * F, F, ks, vs, sgi * F, stream=side)

    def steps28():
        for l in range(L28):
            ring.step(l)

    def wall_us(fn, reps=20):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        cur = torch.cuda.current_stream()
        e0.record()
        for _ in range(reps):
            fn()
            cur.wait_stream(side)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / reps

    def with_side(nseg):
        def f():
            side.wait_stream(torch.cuda.current_stream())
            fetch(nseg)
            steps28()
        return f

    def fetch_only(nseg):
        def f():
            side.wait_stream(torch.cuda.current_stream())
            fetch(nseg)
        return f

    t_steps = wall_us(steps28)
    rec = {"workload": f"28 layers, frame segments of {F} tokens ({2 * F * Hkv * D * 2} bytes per layer and segment), pinned host store",
           "steps_28_layers_us": r3(t_steps), "launch": "eager calls; copies on a side stream, the 28 layer-steps on the main stream"}
    for nseg in (1, 8):
        t_f = wall_us(fetch_only(nseg))
        t_b = wall_us(with_side(nseg))
        nbytes = nseg * L28 * 2 * F * Hkv * D * 2
        rec[f"fetch_{nseg}_segments"] = {"bytes": nbytes, "alone_us": r3(t_f), "h2d_gbs": round(nbytes / t_f / 1e3, 1),
                                          "beside_steps_us": r3(t_b), "exposed_us": r3(max(0.0, t_b - t_steps))}
    res["host_store_fetch"] = rec
    del ring, stores
    torch.cuda.empty_cache()
    return res


def run_profile_workload(args, local_rank):
    """A few eager steps of ONE workload and nothing else: the small command that ncu captures are
    taken on (launch lists and counter sets of single kernels).  Prints a short JSON line, no timing."""
    from paper_2512_10310_b200 import binding as B
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    handle = B.evlnCreate(local_rank)
    name = args.profile_workload
    steps = max(1, args.steps)
    if name == "paged_b4":
        pc = dataclasses.replace(W.PAGED_B16, name="paged_b4", batch=4)
        x = W.make_paged_inputs(pc)
        pb = PagedBatch(B, handle, pc, x, dev, layers=1)
        for _ in range(steps):
            pb.step(0)
        info = {"episodes": 4, "cache_lens": x["cache_lens"]}
    else:
        c = {"step_7b": W.STEP_7B, "long_70b": W.LONG_70B,
             "action_7b": dataclasses.replace(W.STEP_7B, name="action_7b_L20656", cache_len=20656, num_new=8)}[name]
        kv_bytes = 2 * (c.cache_len + c.num_new) * c.num_kv_heads * c.head_dim * 2
        layers = 2 if kv_bytes > 64e6 else min(RING_LAYERS, ring_layers_for(kv_bytes))
        ring = LayerRing(B, handle, c, dev, layers)
        for i in range(steps):
            ring.step(i % layers)
        info = {"cache_len": c.cache_len, "new_tokens": c.num_new, "kv_splits": ring.splits, "ring_layers": layers}
    torch.cuda.synchronize()
    assert B.evlnGetDeviceStatus(handle) == 0
    B.evlnDestroy(handle)
    print(json.dumps({"profiled": name, "steps": steps, **info}), flush=True)


def run_ours(args, rank, world, local_rank, dist):
    from paper_2512_10310_b200 import binding as B

    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    cfg = W.STEP_7B
    peaks, peaks_kind = load_peaks()
    handle = B.evlnCreate(local_rank)

    def barrier():
        if dist is not None:
            dist.barrier()

    def max_over_ranks(x):
        return _max_over_ranks(x, dist, dev)

    def roof_us(flops, abytes):
        return max(flops / (peaks["bf16_tflops"] * 1e12), abytes / (peaks["hbm_gbs"] * 1e9)) * 1e6

    replays = max(MIN_REPLAYS, -(-args.steps // RING_LAYERS))
    steps = replays * RING_LAYERS
    warm_replays = max(3, -(-args.warmup // RING_LAYERS))

    global CLOCKS
    sampler = CLOCKS = ClockSampler(physical_gpu_index(local_rank))
    sampler.start()

    # ---- headline: the 7B-class layer-step (L = 4096, n = 196) ----
    ring = LayerRing(B, handle, cfg, dev, RING_LAYERS, host_copies=True)
    for l in range(RING_LAYERS):
        ring.step(l)
    assert B.evlnGetDeviceStatus(handle) == 0
    g_step = capture(ring.step, RING_LAYERS, before=ring.make_table)
    g_k1 = capture(ring.append_only, RING_LAYERS)
    g_attn = capture(ring.attention_only, RING_LAYERS)
    g_k3 = capture(ring.combine_only, RING_LAYERS)
    t_step = timed_replays(g_step, replays, RING_LAYERS, barrier, warm_replays)
    t_attn = timed_replays(g_attn, replays, RING_LAYERS, barrier, warm_replays)
    t_k1 = timed_replays(g_k1, replays, RING_LAYERS, barrier, warm_replays)
    t_k3 = timed_replays(g_k3, replays, RING_LAYERS, barrier, warm_replays)
    assert B.evlnGetDeviceStatus(handle) == 0, "a kernel gave up on a bounded wait"

    # end to end through the public calls with host buffers
    for l in range(RING_LAYERS):
        ring.step_e2e(l)
    torch.cuda.synchronize()
    g_e2e = ring.capture_e2e()
    e2e_replays = min(replays, 400)
    t_e2e = timed_replays(g_e2e, e2e_replays, RING_LAYERS, barrier, 3)

    us_step = max_over_ranks(t_step["mean"])
    us_attn = max_over_ranks(t_attn["mean"])
    us_e2e = max_over_ranks(t_e2e["mean"])
    h2d = sum(t.numel() * t.element_size() for t in ring.layers[0]["host_in"])
    d2h = ring.layers[0]["host_out"].numel() * ring.layers[0]["host_out"].element_size()
    ring_mib = RING_LAYERS * ring.bytes_per_layer / 2 ** 20
    headline_splits = ring.splits

    by_len, action_steps, by_config, widening = [], [], [], None
    if world == 1 and not args.no_sweep:
        del g_step, g_attn, g_k1, g_k3, g_e2e
        ring.layers.clear()
        torch.cuda.empty_cache()

        def measure(c, tag):
            """Step and attention-only time of one contiguous-cache workload (device-resident inputs)."""
            kv_bytes = 2 * (c.cache_len + c.num_new) * c.num_kv_heads * c.head_dim * 2
            layers = ring_layers_for(kv_bytes)
            r = LayerRing(B, handle, c, dev, layers)
            gs = capture(r.step, layers, before=r.make_table)
            ga = capture(r.attention_only, layers)
            reps = max(MIN_REPLAYS, 6400 // layers) if kv_bytes < 64e6 else MIN_REPLAYS
            ts = timed_replays(gs, reps, layers, barrier)
            ta = timed_replays(ga, reps, layers, barrier)
            roof = roof_us(c.flops(), c.algorithmic_bytes())
            rec = {"workload": tag, "cache_len": c.cache_len, "new_tokens": c.num_new, "kv_splits": r.splits,
                   "us_per_step": r3(ts["median"]), "us_p10": r3(ts["p10"]), "us_p90": r3(ts["p90"]),
                   "attention_us": r3(ta["median"]), "attention_us_p10": r3(ta["p10"]), "attention_us_p90": r3(ta["p90"]),
                   "attention_tflops": round(c.flops() / ta["median"] / 1e6, 1),
                   "attention_frac_of_peak": round(c.flops() / ta["median"] / 1e6 / peaks["bf16_tflops"], 4),
                   "roofline_us": r3(roof), "step_roofline_frac": round(roof / ts["median"], 4),
                   "replays": reps, "ring_layers": layers}
            del gs, ga, r
            torch.cuda.empty_cache()
            return rec, kv_bytes

        # latency against the cache length at the 7B-class shape
        for L in (1024, 2048, 8192, 16384, 32768):
            rec, _ = measure(dataclasses.replace(cfg, name=f"step_7b_L{L}", cache_len=L), f"7B shape, L={L}")
            by_len.append(rec)
        # the streaming episode: frame steps 1, 25, 50, 100 of 100 (n = 204; per layer of the 28)
        for s in (1, 25, 50, 100):
            rec, _ = measure(W.STREAM_7B.step_config(s), f"streaming episode step {s} of 100 (per layer)")
            by_config.append(rec)
        # the 70B-class long-history step
        rec, _ = measure(W.LONG_70B, "70B-class head shape, L=32768, n=256")
        by_config.append(rec)
        # the 8 action tokens that follow a frame (same layer shape): bound by streaming K and V once
        for L in (4096, 20656):
            c = dataclasses.replace(cfg, name=f"action_7b_L{L}", cache_len=L, num_new=8)
            rec, kv_bytes = measure(c, f"action tokens, L={L}")
            rec["kv_gbs"] = round(kv_bytes / rec["us_per_step"] / 1e3, 1)
            rec["hbm_frac"] = round(kv_bytes / rec["us_per_step"] / 1e3 / peaks["hbm_gbs"], 4)
            action_steps.append(rec)
        # batched serving on the page pool: 16 episodes, one launch triple per layer
        pc = W.PAGED_B16
        x = W.make_paged_inputs(pc)
        pb = PagedBatch(B, handle, pc, x, dev, layers=2)
        gs, ga = capture(pb.step, 2), capture(pb.attention_only, 2)
        ts = timed_replays(gs, MIN_REPLAYS, 2, barrier)
        ta = timed_replays(ga, MIN_REPLAYS, 2, barrier)
        roof = roof_us(pb.flops, pb.alg_bytes)
        rec = {"workload": "paged batch: 16 episodes, 64-token pages, L in [1024, 16384], n=196 each",
               "us_per_step": r3(ts["median"]), "us_p10": r3(ts["p10"]), "us_p90": r3(ts["p90"]),
               "attention_us": r3(ta["median"]), "attention_tflops": round(pb.flops / ta["median"] / 1e6, 1),
               "attention_frac_of_peak": round(pb.flops / ta["median"] / 1e6 / peaks["bf16_tflops"], 4),
               "flops": pb.flops, "roofline_us": r3(roof), "step_roofline_frac": round(roof / ts["median"], 4),
               "replays": MIN_REPLAYS, "ring_layers": 2}
        if not args.no_cpu_baseline:
            from oracle import step_oracle as so
            f64 = lambda t: np.ascontiguousarray(t.to(torch.float64).numpy())
            t0 = time.perf_counter()
            so.step_paged(f64(x["q_new"]), f64(x["k_new"]), f64(x["v_new"]), f64(x["k_pool"]), f64(x["v_pool"]),
                          x["page_table"], x["cache_lens"], x["new_offsets"], pc.rope_theta, storage="bf16")
            rec["oracle_s"] = round(time.perf_counter() - t0, 2)
        by_config.append(rec)
        del gs, ga, pb, x
        torch.cuda.empty_cache()
        if not args.no_cpu_baseline:
            dt, _ = cpu_baseline_full_step(W.LONG_70B, reps=1)
            by_config[-2]["oracle_s"] = round(dt, 2)
        widening = measure_widening(B, handle, cfg, dev, barrier, peaks)
        assert B.evlnGetDeviceStatus(handle) == 0, "a kernel gave up on a bounded wait"
    clocks = sampler.stop()
    B.evlnDestroy(handle)
    if rank != 0:
        return None

    flops = cfg.flops()
    abytes = cfg.algorithmic_bytes()
    t_flop_us = flops / (peaks["bf16_tflops"] * 1e12) * 1e6
    t_hbm_us = abytes / (peaks["hbm_gbs"] * 1e9) * 1e6
    achieved_tf = flops / (us_attn * 1e-6) / 1e12
    spread = lambda t: {"median": r3(t["median"]), "p10": r3(t["p10"]), "p90": r3(t["p90"]), "mean": r3(t["mean"]),
                        "replays": t["replays"]}
    line = {
        "metric": "new-frame step-attention latency", "value": round(us_step, 3), "unit": "us/step",
        "n_gpus": world, "steps": steps, "warmup": warm_replays * RING_LAYERS, "ms_per_step": us_step / 1e3,
        "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {
            "workload": f"{cfg.name}: 28q/4kv heads, head_dim 128, L=4096, n=196, theta 1e6, bf16, one layer-step "
                        "= evlnRopeAppend + evlnStepAttention + evlnStepCombine (position table made once per "
                        f"{RING_LAYERS} layer-steps by evlnRopeTable)",
            "kv_splits": headline_splits,
            "launch": f"CUDA graph of {RING_LAYERS} layer-steps, replayed {replays} times (at least {MIN_REPLAYS} "
                      "whatever --steps asks for), CUDA events around every replay",
            "l2": f"inputs larger than L2: ring of {RING_LAYERS} independent layer caches, "
                  f"{ring_mib:.0f} MiB of K/V revisited round-robin",
            "parallelism": "replicas only" if world > 1 else "single GPU",
        },
        "us_per_step": spread(t_step),
        "kernels_us": {"rope_append": spread(t_k1), "attention": spread(t_attn), "combine": spread(t_k3)},
        "tflops": round(flops / (us_step * 1e-6) / 1e12 * world, 2),
        "gbs": round(abytes / (us_step * 1e-6) / 1e9 * world, 1),
        "steps_per_s": round(aggregate_steps_per_s(us_step, world), 1),
        "roofline_us": r3(max(t_flop_us, t_hbm_us)),
        "step_roofline_frac": round(max(t_flop_us, t_hbm_us) / us_step, 4),
        "roofline": {
            "kernel": "attn_pair_kernel (evlnStepAttention)", "bound": "tensor",
            "achieved": round(achieved_tf, 2), "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
            "frac": round(achieved_tf / peaks["bf16_tflops"], 4), "peak_kind": f"{peaks_kind} burst bf16",
            "frac_of_sustained": round(achieved_tf / peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]), 4),
            "traffic": attention_dram_traffic(), "us_per_launch": round(us_attn, 3),
            "us_per_launch_median": r3(t_attn["median"]), "us_per_launch_p10": r3(t_attn["p10"]),
            "us_per_launch_p90": r3(t_attn["p90"]),
            "timing": f"CUDA events around each of {replays} graph replays of {RING_LAYERS} back-to-back attention launches",
            "flops_per_launch": flops,
        },
        "e2e": {"value": round(us_e2e, 3), "unit": "us/step", "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": e2e_replays * RING_LAYERS, "median": r3(t_e2e["median"]),
                "launch": f"CUDA graph of {RING_LAYERS} steps: pinned host-to-device copies, the three calls, "
                          "device-to-host copy; copies on side streams overlap the neighbouring steps' kernels"},
        "gpu_launches": (3 * RING_LAYERS + 1) * replays,
        "clocks": clocks,
    }
    if by_len:
        line["by_cache_len"] = by_len
    if by_config:
        line["by_config"] = by_config
    if action_steps:
        line["action_token_step"] = action_steps
    if widening:
        line["widening"] = widening
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


def cpu_baseline_full_step(cfg, reps=5):
    """Full steps of the oracle (all query rows), threads as the oracle uses them."""
    from oracle import step_oracle as so
    x = W.make_step_inputs(cfg)
    f64 = lambda t: np.ascontiguousarray(t.to(torch.float64).numpy())
    L, n = cfg.cache_len, cfg.num_new
    kc = np.zeros((L + n, cfg.num_kv_heads, cfg.head_dim))
    vc = np.zeros_like(kc)
    kc[:L], vc[:L] = f64(x["k_cache"]), f64(x["v_cache"])
    q, k, v = f64(x["q_new"]), f64(x["k_new"]), f64(x["v_new"])
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
    ap.add_argument("--steps", type=int, default=32768)
    ap.add_argument("--warmup", type=int, default=640)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true", help="skip the other workloads (cache-length sweep, by_config)")
    ap.add_argument("--profile-workload", default=None, choices=["step_7b", "long_70b", "paged_b4", "action_7b"],
                    help="run --steps eager steps of one workload and exit (the command ncu captures are taken on)")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.profile_workload:
        if rank == 0:
            run_profile_workload(args, local_rank)
        return
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
