"""Seeded synthetic inputs for the step-attention path.

This module only draws random tensors and describes shapes; it contains none of the
method's arithmetic (no rotation, no attention), so the CPU oracle's tests and the CUDA
path's tests can both take their inputs from it.

Every tensor is drawn on the CPU from ``torch.Generator().manual_seed(seed)`` as fp32
standard normals, multiplied by ``input_scale`` and cast to the storage dtype, in the fixed
order  k_cache, v_cache, q_new, k_new, v_new.  All tensors are token-major:
``[tokens, heads, head_dim]``.

The five workloads stand in for "one new frame of visual tokens arriving after L cached
instruction + frame tokens" (Sec. 3.2 of the paper); the navigation datasets the paper
evaluates on are not used.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List

import torch


@dataclass(frozen=True)
class StepConfig:
    name: str
    dtype: str            # "bf16" | "f32"  (storage dtype of q/k/v, cache and output)
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    cache_len: int        # L: tokens in the cache before the step
    num_new: int          # n: tokens of the new frame
    rope_theta: float
    input_scale: float
    seed: int

    @property
    def torch_dtype(self):
        return torch.bfloat16 if self.dtype == "bf16" else torch.float32

    @property
    def group(self) -> int:
        return self.num_q_heads // self.num_kv_heads

    def causal_pairs(self) -> int:
        """(query, key) pairs per query head that the causal step evaluates."""
        n, L = self.num_new, self.cache_len
        return n * L + n * (n + 1) // 2

    def flops(self) -> int:
        """QK^T and PV multiply-adds over the causal pairs: 4 * D * Hq * pairs."""
        return 4 * self.head_dim * self.num_q_heads * self.causal_pairs()

    def algorithmic_bytes(self) -> int:
        """Each K/V element read once, Q in, O out, new K/V in and appended."""
        eb = 2 if self.dtype == "bf16" else 4
        T = self.cache_len + self.num_new
        kv = 2 * T * self.num_kv_heads * self.head_dim * eb
        qo = 2 * self.num_new * self.num_q_heads * self.head_dim * eb
        new_kv = 2 * 2 * self.num_new * self.num_kv_heads * self.head_dim * eb
        return kv + qo + new_kv


INV_SQRT_128 = 128.0 ** -0.5

# Tiny fp32 step: 64 instruction tokens + 3 frames x 64 tokens cached, one new frame.
TINY_F32 = StepConfig("tiny_f32", "f32", 2, 1, 64, 256, 64, 1.0e4, 1.0, 0)
# 7B-class single layer (the headline shape).
STEP_7B = StepConfig("step_7b_L4096", "bf16", 28, 4, 128, 4096, 196, 1.0e6, INV_SQRT_128, 1)
# 70B-class head shape, long history.
LONG_70B = StepConfig("long_70b_L32768", "bf16", 64, 8, 128, 32768, 256, 1.0e6, INV_SQRT_128, 4)


@dataclass(frozen=True)
class StreamConfig:
    """Streaming episode: an instruction prefill, then one frame (+ action tokens) per step."""
    name: str = "stream_7b"
    dtype: str = "bf16"
    num_layers: int = 28
    num_q_heads: int = 28
    num_kv_heads: int = 4
    head_dim: int = 128
    instruction_len: int = 256
    num_steps: int = 100
    tokens_per_step: int = 204       # 196 frame tokens + 8 action tokens
    rope_theta: float = 1.0e6
    input_scale: float = INV_SQRT_128
    seed: int = 2

    def call(self, s: int):
        """(L, n) of call ``s``: call 0 is the instruction prefill, calls 1..num_steps the frames."""
        if s == 0:
            return 0, self.instruction_len
        return self.instruction_len + (s - 1) * self.tokens_per_step, self.tokens_per_step

    @property
    def final_len(self) -> int:
        return self.instruction_len + self.num_steps * self.tokens_per_step

    def step_config(self, s: int, layer: int = 0) -> StepConfig:
        L, n = self.call(s)
        return StepConfig(f"{self.name}_s{s}_l{layer}", self.dtype, self.num_q_heads,
                          self.num_kv_heads, self.head_dim, L, n, self.rope_theta,
                          self.input_scale, self.seed * 1_000_003 + layer * 1009 + s)


STREAM_7B = StreamConfig()


@dataclass(frozen=True)
class PagedConfig:
    """Batched serving of concurrent episodes on a paged cache."""
    name: str = "paged_b16"
    dtype: str = "bf16"
    num_q_heads: int = 28
    num_kv_heads: int = 4
    head_dim: int = 128
    batch: int = 16
    page_size: int = 64
    min_len: int = 1024
    max_len: int = 16384
    num_new: int = 196
    rope_theta: float = 1.0e6
    input_scale: float = INV_SQRT_128
    seed: int = 3
    spare_pages: int = 8

    @property
    def torch_dtype(self):
        return torch.bfloat16 if self.dtype == "bf16" else torch.float32


PAGED_B16 = PagedConfig()


def _draw(gen, shape, scale, dtype):
    return (torch.randn(shape, generator=gen, dtype=torch.float32) * scale).to(dtype)


def make_step_inputs(cfg: StepConfig, cache_len: int | None = None):
    """Returns dict(k_cache [L,Hkv,D], v_cache [L,Hkv,D], q_new [n,Hq,D], k_new, v_new).

    ``k_cache`` holds the keys of the L cached tokens as they sit in the cache (i.e. already
    rotated when they were appended); being random, they need no further treatment.
    """
    L = cfg.cache_len if cache_len is None else cache_len
    gen = torch.Generator().manual_seed(cfg.seed)
    dt, sc = cfg.torch_dtype, cfg.input_scale
    Hq, Hkv, D, n = cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, cfg.num_new
    return dict(
        k_cache=_draw(gen, (L, Hkv, D), sc, dt),
        v_cache=_draw(gen, (L, Hkv, D), sc, dt),
        q_new=_draw(gen, (n, Hq, D), sc, dt),
        k_new=_draw(gen, (n, Hkv, D), sc, dt),
        v_new=_draw(gen, (n, Hkv, D), sc, dt),
    )


def make_new_tokens(cfg: StepConfig):
    """Only the new frame's q/k/v (used by chained / streaming runs that build their own cache)."""
    gen = torch.Generator().manual_seed(cfg.seed)
    dt, sc = cfg.torch_dtype, cfg.input_scale
    Hq, Hkv, D, n = cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, cfg.num_new
    return dict(
        q_new=_draw(gen, (n, Hq, D), sc, dt),
        k_new=_draw(gen, (n, Hkv, D), sc, dt),
        v_new=_draw(gen, (n, Hkv, D), sc, dt),
    )


def make_paged_inputs(cfg: PagedConfig, lens: List[int] | None = None, num_new: List[int] | None = None):
    """Ragged batch on a page pool.

    Cache lengths are integers uniform on [min_len, max_len] (not page aligned).  Pages for
    ``L_b + n_b`` tokens of every episode are handed out from a seeded random permutation of
    the pool, dealt round-robin over the episodes so that each episode's pages are scattered
    and interleaved with the others'.  Returns token-major pools
    ``[num_pages, page_size, Hkv, D]`` whose first ``L_b`` slots per episode are random.
    """
    gen = torch.Generator().manual_seed(cfg.seed)
    B, P = cfg.batch, cfg.page_size
    if lens is None:
        lens = torch.randint(cfg.min_len, cfg.max_len + 1, (B,), generator=gen).tolist()
    if num_new is None:
        num_new = [cfg.num_new] * B
    B = len(lens)
    need = [(L + n + P - 1) // P for L, n in zip(lens, num_new)]
    num_pages = sum(need) + cfg.spare_pages
    perm = torch.randperm(num_pages, generator=gen).tolist()
    tables: List[List[int]] = [[] for _ in range(B)]
    cursor = 0
    for r in range(max(need) if need else 0):
        for b in range(B):
            if r < need[b]:
                tables[b].append(perm[cursor])
                cursor += 1
    dt, sc = cfg.torch_dtype, cfg.input_scale
    Hq, Hkv, D = cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim
    k_pool = torch.zeros((num_pages, P, Hkv, D), dtype=dt)
    v_pool = torch.zeros((num_pages, P, Hkv, D), dtype=dt)
    for b in range(B):
        L = lens[b]
        kc = _draw(gen, (L, Hkv, D), sc, dt)
        vc = _draw(gen, (L, Hkv, D), sc, dt)
        for p in range((L + P - 1) // P):
            lo, hi = p * P, min(L, (p + 1) * P)
            k_pool[tables[b][p], : hi - lo] = kc[lo:hi]
            v_pool[tables[b][p], : hi - lo] = vc[lo:hi]
    total_new = sum(num_new)
    offsets = [0]
    for n in num_new:
        offsets.append(offsets[-1] + n)
    return dict(
        cache_lens=lens, new_offsets=offsets, page_table=tables, num_pages=num_pages,
        k_pool=k_pool, v_pool=v_pool,
        q_new=_draw(gen, (total_new, Hq, D), sc, dt),
        k_new=_draw(gen, (total_new, Hkv, D), sc, dt),
        v_new=_draw(gen, (total_new, Hkv, D), sc, dt),
    )
