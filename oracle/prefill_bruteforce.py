"""Brute-force full-sequence causal prefill in NumPy float64 (tiny inputs only).

TEST INFRASTRUCTURE ONLY.  This is the computation the paper's method avoids: rotate every
token of the whole sequence at positions 0..T-1 and run dense causal softmax attention over
all of it (Sec. 3.2: without cache reuse the whole history is re-processed each step).  The
step oracle, fed the same sequence one chunk at a time with a reused cache, has to give the
same rows.  Written with whole-matrix NumPy operations so that it shares no loop structure
with ``evln_oracle.c``.
"""
from __future__ import annotations

import numpy as np


def rope_all(x, theta: float):
    """x [T,H,D] -> rotated at positions 0..T-1, pairs (j, j+D/2)."""
    T, H, D = x.shape
    half = D // 2
    inv_freq = theta ** (-(np.arange(half, dtype=np.float64) * 2.0) / D)       # [half]
    ang = np.arange(T, dtype=np.float64)[:, None] * inv_freq[None, :]          # [T,half]
    cos = np.cos(ang)[:, None, :]
    sin = np.sin(ang)[:, None, :]
    lo, hi = x[..., :half], x[..., half:]
    return np.concatenate([lo * cos - hi * sin, hi * cos + lo * sin], axis=-1)


def full_prefill(q, k, v, theta: float, scale: float | None = None):
    """q [T,Hq,D], k,v [T,Hkv,D] (unrotated) -> (out [T,Hq,D], lse [T,Hq], probs [Hq,T,T])."""
    T, Hq, D = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    qr = rope_all(q, theta)
    kr = rope_all(k, theta)
    kr_full = np.repeat(kr, G, axis=1)            # kv head g serves query heads g*G .. g*G+G-1
    v_full = np.repeat(v, G, axis=1)
    s = np.einsum("ihd,thd->hit", qr, kr_full) * scale
    mask = np.tril(np.ones((T, T), dtype=bool))
    s = np.where(mask[None], s, -np.inf)
    m = s.max(axis=-1, keepdims=True)
    e = np.exp(s - m)
    l = e.sum(axis=-1, keepdims=True)
    p = e / l
    out = np.einsum("hit,thd->ihd", p, v_full)
    lse = (m + np.log(l))[..., 0].T
    return out, lse, p
