"""Oracle for the action-isolating mask of packed training sequences (Sec. 3.3 of the paper).

TEST INFRASTRUCTURE ONLY: plain NumPy on float64, dense masked attention, no code shared with the
CUDA path.

A packed sequence is  I, v_1, a_1, v_2, a_2, ..., v_N, a_N  (instruction tokens, then N frames of
visual tokens, each followed by its action chunk).  Under the action-isolating mask
  - a visual token attends to the instruction and to the visual tokens up to itself
    (never to an action token);
  - an action token of chunk t attends to the instruction, to the visual tokens of v_1..v_t and to
    the tokens of its own chunk up to itself (never to another chunk's tokens).
The paper does not say which position ids the packed tokens carry.  The reading taken here is the
one that makes a packed sequence "M parallel single-step examples sharing a prefix" and matches
inference, where past actions are not in the context: the instruction and the visual tokens are
numbered contiguously as if no action token were there, and the tokens of chunk t continue the
numbering right after v_t.
"""
from __future__ import annotations

import numpy as np


def packed_layout(instr_len: int, frame_tokens: int, action_tokens: int, num_frames: int):
    """Per token of the packed sequence: kind (0 instruction, 1 visual, 2 action), frame index
    (-1 for the instruction) and position id."""
    kind, frame, pos = [], [], []
    for i in range(instr_len):
        kind.append(0); frame.append(-1); pos.append(i)
    for t in range(num_frames):
        base = instr_len + t * frame_tokens
        for i in range(frame_tokens):
            kind.append(1); frame.append(t); pos.append(base + i)
        for i in range(action_tokens):
            kind.append(2); frame.append(t); pos.append(base + frame_tokens + i)
    return np.array(kind), np.array(frame), np.array(pos)


def action_isolating_mask(kind, frame):
    """mask[i, j] = True where query token i may attend to key token j."""
    T = len(kind)
    mask = np.zeros((T, T), dtype=bool)
    for i in range(T):
        for j in range(i + 1):                      # never the future
            if kind[j] == 2:                        # an action key: own chunk only
                mask[i, j] = kind[i] == 2 and frame[i] == frame[j]
            else:                                   # instruction or visual key
                mask[i, j] = True
    return mask


def rope_at(x, pos, theta: float):
    """Half-split RoPE of ``x [T,H,D]`` at the given position ids."""
    T, H, D = x.shape
    half = D // 2
    omega = theta ** (-2.0 * np.arange(half) / D)
    phi = np.asarray(pos, dtype=np.float64)[:, None] * omega[None, :]
    c, s = np.cos(phi)[:, None, :], np.sin(phi)[:, None, :]
    lo, hi = x[..., :half], x[..., half:]
    return np.concatenate([lo * c - hi * s, hi * c + lo * s], axis=-1)


def masked_attention(q, k, v, mask, pos, theta: float, round_k=None):
    """Dense attention of a packed sequence under ``mask``; ``q [T,Hq,D]``, ``k``/``v [T,Hkv,D]``.
    Returns ``out [T,Hq,D]`` and ``lse [T,Hq]`` (natural log).  ``round_k`` (optional) rounds the
    rotated keys to the cache's storage type."""
    T, Hq, D = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    qr = rope_at(q, pos, theta)
    kr = rope_at(k, pos, theta)
    if round_k is not None:
        kr = round_k(kr)
    out = np.zeros((T, Hq, D))
    lse = np.zeros((T, Hq))
    scale = 1.0 / np.sqrt(D)
    for h in range(Hq):
        g = h // G
        s = (qr[:, h, :] @ kr[:, g, :].T) * scale
        s = np.where(mask, s, -np.inf)
        m = s.max(axis=1, keepdims=True)
        p = np.exp(s - m)
        l = p.sum(axis=1, keepdims=True)
        out[:, h, :] = (p / l) @ v[:, g, :]
        lse[:, h] = (m + np.log(l))[:, 0]
    return out, lse
