"""Oracle for the un-rotated store and the frame samplers (Sec. 3.2 of the paper).

TEST INFRASTRUCTURE ONLY (see ``step_oracle``): plain NumPy / Python on float64, no code shared
with the CUDA path.

The paper stores the KV cache *before* the rotation.  Each step a frame sampler chooses the
history frames to keep; the kept tokens (instruction first, then the kept frames in temporal
order, then the new frame) receive contiguous position ids and RoPE is applied with those ids.
Two samplers are named: "uniform" (a fixed number of frames spread over the whole history) and
"sliding window" (the most recent frames, a stride apart).  The paper gives no formula for
either; the readings taken here are the ones documented in the library header.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import numpy as np

from . import step_oracle as so


def sample_uniform(num_frames: int, budget: int) -> List[int]:
    """All frames if they fit the budget, else ``budget`` frames spread evenly over the history
    with the first and the last one kept: frame round(k (N-1)/(B-1)), halves rounded up."""
    if num_frames <= 0 or budget <= 0:
        return []
    if num_frames <= budget:
        return list(range(num_frames))
    if budget == 1:
        return [num_frames - 1]
    out = []
    for k in range(budget):
        x = k * (num_frames - 1) / (budget - 1)
        out.append(int(np.floor(x + 0.5)))
    return out


def sample_sliding(num_frames: int, budget: int, stride: int) -> List[int]:
    """The most recent frames, ``stride`` apart, at most ``budget`` of them, ascending."""
    kept = []
    f = num_frames - 1
    while f >= 0 and len(kept) < budget:
        kept.append(f)
        f -= stride
    return kept[::-1]


def frame_segments(instr_len: int, frame_tokens: int, frames: Sequence[int]) -> List[Tuple[int, int]]:
    """(store slot, length) of the kept segments when the store holds the instruction followed by
    the frames, ``frame_tokens`` tokens each."""
    segs = [(0, instr_len)] if instr_len > 0 else []
    segs += [(instr_len + f * frame_tokens, frame_tokens) for f in frames]
    return segs


def gather_rope(k_store, v_store, segments, theta: float, storage=None):
    """Kept segments laid out back to back; the key landing in slot p is rotated at position p.

    ``k_store``/``v_store``: ``[slots, Hkv, D]`` float64 raw (un-rotated) keys / values.
    Returns ``(k_work, v_work)`` of ``sum(len)`` tokens; keys rounded once to ``storage``.
    """
    ks, vs = [], []
    pos = 0
    for src, length in segments:
        if length == 0:
            continue
        ks.append(so.rope(np.ascontiguousarray(k_store[src:src + length]), pos, theta))
        vs.append(np.array(v_store[src:src + length], dtype=np.float64))
        pos += length
    if not ks:
        shape = (0,) + tuple(k_store.shape[1:])
        return np.zeros(shape), np.zeros(shape)
    k_work = np.concatenate(ks, axis=0)
    if storage == "bf16":
        k_work = so.round_bf16(k_work)
    elif storage == "f32":
        k_work = k_work.astype(np.float32).astype(np.float64)
    return k_work, np.concatenate(vs, axis=0)


def sampled_step(q_new, k_new, v_new, k_store, v_store, segments, theta: float, scale: float = 0.0,
                 storage=None):
    """One step of the paper's scheme: kept history (raw) + new frame, contiguous ids, rotate, attend.

    Returns the step oracle's dict plus the working caches ``k_work``/``v_work`` ``[L'+n, Hkv, D]``.
    """
    k_hist, v_hist = gather_rope(k_store, v_store, segments, theta, storage)
    L, n = k_hist.shape[0], q_new.shape[0]
    Hkv, D = k_store.shape[1], k_store.shape[2]
    kc = np.zeros((L + n, Hkv, D))
    vc = np.zeros((L + n, Hkv, D))
    kc[:L], vc[:L] = k_hist, v_hist
    r = so.step(q_new, k_new, v_new, kc, vc, L, theta, scale, storage=storage)
    r["k_work"], r["v_work"] = kc, vc
    return r
