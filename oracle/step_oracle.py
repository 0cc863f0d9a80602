"""ctypes front end of the fp64 CPU oracle (``evln_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, the smoke check and the benchmark's
``cpu_baseline`` leg.  It never imports the CUDA package and the CUDA package never
imports it.

All arrays are float64 NumPy arrays in token-major layout (see the C file's header).
``build()`` compiles the C file with gcc (``-O2 -fopenmp``, no fast-math) next to it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "evln_oracle.c")
_LIB = os.path.join(_HERE, "libevln_oracle.so")
_lib = None

_dp = ctypes.POINTER(ctypes.c_double)


def build(force: bool = False) -> str:
    """Compile the oracle shared library if it is missing or older than its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-shared", "-fPIC", _SRC, "-o", tmp, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.evln_oracle_round_bf16.restype = ctypes.c_double
        lib.evln_oracle_round_bf16.argtypes = [ctypes.c_double]
        lib.evln_oracle_round_array.argtypes = [_dp, ctypes.c_long, ctypes.c_int]
        lib.evln_oracle_rope.argtypes = [_dp, _dp, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                         ctypes.c_long, ctypes.c_double]
        lib.evln_oracle_step.restype = ctypes.c_int
        lib.evln_oracle_step.argtypes = [_dp, _dp, _dp, _dp, _dp, ctypes.c_long,
                                         ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                         ctypes.c_long, ctypes.c_double, ctypes.c_double,
                                         ctypes.c_int, _dp, _dp, _dp, _dp]
        lib.evln_oracle_attend_range.argtypes = [_dp, _dp, _dp, ctypes.c_int, ctypes.c_int,
                                                 ctypes.c_int, ctypes.c_int, ctypes.c_long,
                                                 ctypes.c_long, ctypes.c_long, ctypes.c_double,
                                                 _dp, _dp]
        lib.evln_oracle_combine.argtypes = [_dp, _dp, ctypes.c_int, ctypes.c_long, ctypes.c_int,
                                            _dp, _dp]
        lib.evln_oracle_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def _p(a):
    return a.ctypes.data_as(_dp) if a is not None else None


def _c(a):
    a = np.ascontiguousarray(a, dtype=np.float64)
    return a


STORAGE = {None: 0, "none": 0, "bf16": 1, "f32": 2}


def num_threads() -> int:
    return int(_load().evln_oracle_num_threads())


def round_bf16(x):
    """Round float64 values to the nearest bfloat16 (ties to even); returns float64."""
    a = np.array(x, dtype=np.float64, copy=True)
    flat = np.ascontiguousarray(a.reshape(-1))
    _load().evln_oracle_round_array(_p(flat), flat.size, 1)
    return flat.reshape(a.shape)


def rope(x, pos0: int, theta: float):
    """Rotate ``x [n,H,D]`` at positions ``pos0 .. pos0+n-1`` (half-split RoPE)."""
    x = _c(x)
    n, H, D = x.shape
    y = np.empty_like(x)
    _load().evln_oracle_rope(_p(x), _p(y), n, H, D, int(pos0), float(theta))
    return y


def step(q_new, k_new, v_new, k_cache, v_cache, L: int, theta: float, scale: float = 0.0,
         storage=None, want_probs: bool = False):
    """One navigation step on a contiguous cache.

    ``k_cache``/``v_cache`` are ``[cap,Hkv,D]`` float64 arrays modified in place (slots
    ``L..L+n-1`` are written).  Returns ``dict(out, lse, q_rot[, probs])``.
    """
    q_new, k_new, v_new = _c(q_new), _c(k_new), _c(v_new)
    assert k_cache.dtype == np.float64 and k_cache.flags.c_contiguous
    assert v_cache.dtype == np.float64 and v_cache.flags.c_contiguous
    n, Hq, D = q_new.shape
    Hkv = k_new.shape[1]
    cap = k_cache.shape[0]
    out = np.empty((n, Hq, D))
    lse = np.empty((n, Hq))
    q_rot = np.empty((n, Hq, D))
    probs = np.empty((n, Hq, L + n)) if want_probs else None
    rc = _load().evln_oracle_step(_p(q_new), _p(k_new), _p(v_new), _p(k_cache), _p(v_cache), cap,
                                  n, Hq, Hkv, D, int(L), float(theta), float(scale),
                                  STORAGE[storage], _p(out), _p(lse), _p(probs), _p(q_rot))
    if rc != 0:
        raise ValueError("oracle step: bad shapes or cache overflow")
    res = dict(out=out, lse=lse, q_rot=q_rot)
    if want_probs:
        res["probs"] = probs
    return res


def attend_range(q_rot, k_cache, v_cache, L: int, t0: int, t1: int, scale: float = 0.0):
    """Attention of rotated queries restricted to cache slots ``[t0, t1)`` (causal bound kept)."""
    q_rot, k_cache, v_cache = _c(q_rot), _c(k_cache), _c(v_cache)
    n, Hq, D = q_rot.shape
    Hkv = k_cache.shape[1]
    out = np.empty((n, Hq, D))
    lse = np.empty((n, Hq))
    _load().evln_oracle_attend_range(_p(q_rot), _p(k_cache), _p(v_cache), n, Hq, Hkv, D, int(L),
                                     int(t0), int(t1), float(scale), _p(out), _p(lse))
    return out, lse


def combine(o_parts, lse_parts):
    """Merge per-split partial results ``o_parts [S,rows,D]``, ``lse_parts [S,rows]``."""
    o_parts, lse_parts = _c(o_parts), _c(lse_parts)
    S, rows, D = o_parts.shape
    out = np.empty((rows, D))
    lse = np.empty((rows,))
    _load().evln_oracle_combine(_p(o_parts), _p(lse_parts), S, rows, D, _p(out), _p(lse))
    return out, lse


def step_paged(q_new, k_new, v_new, k_pool, v_pool, page_table, cache_lens, new_offsets,
               theta: float, scale: float = 0.0, storage=None):
    """A batch of episodes on a paged cache: the same step, episode by episode.

    ``k_pool``/``v_pool``: ``[num_pages, page_size, Hkv, D]`` float64, modified in place.
    ``page_table[b]`` lists the pages of episode ``b`` in order; ``cache_lens[b]`` is its
    length before the step; its new tokens are rows ``new_offsets[b]:new_offsets[b+1]`` of the
    packed ``q_new``/``k_new``/``v_new``.  Each episode's pages are gathered into a contiguous
    cache, stepped, and the touched pages are scattered back.
    """
    P = k_pool.shape[1]
    outs, lses = [], []
    for b, L in enumerate(cache_lens):
        lo, hi = int(new_offsets[b]), int(new_offsets[b + 1])
        n = hi - lo
        npg = (L + n + P - 1) // P
        pages = [int(p) for p in page_table[b][:npg]]
        kc = np.ascontiguousarray(k_pool[pages].reshape(npg * P, *k_pool.shape[2:]))
        vc = np.ascontiguousarray(v_pool[pages].reshape(npg * P, *v_pool.shape[2:]))
        r = step(q_new[lo:hi], k_new[lo:hi], v_new[lo:hi], kc, vc, int(L), theta, scale, storage)
        k_pool[pages] = kc.reshape(npg, P, *k_pool.shape[2:])
        v_pool[pages] = vc.reshape(npg, P, *v_pool.shape[2:])
        outs.append(r["out"])
        lses.append(r["lse"])
    return np.concatenate(outs, axis=0), np.concatenate(lses, axis=0)
