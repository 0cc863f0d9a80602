"""ctypes binding of ``libevln.so``: same names as the C entry points, argument marshalling only.

Every step of the path runs in the library's CUDA kernels.  PyTorch is used for device memory
and streams.  There is no fallback: loading fails loudly when the library has not been built
(``python -c "import __graft_entry__ as g; g.build()"`` or ``build_library()`` below).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from ctypes import (POINTER, Structure, byref, c_char_p, c_double, c_float, c_int, c_long, c_size_t,
                    c_void_p)

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
LIB_PATH = os.path.join(_PKG, "lib", "libevln.so")
_SOURCES = ["evln_api.cu", "attn_pair.cuh", "attn_simt.cuh", "combine.cuh", "rope_append.cuh",
            "common.cuh", "ptx_sm100.cuh", "gather_rope.cuh", "timeline_debug.cuh"]

EVLN_OK, EVLN_INVALID_VALUE, EVLN_NOT_SUPPORTED, EVLN_CACHE_FULL = 0, 1, 2, 3
EVLN_WORKSPACE_TOO_SMALL, EVLN_CUDA_ERROR, EVLN_DEVICE_TIMEOUT = 4, 5, 6
EVLN_BF16, EVLN_F32 = 0, 1
EVLN_KERNEL_AUTO, EVLN_KERNEL_SIMT = 0, 1

EXPORTS = [
    "evlnCreate", "evlnDestroy", "evlnGetErrorString", "evlnGetLastCudaError", "evlnGetDeviceStatus",
    "evlnSelfTestBoundedWait",
    "evlnStepNumSplits", "evlnStepWorkspaceSize", "evlnStepQRotSize",
    "evlnRopeTableBytes", "evlnRopeTable",
    "evlnRopeAppend", "evlnStepAttention", "evlnStepCombine", "evlnStep",
    "evlnPagedWorkspaceSize", "evlnPagedRopeAppend", "evlnPagedStepAttention", "evlnPagedStepCombine",
    "evlnPagedCheckTable",
    "evlnPackedWorkspaceSize", "evlnPackedForward",
    "evlnStepAttentionNoAlloc",
    "evlnSampleFrames", "evlnStoreAppend", "evlnGatherRope", "evlnStoreOffload", "evlnStoreFetch",
]
EVLN_NOALLOC_SCRATCH_BYTES = 32 << 20
EVLN_SELFTEST_STATUS_CODE = 8


class evlnStepParams(Structure):
    _fields_ = [("struct_size", c_size_t), ("dtype", c_int), ("num_q_heads", c_int),
                ("num_kv_heads", c_int), ("head_dim", c_int), ("cache_len", c_int),
                ("num_new", c_int), ("cache_capacity", c_int), ("num_splits", c_int),
                ("kernel", c_int), ("softmax_scale", c_float), ("rope_theta", c_double),
                ("rope_table", c_void_p), ("rope_table_first_pos", c_int), ("rope_table_count", c_int)]


class evlnPagedParams(Structure):
    _fields_ = [("struct_size", c_size_t), ("dtype", c_int), ("num_q_heads", c_int),
                ("num_kv_heads", c_int), ("head_dim", c_int), ("batch", c_int),
                ("page_size", c_int), ("num_pages", c_int), ("max_pages_per_seq", c_int),
                ("kv_chunk_tiles", c_int), ("softmax_scale", c_float), ("rope_theta", c_double),
                ("rope_table", c_void_p), ("rope_table_first_pos", c_int), ("rope_table_count", c_int)]


class evlnPackedParams(Structure):
    _fields_ = [("struct_size", c_size_t), ("dtype", c_int), ("num_q_heads", c_int), ("num_kv_heads", c_int),
                ("head_dim", c_int), ("instr_len", c_int), ("frame_tokens", c_int), ("action_tokens", c_int),
                ("num_frames", c_int), ("cache_capacity", c_int), ("kv_chunk_tiles", c_int),
                ("softmax_scale", c_float), ("rope_theta", c_double)]


class evlnGatherParams(Structure):
    _fields_ = [("struct_size", c_size_t), ("dtype", c_int), ("num_kv_heads", c_int), ("head_dim", c_int),
                ("store_capacity", c_int), ("work_capacity", c_int), ("rope_theta", c_double),
                ("rope_table", c_void_p), ("rope_table_first_pos", c_int), ("rope_table_count", c_int)]


EVLN_SAMPLE_UNIFORM, EVLN_SAMPLE_SLIDING = 0, 1


class EvlnError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {error_string(status)} ({status})")


def build_library(force: bool = False, verbose: bool = False) -> str:
    """Compile the CUDA sources into ``lib/libevln.so`` for sm_100a (in-tree)."""
    src_dir = os.path.join(_PKG, "csrc")
    srcs = [os.path.join(src_dir, s) for s in _SOURCES] + [os.path.join(_ROOT, "include", "evln.h")]
    if not force and os.path.exists(LIB_PATH) and all(
            os.path.getmtime(LIB_PATH) >= os.path.getmtime(s) for s in srcs):
        return LIB_PATH
    os.makedirs(os.path.dirname(LIB_PATH), exist_ok=True)
    tmp = LIB_PATH + f".tmp{os.getpid()}"
    cmd = ["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-o", tmp, os.path.join(src_dir, "evln_api.cu")]
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    subprocess.check_call(cmd)
    os.replace(tmp, LIB_PATH)
    return LIB_PATH


_lib = None


def lib():
    """The loaded library; raises if it has not been built (no fallback of any kind)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with __graft_entry__.build() "
                              "(nvcc, sm_100a); there is no CPU fallback")
        L = ctypes.CDLL(LIB_PATH)
        L.evlnGetErrorString.restype = c_char_p
        L.evlnGetErrorString.argtypes = [c_int]
        L.evlnCreate.argtypes = [POINTER(c_void_p), c_int]
        L.evlnDestroy.argtypes = [c_void_p]
        L.evlnGetLastCudaError.argtypes = [c_void_p]
        L.evlnGetDeviceStatus.argtypes = [c_void_p, c_void_p, POINTER(c_int)]
        L.evlnSelfTestBoundedWait.argtypes = [c_void_p, ctypes.c_longlong, c_void_p]
        L.evlnRopeTableBytes.argtypes = [c_int, c_int]
        L.evlnRopeTableBytes.restype = c_size_t
        L.evlnRopeTable.argtypes = [c_void_p, c_int, c_double, c_int, c_int, c_void_p, c_void_p]
        pp = POINTER(evlnStepParams)
        L.evlnStepNumSplits.argtypes = [c_void_p, pp, POINTER(c_int)]
        L.evlnStepWorkspaceSize.argtypes = [c_void_p, pp, POINTER(c_size_t)]
        L.evlnStepQRotSize.argtypes = [c_void_p, pp, POINTER(c_size_t)]
        L.evlnRopeAppend.argtypes = [c_void_p, pp, c_void_p, c_void_p, c_void_p, c_long, c_long, c_long,
                                     c_void_p, c_void_p, c_void_p, c_void_p]
        L.evlnStep.argtypes = [c_void_p, pp, c_void_p, c_void_p, c_void_p, c_long, c_long, c_long, c_void_p,
                               c_void_p, c_void_p, c_void_p, c_size_t, c_void_p, c_void_p, c_void_p]
        L.evlnStepAttention.argtypes = [c_void_p, pp, c_void_p, c_void_p, c_void_p, c_void_p, c_size_t,
                                        c_void_p]
        L.evlnStepCombine.argtypes = [c_void_p, pp, c_void_p, c_void_p, c_void_p, c_void_p]
        gp = POINTER(evlnPagedParams)
        ip = POINTER(c_int)
        L.evlnPagedWorkspaceSize.argtypes = [c_void_p, gp, ip, ip, POINTER(c_size_t)]
        L.evlnPagedRopeAppend.argtypes = [c_void_p, gp, c_void_p, c_void_p, c_void_p, ip, ip, c_void_p,
                                          c_void_p, c_void_p, c_void_p, c_void_p]
        L.evlnPagedStepAttention.argtypes = [c_void_p, gp, c_void_p, c_void_p, c_void_p, ip, ip, c_void_p,
                                             c_void_p, c_size_t, c_void_p]
        L.evlnPagedStepCombine.argtypes = [c_void_p, gp, c_void_p, ip, ip, c_void_p, c_void_p, c_void_p]
        L.evlnPagedCheckTable.argtypes = [gp, ip, ip, ip, ip, ip]
        kp = POINTER(evlnPackedParams)
        L.evlnPackedWorkspaceSize.argtypes = [c_void_p, kp, POINTER(c_size_t)]
        L.evlnPackedForward.argtypes = [c_void_p, kp, c_void_p, c_void_p, c_void_p, c_long, c_long, c_long, c_void_p,
                                        c_void_p, c_void_p, c_size_t, c_void_p, c_void_p, c_void_p]
        L.evlnStepAttentionNoAlloc.argtypes = [pp, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
        qp = POINTER(evlnGatherParams)
        L.evlnSampleFrames.argtypes = [c_int, c_int, c_int, c_int, POINTER(c_int)]
        L.evlnStoreAppend.argtypes = [c_void_p, qp, c_void_p, c_void_p, c_long, c_long, c_int, c_int, c_void_p,
                                      c_void_p, c_void_p]
        L.evlnGatherRope.argtypes = [c_void_p, qp, c_int, POINTER(c_int), POINTER(c_int), c_void_p, c_void_p,
                                     c_void_p, c_void_p, POINTER(c_int), c_void_p]
        L.evlnStoreOffload.argtypes = [c_void_p, qp, c_void_p, c_void_p, c_int, c_int, c_void_p, c_void_p, c_int, c_int,
                                       c_void_p]
        L.evlnStoreFetch.argtypes = [c_void_p, qp, c_void_p, c_void_p, c_int, c_int, c_int, c_void_p, c_void_p, c_int,
                                     c_void_p]
        for name in EXPORTS:
            if name not in ("evlnGetErrorString", "evlnRopeTableBytes"):
                getattr(L, name).restype = c_int
        _lib = L
    return _lib


def error_string(status: int) -> str:
    return lib().evlnGetErrorString(int(status)).decode()


def _check(status: int, where: str):
    if status != EVLN_OK:
        raise EvlnError(status, where)


def _ptr(t):
    """Device (or host) address of a tensor, None -> NULL; raw ints pass through."""
    if t is None:
        return None
    if isinstance(t, int):
        return c_void_p(t)
    return c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        import torch
        return c_void_p(torch.cuda.current_stream().cuda_stream)
    if isinstance(stream, int):
        return c_void_p(stream)
    return c_void_p(stream.cuda_stream)


def _ints(seq):
    arr = (c_int * len(seq))(*[int(v) for v in seq])
    return arr


def step_params(dtype, num_q_heads, num_kv_heads, head_dim, cache_len, num_new, cache_capacity,
                rope_theta, softmax_scale=0.0, num_splits=0, kernel=EVLN_KERNEL_AUTO,
                rope_table=None, rope_table_first_pos=0, rope_table_count=0) -> evlnStepParams:
    """``rope_table``: a tensor written by evlnRopeTable (or None) covering the step's positions."""
    code = {"bf16": EVLN_BF16, "f32": EVLN_F32}.get(dtype, dtype)
    return evlnStepParams(ctypes.sizeof(evlnStepParams), code, num_q_heads, num_kv_heads, head_dim,
                          cache_len, num_new, cache_capacity, num_splits, kernel, softmax_scale, rope_theta,
                          _ptr(rope_table), rope_table_first_pos, rope_table_count)


def paged_params(num_q_heads, num_kv_heads, head_dim, batch, page_size, num_pages, max_pages_per_seq,
                 rope_theta, softmax_scale=0.0, kv_chunk_tiles=0, dtype=EVLN_BF16, rope_table=None,
                 rope_table_first_pos=0, rope_table_count=0) -> evlnPagedParams:
    return evlnPagedParams(ctypes.sizeof(evlnPagedParams), dtype, num_q_heads, num_kv_heads, head_dim,
                           batch, page_size, num_pages, max_pages_per_seq, kv_chunk_tiles, softmax_scale,
                           rope_theta, _ptr(rope_table),
                           int(rope_table_first_pos), int(rope_table_count))


# ---- the entry points, by their C names ----------------------------------------------------

def evlnCreate(device: int = 0):
    h = c_void_p()
    _check(lib().evlnCreate(byref(h), int(device)), "evlnCreate")
    return h


def evlnDestroy(handle):
    _check(lib().evlnDestroy(handle), "evlnDestroy")


def evlnGetLastCudaError(handle) -> int:
    return int(lib().evlnGetLastCudaError(handle))


def evlnGetDeviceStatus(handle, stream=None) -> int:
    """Synchronises the stream; returns the device status word (0 = no bounded wait expired).
    ``handle=None`` reads the status word of the allocation-free call on the current device."""
    v = c_int(0)
    st = lib().evlnGetDeviceStatus(handle, _stream(stream), byref(v))
    if st not in (EVLN_OK, EVLN_DEVICE_TIMEOUT):
        raise EvlnError(st, "evlnGetDeviceStatus")
    return int(v.value)


def evlnSelfTestBoundedWait(handle, limit_cycles: int = 100000, stream=None):
    """Launches the self-test kernel whose bounded wait must run out (see include/evln.h)."""
    _check(lib().evlnSelfTestBoundedWait(handle, int(limit_cycles), _stream(stream)), "evlnSelfTestBoundedWait")


def evlnRopeTableBytes(head_dim: int, count: int) -> int:
    return int(lib().evlnRopeTableBytes(int(head_dim), int(count)))


def evlnRopeTable(handle, head_dim, rope_theta, first_pos, count, table, stream=None):
    """(cos, sin) of the positions first_pos .. first_pos+count-1 into ``table`` (device memory)."""
    _check(lib().evlnRopeTable(handle, int(head_dim), float(rope_theta), int(first_pos), int(count), _ptr(table),
                               _stream(stream)), "evlnRopeTable")


def evlnPagedCheckTable(params, cache_lens, new_offsets, page_table_rows):
    """Host check of a page table given as ``[batch][max_pages_per_seq]`` ints (flattened or nested).
    Returns (status, bad_episode, bad_index)."""
    flat = [int(v) for row in page_table_rows for v in (row if hasattr(row, "__iter__") else [row])]
    be, bi = c_int(-1), c_int(-1)
    st = lib().evlnPagedCheckTable(byref(params), _ints(cache_lens), _ints(new_offsets), _ints(flat), byref(be), byref(bi))
    return int(st), int(be.value), int(bi.value)


def evlnStepNumSplits(handle, params) -> int:
    v = c_int(0)
    _check(lib().evlnStepNumSplits(handle, byref(params), byref(v)), "evlnStepNumSplits")
    return int(v.value)


def evlnStepWorkspaceSize(handle, params) -> int:
    v = c_size_t(0)
    _check(lib().evlnStepWorkspaceSize(handle, byref(params), byref(v)), "evlnStepWorkspaceSize")
    return int(v.value)


def evlnStepQRotSize(handle, params) -> int:
    v = c_size_t(0)
    _check(lib().evlnStepQRotSize(handle, byref(params), byref(v)), "evlnStepQRotSize")
    return int(v.value)


def evlnRopeAppend(handle, params, q_new, k_new, v_new, q_rot, k_cache, v_cache, stream=None,
                   strides=None):
    """q_new/k_new/v_new: [n,H,D] tensors (last two dims contiguous) or raw addresses + strides."""
    if strides is None:
        strides = (q_new.stride(0), k_new.stride(0), v_new.stride(0))
    _check(lib().evlnRopeAppend(handle, byref(params), _ptr(q_new), _ptr(k_new), _ptr(v_new),
                                int(strides[0]), int(strides[1]), int(strides[2]), _ptr(q_rot),
                                _ptr(k_cache), _ptr(v_cache), _stream(stream)), "evlnRopeAppend")


def evlnStepAttention(handle, params, q_rot, k_cache, v_cache, workspace, workspace_bytes=None,
                      stream=None):
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    _check(lib().evlnStepAttention(handle, byref(params), _ptr(q_rot), _ptr(k_cache), _ptr(v_cache),
                                   _ptr(workspace), int(workspace_bytes), _stream(stream)),
           "evlnStepAttention")


def evlnStepCombine(handle, params, workspace, out, lse_out=None, stream=None):
    _check(lib().evlnStepCombine(handle, byref(params), _ptr(workspace), _ptr(out), _ptr(lse_out),
                                 _stream(stream)), "evlnStepCombine")


def evlnStep(handle, params, q_new, k_new, v_new, q_rot, k_cache, v_cache, workspace, out, lse_out=None,
             workspace_bytes=None, stream=None, strides=None):
    """The three calls of a step in one."""
    if strides is None:
        strides = (q_new.stride(0), k_new.stride(0), v_new.stride(0))
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    _check(lib().evlnStep(handle, byref(params), _ptr(q_new), _ptr(k_new), _ptr(v_new), int(strides[0]),
                          int(strides[1]), int(strides[2]), _ptr(q_rot), _ptr(k_cache), _ptr(v_cache),
                          _ptr(workspace), int(workspace_bytes), _ptr(out), _ptr(lse_out), _stream(stream)),
           "evlnStep")


def evlnPagedWorkspaceSize(handle, params, cache_lens, new_offsets) -> int:
    v = c_size_t(0)
    _check(lib().evlnPagedWorkspaceSize(handle, byref(params), _ints(cache_lens), _ints(new_offsets),
                                        byref(v)), "evlnPagedWorkspaceSize")
    return int(v.value)


def evlnPagedRopeAppend(handle, params, q_new, k_new, v_new, cache_lens, new_offsets, page_table,
                        q_rot, k_pool, v_pool, stream=None):
    _check(lib().evlnPagedRopeAppend(handle, byref(params), _ptr(q_new), _ptr(k_new), _ptr(v_new),
                                     _ints(cache_lens), _ints(new_offsets), _ptr(page_table),
                                     _ptr(q_rot), _ptr(k_pool), _ptr(v_pool), _stream(stream)),
           "evlnPagedRopeAppend")


def evlnPagedStepAttention(handle, params, q_rot, k_pool, v_pool, cache_lens, new_offsets, page_table,
                           workspace, workspace_bytes=None, stream=None):
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    _check(lib().evlnPagedStepAttention(handle, byref(params), _ptr(q_rot), _ptr(k_pool), _ptr(v_pool),
                                        _ints(cache_lens), _ints(new_offsets), _ptr(page_table),
                                        _ptr(workspace), int(workspace_bytes), _stream(stream)),
           "evlnPagedStepAttention")


def evlnPagedStepCombine(handle, params, workspace, cache_lens, new_offsets, out, lse_out=None,
                         stream=None):
    _check(lib().evlnPagedStepCombine(handle, byref(params), _ptr(workspace), _ints(cache_lens),
                                      _ints(new_offsets), _ptr(out), _ptr(lse_out), _stream(stream)),
           "evlnPagedStepCombine")


def packed_params(num_q_heads, num_kv_heads, head_dim, instr_len, frame_tokens, action_tokens, num_frames,
                  cache_capacity, rope_theta, softmax_scale=0.0, kv_chunk_tiles=0, dtype=EVLN_BF16) -> evlnPackedParams:
    return evlnPackedParams(ctypes.sizeof(evlnPackedParams), dtype, num_q_heads, num_kv_heads, head_dim, instr_len,
                            frame_tokens, action_tokens, num_frames, cache_capacity, kv_chunk_tiles, softmax_scale,
                            rope_theta)


def evlnPackedWorkspaceSize(handle, params) -> int:
    v = c_size_t(0)
    _check(lib().evlnPackedWorkspaceSize(handle, byref(params), byref(v)), "evlnPackedWorkspaceSize")
    return int(v.value)


def evlnPackedForward(handle, params, q, k, v, k_cache, v_cache, workspace, out, lse_out=None, stream=None):
    """A packed sequence I, v_1, a_1, ..., v_N, a_N under the action-isolating mask, in one call."""
    _check(lib().evlnPackedForward(handle, byref(params), _ptr(q), _ptr(k), _ptr(v), int(q.stride(0)), int(k.stride(0)),
                                   int(v.stride(0)), _ptr(k_cache), _ptr(v_cache), _ptr(workspace),
                                   int(workspace.numel() * workspace.element_size()), _ptr(out), _ptr(lse_out),
                                   _stream(stream)), "evlnPackedForward")


def evlnStepAttentionNoAlloc(params, q_rot, k_cache, v_cache, out, lse_out=None, stream=None):
    """Attention + combine without a handle or a caller workspace: the split partials go to a
    scratch array built into the library (at most EVLN_NOALLOC_SCRATCH_BYTES).  For callers that
    must not allocate device memory; calls sharing a device must not overlap."""
    _check(lib().evlnStepAttentionNoAlloc(byref(params), _ptr(q_rot), _ptr(k_cache), _ptr(v_cache),
                                          _ptr(out), _ptr(lse_out), _stream(stream)),
           "evlnStepAttentionNoAlloc")


def gather_params(dtype, num_kv_heads, head_dim, store_capacity, work_capacity, rope_theta,
                  rope_table=None, rope_table_first_pos=0, rope_table_count=0) -> evlnGatherParams:
    code = {"bf16": EVLN_BF16, "f32": EVLN_F32}.get(dtype, dtype)
    return evlnGatherParams(ctypes.sizeof(evlnGatherParams), code, num_kv_heads, head_dim, store_capacity,
                            work_capacity, rope_theta, _ptr(rope_table), rope_table_first_pos, rope_table_count)


def evlnSampleFrames(sampler: int, num_frames: int, budget: int, stride: int = 1):
    """Host helper: indices of the history frames the sampler keeps (ascending)."""
    buf = (c_int * max(budget, 1))()
    cnt = lib().evlnSampleFrames(int(sampler), int(num_frames), int(budget), int(stride), buf)
    if cnt < 0:
        raise EvlnError(EVLN_INVALID_VALUE, "evlnSampleFrames")
    return [int(buf[i]) for i in range(cnt)]


def evlnStoreAppend(handle, params, k_new, v_new, store_len, k_store, v_store, stream=None):
    _check(lib().evlnStoreAppend(handle, byref(params), _ptr(k_new), _ptr(v_new), int(k_new.stride(0)),
                                 int(v_new.stride(0)), int(store_len), int(k_new.shape[0]), _ptr(k_store),
                                 _ptr(v_store), _stream(stream)), "evlnStoreAppend")


def evlnGatherRope(handle, params, seg_src, seg_len, k_store, v_store, k_work, v_work, stream=None) -> int:
    """Lays the kept store segments out in the working cache; returns the number of tokens laid out."""
    total = c_int(0)
    _check(lib().evlnGatherRope(handle, byref(params), len(seg_src), _ints(seg_src), _ints(seg_len), _ptr(k_store),
                                _ptr(v_store), _ptr(k_work), _ptr(v_work), byref(total), _stream(stream)),
           "evlnGatherRope")
    return int(total.value)


def evlnStoreOffload(handle, params, k_store, v_store, src_slot, length, h_k_store, h_v_store, dst_slot, stream=None):
    """Device store slots -> pinned host store ``[Hkv, host_capacity, D]`` (asynchronous DMA)."""
    _check(lib().evlnStoreOffload(handle, byref(params), _ptr(k_store), _ptr(v_store), int(src_slot), int(length),
                                  _ptr(h_k_store), _ptr(h_v_store), int(h_k_store.shape[1]), int(dst_slot),
                                  _stream(stream)), "evlnStoreOffload")


def evlnStoreFetch(handle, params, h_k_store, h_v_store, src_slot, length, k_store, v_store, dst_slot, stream=None):
    """Pinned host store slots -> device store slots (asynchronous DMA)."""
    _check(lib().evlnStoreFetch(handle, byref(params), _ptr(h_k_store), _ptr(h_v_store), int(h_k_store.shape[1]),
                                int(src_slot), int(length), _ptr(k_store), _ptr(v_store), int(dst_slot),
                                _stream(stream)), "evlnStoreFetch")
