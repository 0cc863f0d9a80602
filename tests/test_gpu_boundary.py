"""Boundary behaviour on the GPU that needs no oracle: the position table gives the same bits as
the in-kernel trigonometry, a bounded wait that runs out is reported and leaves the context
usable, and creating a handle does not move the caller's current device."""
import dataclasses

import pytest
import torch

from paper_2512_10310_b200 import binding as B
from paper_2512_10310_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def handle():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    h = B.evlnCreate(0)
    yield h
    B.evlnDestroy(h)


def _append(handle, cfg, x, table=None, first=0, count=0):
    dev = "cuda:0"
    L, n, Hq, Hkv, D = cfg.cache_len, cfg.num_new, cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim
    p = B.step_params(cfg.dtype, Hq, Hkv, D, L, n, L + n, cfg.rope_theta, rope_table=table,
                      rope_table_first_pos=first, rope_table_count=count)
    dt = cfg.torch_dtype
    kc = torch.zeros((Hkv, L + n, D), dtype=dt, device=dev)
    vc = torch.zeros((Hkv, L + n, D), dtype=dt, device=dev)
    q, k, v = (x[s].to(dev) for s in ("q_new", "k_new", "v_new"))
    q_rot = torch.zeros(B.evlnStepQRotSize(handle, p), dtype=torch.uint8, device=dev)
    B.evlnRopeAppend(handle, p, q, k, v, q_rot, kc, vc)
    torch.cuda.synchronize()
    return q_rot, kc, vc


@pytest.mark.parametrize("base", [W.STEP_7B, W.TINY_F32])
def test_position_table_gives_the_same_bits(handle, base):
    cfg = dataclasses.replace(base, name="table", cache_len=20500 if base.dtype == "bf16" else 256, num_new=37)
    x = W.make_new_tokens(cfg)
    L, n, D = cfg.cache_len, cfg.num_new, cfg.head_dim
    # a table that starts before L and ends after L + n, as a model would make it for a whole step
    first, count = L - 5, n + 9
    table = torch.zeros(B.evlnRopeTableBytes(D, count), dtype=torch.uint8, device="cuda:0")
    B.evlnRopeTable(handle, D, cfg.rope_theta, first, count, table)
    ref = _append(handle, cfg, x)
    got = _append(handle, cfg, x, table, first, count)
    for a, b in zip(ref, got):
        assert torch.equal(a, b)
    # entry (p, 0) is (cos, sin) of the position itself (theta^0 = 1)
    t = table.view(torch.float64).view(count, D // 2, 2)
    pos = torch.arange(first, first + count, dtype=torch.float64, device="cuda:0")
    # (the angle goes through pos * omega / pi in double: ~pos * 2e-16 rad of rounding)
    assert (t[:, 0, 0] - torch.cos(pos)).abs().max().item() < 1e-10
    assert (t[:, 0, 1] - torch.sin(pos)).abs().max().item() < 1e-10


def test_position_table_must_cover_the_step(handle):
    cfg = W.STEP_7B
    table = torch.zeros(B.evlnRopeTableBytes(128, 196), dtype=torch.uint8, device="cuda:0")
    for first, count in ((4097, 196), (4096, 195), (4000, 100)):
        p = B.step_params("bf16", 28, 4, 128, 4096, 196, 4292, cfg.rope_theta, rope_table=table,
                          rope_table_first_pos=first, rope_table_count=count)
        with pytest.raises(B.EvlnError) as e:
            B.evlnStepWorkspaceSize(handle, p)
        assert e.value.status == B.EVLN_INVALID_VALUE


def test_bounded_wait_that_runs_out_is_reported_and_harmless(handle):
    assert B.evlnGetDeviceStatus(handle) == 0
    B.evlnSelfTestBoundedWait(handle, 100000)
    # the kernel returned by itself; the word carries the self-test's code and the call says "timeout"
    v = B.c_int(0)
    st = B.lib().evlnGetDeviceStatus(handle, B._stream(None), B.byref(v))
    assert st == B.EVLN_DEVICE_TIMEOUT and v.value == B.EVLN_SELFTEST_STATUS_CODE
    # reading cleared it
    assert B.evlnGetDeviceStatus(handle) == 0
    # ... and the context still runs a step
    cfg = dataclasses.replace(W.STEP_7B, name="after_timeout", cache_len=300, num_new=40)
    x = W.make_new_tokens(cfg)
    _append(handle, cfg, x)
    assert B.evlnGetDeviceStatus(handle) == 0
    with pytest.raises(B.EvlnError):
        B.evlnSelfTestBoundedWait(handle, 10)          # limits below 1000 cycles are refused


def test_create_leaves_the_current_device_alone():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    before = torch.cuda.current_device()
    h = B.evlnCreate(0)
    try:
        assert torch.cuda.current_device() == before
    finally:
        B.evlnDestroy(h)
