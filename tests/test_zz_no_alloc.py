"""The allocation-free entry point gives the same result as the regular attention + combine.

Some users of this library cannot allocate device memory once they are running (all of it
belongs to their own arena, or cudaMalloc's device-wide synchronisation is unacceptable in
their control loop), so they can create neither a handle nor a workspace.
evlnStepAttentionNoAlloc serves them from a scratch array inside the library.  Here it is
called twice in a row through the C-ABI, on different inputs, and each result is compared with
the handle + caller-workspace path within the tolerance of the other parity tests (the second
call also shows that what the first left in the shared scratch does no harm), and with the fp64
oracle on the same inputs, so that the two CUDA paths cannot agree on a wrong answer.  The status
word of the allocation-free path (read through evlnGetDeviceStatus without a handle) must stay
clear.  Collected last on purpose, so that a run stopping at the first failure has already run
everything else.
"""
import dataclasses

import pytest
import torch

from paper_2512_10310_b200 import binding as B
from paper_2512_10310_b200 import workloads as W
from tests.helpers import check_output, oracle_step

pytestmark = pytest.mark.gpu


def _regular(handle, p, q, k, v, kc, vc, n, Hq, D):
    dev = q.device
    q_rot = torch.empty(B.evlnStepQRotSize(handle, p), dtype=torch.uint8, device=dev)
    ws = torch.empty(B.evlnStepWorkspaceSize(handle, p), dtype=torch.uint8, device=dev)
    out = torch.empty((n, Hq, D), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((n, Hq), dtype=torch.float32, device=dev)
    B.evlnRopeAppend(handle, p, q, k, v, q_rot, kc, vc)
    B.evlnStepAttention(handle, p, q_rot, kc, vc, ws)
    B.evlnStepCombine(handle, p, ws, out, lse)
    assert B.evlnGetDeviceStatus(handle) == 0
    return q_rot, out, lse


def test_no_alloc_matches_regular_path_twice():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    dev = "cuda:0"
    torch.cuda.set_device(0)
    handle = B.evlnCreate(0)
    try:
        for call, (L, n, seed) in enumerate([(1500, 196, 21), (700, 130, 22)]):
            cfg = dataclasses.replace(W.STEP_7B, name=f"noalloc{call}", cache_len=L, num_new=n, seed=seed)
            x = W.make_step_inputs(cfg)
            Hq, Hkv, D = cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim
            p = B.step_params("bf16", Hq, Hkv, D, L, n, L + n, cfg.rope_theta)
            kc = torch.zeros((Hkv, L + n, D), dtype=torch.bfloat16, device=dev)
            vc = torch.zeros((Hkv, L + n, D), dtype=torch.bfloat16, device=dev)
            kc[:, :L] = x["k_cache"].to(dev).permute(1, 0, 2)
            vc[:, :L] = x["v_cache"].to(dev).permute(1, 0, 2)
            q, k, v = (x[s].to(dev) for s in ("q_new", "k_new", "v_new"))
            q_rot, ref_out, ref_lse = _regular(handle, p, q, k, v, kc, vc, n, Hq, D)

            out = torch.full((n, Hq, D), float("nan"), dtype=torch.bfloat16, device=dev)
            lse = torch.full((n, Hq), float("nan"), dtype=torch.float32, device=dev)
            B.evlnStepAttentionNoAlloc(p, q_rot, kc, vc, out, lse)
            torch.cuda.synchronize()
            err = (out.float() - ref_out.float()).abs()
            assert torch.isfinite(out.float()).all()
            assert err.max().item() <= 1e-2 and err.mean().item() <= 1e-3
            rel = (out.float() - ref_out.float()).norm() / ref_out.float().norm()
            assert rel.item() <= 1e-2
            assert (lse - ref_lse).abs().max().item() <= 1e-3
            assert B.evlnGetDeviceStatus(None) == 0, "a kernel of the allocation-free call gave up on a bounded wait"
            r = oracle_step("bf16", x["k_cache"], x["v_cache"], x["q_new"], x["k_new"], x["v_new"], L, cfg.rope_theta)
            check_output("bf16", out, lse, r["out"], r["lse"])
            check_output("bf16", ref_out, ref_lse, r["out"], r["lse"])
    finally:
        B.evlnDestroy(handle)


def test_no_alloc_rejects_oversized_problems():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    torch.cuda.set_device(0)
    # 70B-class long-history shape with 8 KV splits asked for: 67 MB of split partials, far beyond
    # the built-in scratch (the check comes before any launch, so the dummy buffers are never used)
    cfg = W.LONG_70B
    p = B.step_params("bf16", cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, cfg.cache_len, cfg.num_new,
                      cfg.cache_len + cfg.num_new, cfg.rope_theta, num_splits=8)
    buf = torch.zeros(4096, dtype=torch.uint8, device="cuda:0")
    with pytest.raises(B.EvlnError) as e:
        B.evlnStepAttentionNoAlloc(p, buf, buf, buf, buf, None)
    assert e.value.status == B.EVLN_WORKSPACE_TOO_SMALL
