"""GPU parity for packed sequences under the action-isolating mask (Sec. 3.3).

The CUDA path has no mask argument.  evlnPackedForward runs the instruction and visual rows as one
causal step and all action chunks as one batch of items that share prefixes of the cache; the same
rows also come out of a loop of ordinary steps (a frame is a step that stays in the cache, its
action chunk a step at the advanced length whose appended keys the next frame overwrites).  Every
row of either is compared with dense masked attention of the whole packed sequence computed by the
oracle.
"""
import numpy as np
import pytest
import torch

from oracle import packed_mask_oracle as pm
from oracle import step_oracle as so
from paper_2512_10310_b200 import binding as B
from tests.helpers import GpuStep, bf16_ulp_distance, check_output, f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def handle():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    h = B.evlnCreate(0)
    yield h
    B.evlnDestroy(h)


@pytest.mark.parametrize("I,F,A,N", [(60, 196, 6, 5), (37, 64, 8, 9)])
def test_packed_sequence_with_action_isolation(handle, I, F, A, N):
    Hq, Hkv, D, theta = 28, 4, 128, 1.0e6
    T = I + N * (F + A)
    gen = torch.Generator().manual_seed(100 + N)
    q = (torch.randn((T, Hq, D), generator=gen) * 0.3).to(torch.bfloat16)
    k = (torch.randn((T, Hkv, D), generator=gen) * 0.3).to(torch.bfloat16)
    v = torch.randn((T, Hkv, D), generator=gen).to(torch.bfloat16)
    kind, frame, pos = pm.packed_layout(I, F, A, N)
    mask = pm.action_isolating_mask(kind, frame)
    ref_out, ref_lse = pm.masked_attention(f64(q), f64(k), f64(v), mask, pos, theta, round_k=so.round_bf16)

    gs = GpuStep(handle, "bf16", Hq, Hkv, D, I + N * F + A, theta, max(I, F))
    rows = torch.from_numpy(np.where(kind == 0)[0])
    g = gs.step(0, q[rows], k[rows], v[rows])
    check_output("bf16", g["out"], g["lse"], ref_out[rows], ref_lse[rows])
    L = I
    for t in range(N):
        rows = torch.from_numpy(np.where((kind == 1) & (frame == t))[0])
        g = gs.step(L, q[rows], k[rows], v[rows])
        check_output("bf16", g["out"], g["lse"], ref_out[rows], ref_lse[rows])
        L += F
        rows = torch.from_numpy(np.where((kind == 2) & (frame == t))[0])
        g = gs.step(L, q[rows], k[rows], v[rows])              # L stays: the chunk is not kept
        check_output("bf16", g["out"], g["lse"], ref_out[rows], ref_lse[rows])


def _packed_inputs(I, F, A, N, seed):
    Hq, Hkv, D = 28, 4, 128
    T = I + N * (F + A)
    gen = torch.Generator().manual_seed(seed)
    q = (torch.randn((T, Hq, D), generator=gen) * 0.3).to(torch.bfloat16)
    k = (torch.randn((T, Hkv, D), generator=gen) * 0.3).to(torch.bfloat16)
    v = torch.randn((T, Hkv, D), generator=gen).to(torch.bfloat16)
    return q, k, v


@pytest.mark.parametrize("I,F,A,N,chunk", [
    (60, 196, 6, 5, 0),       # the shapes of the loop test
    (37, 64, 8, 9, 0),
    (37, 64, 8, 9, 1),        # one KV tile per work item: every chunk is split, prefix and own tiles apart
    (256, 196, 8, 12, 0),     # a longer episode: chunks with 4 to 21 cache tiles
    (130, 70, 20, 3, 2),      # 140 rows per chunk and kv head: both query tiles of a pair in use
    (5, 3, 1, 4, 0),          # everything shorter than one tile
    (64, 128, 0, 2, 0),       # no action tokens at all
    (50, 0, 4, 3, 0),         # no visual tokens: every chunk follows the instruction directly
])
def test_packed_forward_call(handle, I, F, A, N, chunk):
    Hq, Hkv, D, theta = 28, 4, 128, 1.0e6
    dev = "cuda:0"
    q, k, v = _packed_inputs(I, F, A, N, 200 + N + A)
    T = q.shape[0]
    kind, frame, pos = pm.packed_layout(I, F, A, N)
    mask = pm.action_isolating_mask(kind, frame)
    ref_out, ref_lse = pm.masked_attention(f64(q), f64(k), f64(v), mask, pos, theta, round_k=so.round_bf16)

    n_vis = I + N * F
    cap = n_vis + 3
    p = B.packed_params(Hq, Hkv, D, I, F, A, N, cap, theta, kv_chunk_tiles=chunk)
    ws = torch.empty(B.evlnPackedWorkspaceSize(handle, p), dtype=torch.uint8, device=dev)
    # the packed tokens arrive as one fused [T, Hq + 2 Hkv, D] buffer: strided views
    qkv = torch.cat([q, k, v], dim=1).contiguous().to(dev)
    kc = torch.full((Hkv, cap, D), 7.0, dtype=torch.bfloat16, device=dev)
    vc = torch.full((Hkv, cap, D), -3.0, dtype=torch.bfloat16, device=dev)
    out = torch.full((T, Hq, D), float("nan"), dtype=torch.bfloat16, device=dev)
    lse = torch.full((T, Hq), float("nan"), dtype=torch.float32, device=dev)
    B.evlnPackedForward(handle, p, qkv[:, :Hq], qkv[:, Hq:Hq + Hkv], qkv[:, Hq + Hkv:], kc, vc, ws, out, lse)
    assert B.evlnGetDeviceStatus(handle) == 0
    check_output("bf16", out, lse, ref_out, ref_lse)
    # ... and per kind of row, so that the few action rows cannot hide behind the visual ones
    for sel in (kind != 2, kind == 2):
        rows = torch.from_numpy(np.where(sel)[0])
        if len(rows):
            check_output("bf16", out[rows], lse[rows], ref_out[rows.numpy()], ref_lse[rows.numpy()])
    # the cache holds the instruction + visual tokens at contiguous slots: rotated keys within one
    # ulp of the oracle's, values bit for bit; slots past them untouched
    vis = np.where(kind != 2)[0]
    kr = so.round_bf16(pm.rope_at(f64(k), pos, theta))[vis]
    assert bf16_ulp_distance(kc[:, :n_vis].permute(1, 0, 2), kr).max() <= 1
    assert np.array_equal(f64(vc[:, :n_vis].permute(1, 0, 2)), f64(v)[vis])
    assert bool((kc[:, n_vis:] == 7.0).all()) and bool((vc[:, n_vis:] == -3.0).all())


def test_packed_forward_argument_errors(handle):
    p = B.packed_params(28, 4, 128, 60, 196, 6, 5, 100, 1e6)          # 1040 visual tokens do not fit 100 slots
    with pytest.raises(B.EvlnError) as e:
        B.evlnPackedWorkspaceSize(handle, p)
    assert e.value.status == B.EVLN_CACHE_FULL
    p = B.packed_params(28, 4, 64, 60, 196, 6, 5, 2000, 1e6)
    with pytest.raises(B.EvlnError) as e:
        B.evlnPackedWorkspaceSize(handle, p)
    assert e.value.status == B.EVLN_NOT_SUPPORTED
