"""GPU parity for packed sequences under the action-isolating mask (Sec. 3.3).

The CUDA path has no mask argument: a frame is a step that stays in the cache, its action chunk is
a step at the advanced length whose appended keys the next frame overwrites.  Every row of that
loop is compared with dense masked attention of the whole packed sequence computed by the oracle.
"""
import numpy as np
import pytest
import torch

from oracle import packed_mask_oracle as pm
from oracle import step_oracle as so
from paper_2512_10310_b200 import binding as B
from tests.helpers import GpuStep, check_output, f64

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
