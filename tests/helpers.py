"""Shared test plumbing: run a step through the C-ABI on the GPU, run it through the oracle,
and compare.  The two sides only share the seeded inputs."""
from __future__ import annotations

import numpy as np
import torch

from oracle import step_oracle as so
from paper_2512_10310_b200 import binding as B


def f64(t: torch.Tensor) -> np.ndarray:
    return np.ascontiguousarray(t.detach().cpu().to(torch.float64).numpy())


def bf16_ordered_bits(t: torch.Tensor) -> np.ndarray:
    """Map bf16 values to integers whose difference counts representable values between them."""
    bits = t.detach().cpu().contiguous().view(torch.int16).numpy().astype(np.int64) & 0xFFFF
    return np.where(bits & 0x8000, -(bits & 0x7FFF), bits)


def bf16_ulp_distance(gpu_bf16: torch.Tensor, ref_f64: np.ndarray) -> np.ndarray:
    ref = torch.from_numpy(ref_f64).to(torch.float32).to(torch.bfloat16)   # exact: already bf16 values
    return np.abs(bf16_ordered_bits(gpu_bf16) - bf16_ordered_bits(ref))


class GpuStep:
    """Device buffers of one layer + the three calls of a step, all through the C-ABI."""

    def __init__(self, handle, dtype, Hq, Hkv, D, capacity, theta, max_new, scale=0.0,
                 num_splits=0, kernel=B.EVLN_KERNEL_AUTO, device="cuda:0", fused=False):
        self.h, self.dtype, self.Hq, self.Hkv, self.D = handle, dtype, Hq, Hkv, D
        self.cap, self.theta, self.scale = capacity, theta, scale
        self.num_splits, self.kernel = num_splits, kernel
        self.tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
        self.dev = device
        # canaries: cache slots the step must not touch keep this bit pattern
        self.k_cache = torch.full((Hkv, capacity, D), 7.0, dtype=self.tdt, device=device)
        self.v_cache = torch.full((Hkv, capacity, D), -3.0, dtype=self.tdt, device=device)
        self.max_new = max_new
        self.fused = fused        # evlnStep instead of the three calls

    def load_cache(self, k_tok_major, v_tok_major):
        L = k_tok_major.shape[0]
        self.k_cache[:, :L] = k_tok_major.to(self.dev).permute(1, 0, 2)
        self.v_cache[:, :L] = v_tok_major.to(self.dev).permute(1, 0, 2)

    def params(self, L, n):
        return B.step_params(self.dtype, self.Hq, self.Hkv, self.D, L, n, self.cap, self.theta,
                             self.scale, self.num_splits, self.kernel)

    def step(self, L, q_new, k_new, v_new):
        n = q_new.shape[0]
        p = self.params(L, n)
        q_new, k_new, v_new = (t.to(self.dev).contiguous() for t in (q_new, k_new, v_new))
        q_rot = torch.empty(B.evlnStepQRotSize(self.h, p), dtype=torch.uint8, device=self.dev)
        ws = torch.empty(max(B.evlnStepWorkspaceSize(self.h, p), 16), dtype=torch.uint8, device=self.dev)
        out = torch.full((n, self.Hq, self.D), float("nan"), dtype=self.tdt, device=self.dev)
        lse = torch.full((n, self.Hq), float("nan"), dtype=torch.float32, device=self.dev)
        if self.fused:
            B.evlnStep(self.h, p, q_new, k_new, v_new, q_rot, self.k_cache, self.v_cache, ws, out, lse)
        else:
            B.evlnRopeAppend(self.h, p, q_new, k_new, v_new, q_rot, self.k_cache, self.v_cache)
            B.evlnStepAttention(self.h, p, q_rot, self.k_cache, self.v_cache, ws)
            B.evlnStepCombine(self.h, p, ws, out, lse)
        status = B.evlnGetDeviceStatus(self.h)
        assert status == 0, f"device status {status}: a bounded wait expired"
        G = self.Hq // self.Hkv
        q_rot_t = q_rot[: n * self.Hq * self.D * q_new.element_size()].view(self.tdt).view(self.Hkv, n, G, self.D)
        q_rot_tok = q_rot_t.permute(1, 0, 2, 3).reshape(n, self.Hq, self.D)
        return dict(out=out, lse=lse, q_rot=q_rot_tok, splits=B.evlnStepNumSplits(self.h, p))


def oracle_step(dtype, k_cache_tok, v_cache_tok, q_new, k_new, v_new, L, theta, cap=None, scale=0.0):
    """Oracle on the same inputs; returns result dict + the float64 caches [cap,Hkv,D]."""
    n, Hkv, D = k_new.shape
    cap = cap or (L + n)
    kc = np.zeros((cap, Hkv, D))
    vc = np.zeros((cap, Hkv, D))
    kc[:L] = f64(k_cache_tok[:L])
    vc[:L] = f64(v_cache_tok[:L])
    r = so.step(f64(q_new), f64(k_new), f64(v_new), kc, vc, L, theta, scale, storage=dtype)
    r["k_cache"], r["v_cache"] = kc, vc
    return r


def check_cache(gs: GpuStep, ref, L, n):
    """Appended K within 1 ulp (bf16) / 1e-6 (f32) of the oracle, V bit-exact, other slots untouched."""
    kc = gs.k_cache[:, L:L + n].permute(1, 0, 2)
    vc = gs.v_cache[:, L:L + n].permute(1, 0, 2)
    if gs.dtype == "bf16":
        d = bf16_ulp_distance(kc, ref["k_cache"][L:L + n])
        assert d.max() <= 1, f"K cache off by {d.max()} bf16 ulp"
        assert (d > 0).mean() < 0.05, "too many K elements off by one ulp"
    else:
        assert np.abs(f64(kc) - ref["k_cache"][L:L + n]).max() <= 1e-6
    assert np.array_equal(f64(vc), ref["v_cache"][L:L + n]), "V must be stored bit-exactly"
    assert bool((gs.k_cache[:, L + n:] == 7.0).all()) and bool((gs.v_cache[:, L + n:] == -3.0).all()), \
        "slots past L+n were touched"


def check_output(dtype, out, lse, ref_out, ref_lse, lse_tol=1e-3, rel_tol=1e-2, abs_tol=1e-2, elem_tol=1e-2):
    """Gates of the bf16 path: the mandated absolute ones (max-abs 1e-2, mean-abs 1e-3), the relative
    Frobenius error, and an element-wise one tied to the scale of the reference,
    |d| <= elem_tol (|ref| + rms of the element's own row of ref): at the mandated input scale the
    outputs are ~1e-3, so the absolute gates alone would let a wrong row through, and one wrong
    element moves the Frobenius norm by next to nothing.  Measured on the workloads here the worst
    element reaches 0.37 - 0.60 % of (|ref| + row rms) (bf16 P and Q operands, one bf16 rounding of
    the result: ~2^-9 relative each, spread over the row), so a bound of 1 % fails one wrong element
    or one row off by a few per cent while leaving the arithmetic a margin of 1.7."""
    o, r = f64(out), ref_out
    err = np.abs(o - r)
    assert np.isfinite(o).all(), "non-finite output"
    if dtype == "bf16":
        assert err.max() <= abs_tol, f"max-abs {err.max():.3e} > {abs_tol}"
        assert err.mean() <= abs_tol / 10, f"mean-abs {err.mean():.3e} > {abs_tol / 10}"
        rel = np.linalg.norm(o - r) / np.linalg.norm(r)
        assert rel <= rel_tol, f"relative Frobenius error {rel:.3e} > {rel_tol}"
        if elem_tol is not None:
            rms = np.sqrt(np.mean(r * r, axis=-1, keepdims=True))
            bound = elem_tol * (np.abs(r) + rms) + 1e-30
            worst = float((err / bound).max())
            assert worst <= 1.0, f"element-wise error {worst:.2f} x {elem_tol:.2e} (|ref| + row rms(ref))"
    else:
        assert err.max() <= 1e-5, f"max-abs {err.max():.3e} > 1e-5"
        rel = np.linalg.norm(o - r) / np.linalg.norm(r)
        assert rel <= 1e-5, f"relative Frobenius error {rel:.3e}"
    if lse is not None:
        le = np.abs(f64(lse) - ref_lse).max()
        assert le <= (lse_tol if dtype == "bf16" else 1e-5), f"lse max-abs {le:.3e}"
