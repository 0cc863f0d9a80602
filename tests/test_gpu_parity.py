"""GPU parity: the CUDA path, called through the C-ABI, against the fp64 CPU oracle on the
same seeded inputs.  Tolerances: appended K within 1 bf16 ulp (1e-6 abs for fp32), V
bit-exact, attention output max-abs 1e-2 and mean-abs 1e-3 for bf16 (1e-5 for fp32), plus a
relative Frobenius gate of 1e-2 because the absolute gates are loose at the small input
scale of the 7B / 70B workloads."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import step_oracle as so
from paper_2512_10310_b200 import binding as B
from paper_2512_10310_b200 import workloads as W
from tests.helpers import GpuStep, check_cache, check_output, f64, oracle_step

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def handle():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    h = B.evlnCreate(0)
    yield h
    B.evlnDestroy(h)


def _run(handle, cfg, kernel=B.EVLN_KERNEL_AUTO, num_splits=0, extra_cap=37, lse_tol=1e-3, rel_tol=1e-2,
         inputs=None, round_q=False, abs_tol=1e-2, fused=False, elem_tol=1e-2):
    x = inputs or W.make_step_inputs(cfg)
    L, n = cfg.cache_len, cfg.num_new
    gs = GpuStep(handle, cfg.dtype, cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, L + n + extra_cap,
                 cfg.rope_theta, n, num_splits=num_splits, kernel=kernel, fused=fused)
    gs.load_cache(x["k_cache"], x["v_cache"])
    g = gs.step(L, x["q_new"], x["k_new"], x["v_new"])
    r = oracle_step(cfg.dtype, x["k_cache"], x["v_cache"], x["q_new"], x["k_new"], x["v_new"], L,
                    cfg.rope_theta)
    check_cache(gs, r, L, n)
    ref_out, ref_lse = r["out"], r["lse"]
    if round_q:
        # the tensor-core operand is the bf16-rounded rotated query: feed the oracle the same
        # rounded q so that the comparison isolates the kernel from that input rounding
        ref_out, ref_lse = so.attend_range(so.round_bf16(r["q_rot"]), r["k_cache"], r["v_cache"], L, 0, L + n)
    check_output(cfg.dtype, g["out"], g["lse"], ref_out, ref_lse, lse_tol=lse_tol, rel_tol=rel_tol,
                 abs_tol=abs_tol, elem_tol=elem_tol)
    # rotated queries: bf16 rounding of the oracle's q_rot, at most one ulp apart
    if cfg.dtype == "bf16":
        from tests.helpers import bf16_ulp_distance
        assert bf16_ulp_distance(g["q_rot"], so.round_bf16(r["q_rot"])).max() <= 1
    else:
        assert np.abs(f64(g["q_rot"]) - r["q_rot"]).max() <= 1e-6
    return g, r


def test_tiny_fp32_step(handle):
    _run(handle, W.TINY_F32)


@pytest.mark.parametrize("splits", [1, 3])
def test_tiny_fp32_step_forced_splits(handle, splits):
    _run(handle, W.TINY_F32, num_splits=splits)


def test_simt_kernel_bf16_small(handle):
    cfg = dataclasses.replace(W.STEP_7B, name="simt_small", cache_len=300, num_new=50)
    _run(handle, cfg, kernel=B.EVLN_KERNEL_SIMT)


def test_simt_kernel_bf16_d64(handle):
    cfg = W.StepConfig("d64", "bf16", 4, 2, 64, 200, 33, 1e4, 0.3, 11)
    _run(handle, cfg)


# ---- tensor-core kernel ---------------------------------------------------------------------

@pytest.mark.parametrize("L,n,splits", [
    (0, 128, 1),          # instruction prefill, one exact tile pair per head... (G=7 -> ragged rows)
    (0, 5, 0),            # shorter than one KV tile
    (100, 1, 1),          # a single new token
    (128, 37, 2),         # second query tile absent (259 rows -> 1.02 units)
    (300, 50, 0),
    (1000, 196, 3),
    (2047, 130, 5),       # cache length not a multiple of anything
])
def test_tc_kernel_shapes(handle, L, n, splits):
    cfg = dataclasses.replace(W.STEP_7B, name=f"tc_{L}_{n}", cache_len=L, num_new=n, seed=100 + L + n)
    _run(handle, cfg, num_splits=splits)


def test_tc_kernel_more_splits_than_tiles(handle):
    cfg = dataclasses.replace(W.STEP_7B, name="oversplit", cache_len=200, num_new=20, seed=5)
    _run(handle, cfg, num_splits=7)       # 2 KV tiles, 7 splits: five splits are empty


def test_tc_kernel_sharp_logits(handle):
    # unit-variance q and k: logits ~ N(0,1), softmax far from uniform
    cfg = dataclasses.replace(W.STEP_7B, name="sharp", cache_len=1500, num_new=100, input_scale=1.0, seed=6)
    # (the oracle's unrounded query and the bf16 operand differ by ~1 % in these logits: Frobenius gate only)
    _run(handle, cfg, lse_tol=2e-2, rel_tol=1.5e-2, elem_tol=None)


def test_tc_kernel_planted_high_logit_keys(handle):
    # a few cached keys aligned with the queries dominate the softmax; the running maximum has to
    # move by far more than the lazy-rescale threshold in a late tile
    cfg = dataclasses.replace(W.STEP_7B, name="planted", cache_len=900, num_new=64, input_scale=1.0, seed=7)
    x = W.make_step_inputs(cfg)
    x["k_cache"][850:853] *= 6.0
    x["k_new"][40:42] *= 8.0
    # logits reach ~30 here, so the bf16 rounding of the rotated query alone moves them by ~1e-2;
    # outputs are O(1): the absolute gate scales with them
    _run(handle, cfg, num_splits=1, lse_tol=1e-3, rel_tol=1e-2, inputs=x, round_q=True, abs_tol=4e-2, elem_tol=2e-2)
    _run(handle, cfg, num_splits=3, lse_tol=1e-3, rel_tol=1e-2, inputs=x, round_q=True, abs_tol=4e-2, elem_tol=2e-2)


def test_tc_kernel_reference_moves_in_late_tiles(handle):
    # Cached keys scaled up so far that, for about half of the rows, a score in a late KV tile
    # exceeds the row's first-tile maximum by much more than 2^64 (twice, and once more inside the
    # new frame): the softmax threads have to move the row's reference and rescale what they have
    # accumulated and handed over.  Rows for which the scaled key scores negative must not move.
    cfg = dataclasses.replace(W.STEP_7B, name="moves", cache_len=1700, num_new=96, input_scale=1.0, seed=11)
    x = W.make_step_inputs(cfg)
    x["k_cache"][700] *= 48.0
    x["k_cache"][1410:1412] *= 128.0
    x["k_new"][50] *= 250.0
    x["k_new"][95] *= 400.0       # the very last key: its rows' threads are already exchanging their sums
    # the winning scores are several hundred: fp32 accumulation on the tensor core resolves them to
    # a few 1e-5 relative, which is what the log-sum-exp gate allows here
    for splits in (1, 2):
        _run(handle, cfg, num_splits=splits, lse_tol=5e-2, rel_tol=1e-2, inputs=x, round_q=True, abs_tol=5e-2, elem_tol=2e-2)


# ---- few new tokens: one CTA per (kv head, split) --------------------------------------------

@pytest.mark.parametrize("L,n,splits", [
    (4096, 8, 0),         # an action chunk after a frame, schedule chosen by the library
    (4096, 1, 0),         # one token
    (20656, 8, 0),        # end of a 100-step episode
    (4090, 8, 0),         # the new tokens straddle two KV tiles
    (1000, 18, 4),        # 126 rows: the most one tile takes
    (1000, 19, 3),        # 133 rows: back on CTA pairs
    (130, 4, 2),          # one tile per split
    (0, 3, 1),            # no history at all
    (300, 16, 9),         # more splits than KV tiles: empty splits
    (257, 5, 0),          # rows in the first lane quarter only
    (3000, 10, 32),       # the largest split count
])
def test_tc_kernel_few_new_tokens(handle, L, n, splits):
    cfg = dataclasses.replace(W.STEP_7B, name=f"few_{L}_{n}", cache_len=L, num_new=n, seed=300 + L + n)
    _run(handle, cfg, num_splits=splits)


@pytest.mark.parametrize("L,n,splits", [
    (4096, 8, 0), (4096, 1, 0), (20656, 8, 0), (4090, 8, 0), (4095, 2, 5), (1000, 18, 4), (130, 4, 2), (0, 3, 1),
    (300, 16, 9), (257, 5, 0), (3000, 10, 32), (3000, 10, 1), (127, 1, 0), (128, 1, 0),
])
def test_one_call_step_of_few_new_tokens(handle, L, n, splits):
    cfg = dataclasses.replace(W.STEP_7B, name=f"one_{L}_{n}", cache_len=L, num_new=n, seed=500 + L + n)
    _run(handle, cfg, num_splits=splits, fused=True)


def test_few_new_tokens_reference_moves(handle):
    # as test_tc_kernel_reference_moves_in_late_tiles, on the one-CTA kernel with idle lane quarters
    cfg = dataclasses.replace(W.STEP_7B, name="few_moves", cache_len=1700, num_new=8, input_scale=1.0, seed=12)
    x = W.make_step_inputs(cfg)
    x["k_cache"][700] *= 48.0
    x["k_cache"][1410:1412] *= 128.0
    x["k_new"][5] *= 250.0
    x["k_new"][7] *= 400.0
    for splits in (1, 2):
        _run(handle, cfg, num_splits=splits, lse_tol=5e-2, rel_tol=1e-2, inputs=x, round_q=True, abs_tol=5e-2, elem_tol=2e-2)
        _run(handle, cfg, num_splits=splits, lse_tol=5e-2, rel_tol=1e-2, inputs=x, round_q=True, abs_tol=5e-2,
             fused=True, elem_tol=2e-2)


@pytest.mark.parametrize("L,n", [(4096, 196), (4096, 8), (700, 130), (2000, 1), (4090, 8), (20656, 8)])
def test_fused_step_call_is_bitwise_the_three_calls(handle, L, n):
    cfg = dataclasses.replace(W.STEP_7B, name=f"fused_{L}_{n}", cache_len=L, num_new=n, seed=400 + n)
    x = W.make_step_inputs(cfg)
    res = []
    for fused in (False, True):
        gs = GpuStep(handle, "bf16", cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, L + n + 5, cfg.rope_theta, n,
                     fused=fused)
        gs.load_cache(x["k_cache"], x["v_cache"])
        g = gs.step(L, x["q_new"], x["k_new"], x["v_new"])
        res.append((g, gs))
    (a, gsa), (b, gsb) = res
    assert torch.equal(a["out"].view(torch.int16), b["out"].view(torch.int16))
    assert torch.equal(a["lse"], b["lse"])
    assert torch.equal(gsa.k_cache.view(torch.int16), gsb.k_cache.view(torch.int16))
    assert torch.equal(gsa.v_cache.view(torch.int16), gsb.v_cache.view(torch.int16))
    r = oracle_step("bf16", x["k_cache"], x["v_cache"], x["q_new"], x["k_new"], x["v_new"], L, cfg.rope_theta)
    check_output("bf16", b["out"], b["lse"], r["out"], r["lse"])


def test_fused_step_calls_in_a_chain(handle):
    # frame step, action step, next frame at the same length (the action keys are overwritten),
    # all through the one-call form back to back on one stream
    Hq, Hkv, D, theta = 28, 4, 128, 1.0e6
    I, F, A, N = 100, 196, 8, 4
    gen = torch.Generator().manual_seed(77)
    mk = lambda n, H, sc: (torch.randn((n, H, D), generator=gen) * sc).to(torch.bfloat16)
    cap = I + N * F + A
    gs = GpuStep(handle, "bf16", Hq, Hkv, D, cap, theta, F, fused=True)
    kc, vc = np.zeros((cap, Hkv, D)), np.zeros((cap, Hkv, D))
    L = 0
    steps = [(I, True)]
    for _ in range(N):
        steps += [(F, True), (A, False)]
    for n, keep in steps:
        q, k, v = mk(n, Hq, 0.3), mk(n, Hkv, 0.3), mk(n, Hkv, 1.0)
        g = gs.step(L, q, k, v)
        r = so.step(f64(q), f64(k), f64(v), kc, vc, L, theta, 0.0, storage="bf16")
        check_output("bf16", g["out"], g["lse"], r["out"], r["lse"])
        if keep:
            L += n


@pytest.mark.parametrize("n", [196, 8])
def test_strided_views_of_a_fused_qkv_buffer(handle, n):
    # q, k and v as the three views of one [n, Hq + 2 Hkv, D] buffer (token stride 36 * 128 elements)
    cfg = dataclasses.replace(W.STEP_7B, name=f"fusedqkv_{n}", cache_len=1500, num_new=n, seed=600 + n)
    x = W.make_step_inputs(cfg)
    Hq, Hkv, D, L = cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, cfg.cache_len
    qkv = torch.cat([x["q_new"], x["k_new"], x["v_new"]], dim=1).contiguous().to("cuda:0")
    q, k, v = qkv[:, :Hq], qkv[:, Hq:Hq + Hkv], qkv[:, Hq + Hkv:]
    assert not q.is_contiguous() and q.stride(0) == (Hq + 2 * Hkv) * D
    gs = GpuStep(handle, "bf16", Hq, Hkv, D, L + n, cfg.rope_theta, n)
    gs.load_cache(x["k_cache"], x["v_cache"])
    p = gs.params(L, n)
    q_rot = torch.empty(B.evlnStepQRotSize(handle, p), dtype=torch.uint8, device="cuda:0")
    ws = torch.empty(max(B.evlnStepWorkspaceSize(handle, p), 16), dtype=torch.uint8, device="cuda:0")
    out = torch.full((n, Hq, D), float("nan"), dtype=torch.bfloat16, device="cuda:0")
    lse = torch.full((n, Hq), float("nan"), dtype=torch.float32, device="cuda:0")
    B.evlnStep(handle, p, q, k, v, q_rot, gs.k_cache, gs.v_cache, ws, out, lse)
    assert B.evlnGetDeviceStatus(handle) == 0
    r = oracle_step("bf16", x["k_cache"], x["v_cache"], x["q_new"], x["k_new"], x["v_new"], L, cfg.rope_theta)
    check_cache(gs, r, L, n)
    check_output("bf16", out, lse, r["out"], r["lse"])


def test_one_call_step_fp32(handle):
    # the one-call form on the fp32 configuration (SIMT attention kernel)
    cfg = W.TINY_F32
    x = W.make_step_inputs(cfg)
    L, n = cfg.cache_len, cfg.num_new
    gs = GpuStep(handle, "f32", cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, L + n, cfg.rope_theta, n, fused=True)
    gs.load_cache(x["k_cache"], x["v_cache"])
    g = gs.step(L, x["q_new"], x["k_new"], x["v_new"])
    r = oracle_step("f32", x["k_cache"], x["v_cache"], x["q_new"], x["k_new"], x["v_new"], L, cfg.rope_theta)
    check_cache(gs, r, L, n)
    check_output("f32", g["out"], g["lse"], r["out"], r["lse"])


def test_tc_matches_simt_kernel_on_device(handle):
    cfg = dataclasses.replace(W.STEP_7B, name="cross", cache_len=700, num_new=90, seed=8)
    a, _ = _run(handle, cfg)
    b, _ = _run(handle, cfg, kernel=B.EVLN_KERNEL_SIMT)
    assert (a["out"].float() - b["out"].float()).abs().max().item() <= 2e-3


def test_step_7b_full(handle):
    g, _ = _run(handle, W.STEP_7B)
    assert g["splits"] >= 2


def test_results_are_bitwise_reproducible(handle):
    cfg = dataclasses.replace(W.STEP_7B, name="repro", cache_len=1024, num_new=196, seed=9)
    a, _ = _run(handle, cfg)
    b, _ = _run(handle, cfg)
    assert torch.equal(a["out"].view(torch.int16), b["out"].view(torch.int16))
    assert torch.equal(a["lse"], b["lse"])


def test_chained_steps_reuse_the_cache(handle):
    # instruction prefill then three frames through the same cache: equals the oracle chain
    cfg = dataclasses.replace(W.STEP_7B, name="chain", cache_len=0, num_new=0, seed=10)
    chunks = [256, 204, 204, 204]
    T = sum(chunks)
    gs = GpuStep(handle, "bf16", 28, 4, 128, T + 5, cfg.rope_theta, max(chunks))
    kc = np.zeros((T + 5, 4, 128))
    vc = np.zeros((T + 5, 4, 128))
    L = 0
    for s, n in enumerate(chunks):
        x = W.make_new_tokens(dataclasses.replace(cfg, num_new=n, seed=1000 + s))
        g = gs.step(L, x["q_new"], x["k_new"], x["v_new"])
        r = so.step(f64(x["q_new"]), f64(x["k_new"]), f64(x["v_new"]), kc, vc, L, cfg.rope_theta,
                    storage="bf16")
        check_output("bf16", g["out"], g["lse"], r["out"], r["lse"])
        L += n
    from tests.helpers import bf16_ulp_distance
    assert bf16_ulp_distance(gs.k_cache[:, :T].permute(1, 0, 2), kc[:T]).max() <= 1
    assert np.array_equal(f64(gs.v_cache[:, :T].permute(1, 0, 2)), vc[:T])


def test_long_70b_all_rows(handle):
    # full-size launch (L = 32768, 64 query heads, n = 256); the oracle computes every row
    cfg = W.LONG_70B
    x = W.make_step_inputs(cfg)
    L, n = cfg.cache_len, cfg.num_new
    gs = GpuStep(handle, "bf16", cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, L + n, cfg.rope_theta, n)
    gs.load_cache(x["k_cache"], x["v_cache"])
    g = gs.step(L, x["q_new"], x["k_new"], x["v_new"])
    ref = oracle_step("bf16", x["k_cache"], x["v_cache"], x["q_new"], x["k_new"], x["v_new"], L, cfg.rope_theta)
    check_cache(gs, ref, L, n)
    check_output("bf16", g["out"], g["lse"], ref["out"], ref["lse"])


# ---- boundary behaviour (argument errors launch nothing) ------------------------------------

def test_argument_errors(handle):
    p = B.step_params("bf16", 28, 4, 128, 10, 5, 12, 1e6)
    with pytest.raises(B.EvlnError) as e:
        B.evlnStepWorkspaceSize(handle, p)
    assert e.value.status == B.EVLN_CACHE_FULL
    p = B.step_params("bf16", 28, 5, 128, 10, 5, 100, 1e6)
    with pytest.raises(B.EvlnError) as e:
        B.evlnStepWorkspaceSize(handle, p)
    assert e.value.status == B.EVLN_INVALID_VALUE
    p = B.step_params("bf16", 28, 4, 96, 10, 5, 100, 1e6)
    with pytest.raises(B.EvlnError) as e:
        B.evlnStepWorkspaceSize(handle, p)
    assert e.value.status == B.EVLN_NOT_SUPPORTED
    # misaligned pointer, null pointer, short workspace
    p = B.step_params("bf16", 28, 4, 128, 10, 5, 100, 1e6)
    buf = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda:0")
    base = buf.data_ptr()
    with pytest.raises(B.EvlnError) as e:
        B.evlnRopeAppend(handle, p, base + 2, base, base, base, base, base, strides=(28 * 128, 512, 512))
    assert e.value.status == B.EVLN_INVALID_VALUE
    with pytest.raises(B.EvlnError) as e:
        B.evlnRopeAppend(handle, p, None, base, base, base, base, base, strides=(28 * 128, 512, 512))
    assert e.value.status == B.EVLN_INVALID_VALUE
    with pytest.raises(B.EvlnError) as e:
        B.evlnStepAttention(handle, p, base, base, base, base, workspace_bytes=64)
    assert e.value.status == B.EVLN_WORKSPACE_TOO_SMALL
    # n = 0 is a no-op
    p0 = B.step_params("bf16", 28, 4, 128, 10, 0, 100, 1e6)
    B.evlnRopeAppend(handle, p0, base, base, base, base, base, base, strides=(28 * 128, 512, 512))
    assert B.evlnGetDeviceStatus(handle) == 0
