"""GPU parity of the un-rotated store path (evlnStoreAppend / evlnSampleFrames / evlnGatherRope
followed by the usual step) against the re-indexing oracle."""
import numpy as np
import pytest
import torch

from oracle import reindex_oracle as ro
from paper_2512_10310_b200 import binding as B
from tests.helpers import GpuStep, bf16_ulp_distance, check_output, f64

pytestmark = pytest.mark.gpu

Hq, Hkv, D, THETA = 28, 4, 128, 1.0e6
I_LEN, F_TOK = 256, 196            # instruction tokens, tokens per frame


@pytest.fixture(scope="module")
def handle():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    h = B.evlnCreate(0)
    yield h
    B.evlnDestroy(h)


def _draw(gen, shape, scale=128.0 ** -0.5):
    return (torch.randn(shape, generator=gen, dtype=torch.float32) * scale).to(torch.bfloat16)


def test_sampler_matches_the_oracle(handle):
    for n in (0, 1, 5, 16, 17, 31, 100, 333):
        for budget in (1, 4, 16):
            assert B.evlnSampleFrames(B.EVLN_SAMPLE_UNIFORM, n, budget) == ro.sample_uniform(n, budget)
            for stride in (1, 4):
                assert B.evlnSampleFrames(B.EVLN_SAMPLE_SLIDING, n, budget, stride) == ro.sample_sliding(n, budget, stride)


def test_gather_rope_against_oracle(handle):
    gen = torch.Generator().manual_seed(41)
    slots, work_cap = 3000, 1700
    k_raw, v_raw = _draw(gen, (slots, Hkv, D)), _draw(gen, (slots, Hkv, D))
    dev = "cuda:0"
    k_store = k_raw.to(dev).permute(1, 0, 2).contiguous()
    v_store = v_raw.to(dev).permute(1, 0, 2).contiguous()
    k_work = torch.full((Hkv, work_cap, D), 7.0, dtype=torch.bfloat16, device=dev)
    v_work = torch.full((Hkv, work_cap, D), -3.0, dtype=torch.bfloat16, device=dev)
    segs = [(0, 256), (452, 196), (1040, 196), (2804, 196), (13, 1), (2999, 1), (700, 0), (100, 333)]
    p = B.gather_params("bf16", Hkv, D, slots, work_cap, THETA)
    total = B.evlnGatherRope(handle, p, [s for s, _ in segs], [l for _, l in segs], k_store, v_store, k_work, v_work)
    torch.cuda.synchronize()
    kw, vw = ro.gather_rope(f64(k_raw), f64(v_raw), segs, THETA, storage="bf16")
    assert total == kw.shape[0] == sum(l for _, l in segs)
    d = bf16_ulp_distance(k_work[:, :total].permute(1, 0, 2), kw)
    assert d.max() <= 1 and (d > 0).mean() < 0.05
    assert np.array_equal(f64(v_work[:, :total].permute(1, 0, 2)), vw)
    assert bool((k_work[:, total:] == 7.0).all()) and bool((v_work[:, total:] == -3.0).all())
    # argument errors launch nothing
    with pytest.raises(B.EvlnError) as e:
        B.evlnGatherRope(handle, p, [2900], [200], k_store, v_store, k_work, v_work)
    assert e.value.status == B.EVLN_INVALID_VALUE
    with pytest.raises(B.EvlnError) as e:
        B.evlnGatherRope(handle, p, [0, 0], [1000, 1000], k_store, v_store, k_work, v_work)
    assert e.value.status == B.EVLN_CACHE_FULL


@pytest.mark.parametrize("sampler,stride", [("uniform", 1), ("sliding", 4)])
def test_sampled_episode_matches_the_oracle(handle, sampler, stride):
    # an episode with an un-rotated store: every step appends the raw frame, samples 8 history
    # frames, lays them out with contiguous ids and attends; the oracle does the same in fp64
    gen = torch.Generator().manual_seed(42 + stride)
    steps, budget = 14, 8
    slots = I_LEN + steps * F_TOK
    work_cap = I_LEN + (budget + 1) * F_TOK
    dev = "cuda:0"
    k_store = torch.zeros((Hkv, slots, D), dtype=torch.bfloat16, device=dev)
    v_store = torch.zeros((Hkv, slots, D), dtype=torch.bfloat16, device=dev)
    k_raw = np.zeros((slots, Hkv, D))
    v_raw = np.zeros((slots, Hkv, D))
    gp = B.gather_params("bf16", Hkv, D, slots, work_cap, THETA)
    gs = GpuStep(handle, "bf16", Hq, Hkv, D, work_cap, THETA, F_TOK)
    # instruction tokens into the store
    ki, vi = _draw(gen, (I_LEN, Hkv, D)), _draw(gen, (I_LEN, Hkv, D))
    B.evlnStoreAppend(handle, gp, ki.to(dev), vi.to(dev), 0, k_store, v_store)
    k_raw[:I_LEN], v_raw[:I_LEN] = f64(ki), f64(vi)
    store_len = I_LEN
    code = B.EVLN_SAMPLE_UNIFORM if sampler == "uniform" else B.EVLN_SAMPLE_SLIDING
    for t in range(steps):
        q, k, v = _draw(gen, (F_TOK, Hq, D)), _draw(gen, (F_TOK, Hkv, D)), _draw(gen, (F_TOK, Hkv, D))
        kept = B.evlnSampleFrames(code, t, budget, stride)
        segs = ro.frame_segments(I_LEN, F_TOK, kept)
        L = B.evlnGatherRope(handle, gp, [s for s, _ in segs], [l for _, l in segs], k_store, v_store,
                             gs.k_cache, gs.v_cache)
        assert L == I_LEN + len(kept) * F_TOK
        g = gs.step(L, q, k, v)
        B.evlnStoreAppend(handle, gp, k.to(dev), v.to(dev), store_len, k_store, v_store)
        if t in (0, 1, 5, steps - 1):
            r = ro.sampled_step(f64(q), f64(k), f64(v), k_raw, v_raw, segs, THETA, storage="bf16")
            check_output("bf16", g["out"], g["lse"], r["out"], r["lse"])
            d = bf16_ulp_distance(gs.k_cache[:, :L + F_TOK].permute(1, 0, 2), r["k_work"])
            assert d.max() <= 1
            assert np.array_equal(f64(gs.v_cache[:, :L + F_TOK].permute(1, 0, 2)), r["v_work"])
        k_raw[store_len:store_len + F_TOK], v_raw[store_len:store_len + F_TOK] = f64(k), f64(v)
        store_len += F_TOK
    # the store holds the raw tokens bit-exactly
    assert np.array_equal(f64(k_store.permute(1, 0, 2)), k_raw)
    assert np.array_equal(f64(v_store.permute(1, 0, 2)), v_raw)


def test_offloaded_store_episode_matches_the_oracle(handle):
    # Sec. 3.2, memory management: the whole raw store lives in pinned host memory; the device store
    # has the instruction + 9 frame slots.  Every step offloads the new frame, fetches the kept
    # frames that are not resident and runs the sampled step; results equal the oracle's, and the
    # uniform sampler moves about half of its budget per step.
    from paper_2512_10310_b200.residency import FrameResidency
    gen = torch.Generator().manual_seed(77)
    steps, budget = 22, 8
    host_slots = I_LEN + steps * F_TOK
    dev_slots = I_LEN + (budget + 1) * F_TOK
    work_cap = I_LEN + (budget + 1) * F_TOK
    dev = "cuda:0"
    h_k = torch.zeros((Hkv, host_slots, D), dtype=torch.bfloat16).pin_memory()
    h_v = torch.zeros((Hkv, host_slots, D), dtype=torch.bfloat16).pin_memory()
    k_store = torch.zeros((Hkv, dev_slots, D), dtype=torch.bfloat16, device=dev)
    v_store = torch.zeros((Hkv, dev_slots, D), dtype=torch.bfloat16, device=dev)
    k_raw = np.zeros((host_slots, Hkv, D))
    v_raw = np.zeros((host_slots, Hkv, D))
    gp = B.gather_params("bf16", Hkv, D, dev_slots, work_cap, THETA)
    gs = GpuStep(handle, "bf16", Hq, Hkv, D, work_cap, THETA, F_TOK)
    res = FrameResidency(budget + 1, I_LEN, F_TOK)
    host_start = lambda f: I_LEN + f * F_TOK
    ki, vi = _draw(gen, (I_LEN, Hkv, D)), _draw(gen, (I_LEN, Hkv, D))
    B.evlnStoreAppend(handle, gp, ki.to(dev), vi.to(dev), 0, k_store, v_store)
    B.evlnStoreOffload(handle, gp, k_store, v_store, 0, I_LEN, h_k, h_v, 0)
    k_raw[:I_LEN], v_raw[:I_LEN] = f64(ki), f64(vi)
    moved = []
    for t in range(steps):
        q, k, v = _draw(gen, (F_TOK, Hq, D)), _draw(gen, (F_TOK, Hkv, D)), _draw(gen, (F_TOK, Hkv, D))
        kept = B.evlnSampleFrames(B.EVLN_SAMPLE_UNIFORM, t, budget)
        fetches, segs = res.plan(kept, host_start)
        for _, src, dst in fetches:
            B.evlnStoreFetch(handle, gp, h_k, h_v, src, F_TOK, k_store, v_store, dst)
        moved.append(len(fetches))
        L = B.evlnGatherRope(handle, gp, [s for s, _ in segs], [l for _, l in segs], k_store, v_store,
                             gs.k_cache, gs.v_cache)
        g = gs.step(L, q, k, v)
        # the new frame: raw K/V into a free device slot if there is one, and to the host store either way
        slot = res.admit(t)
        stage = slot if slot >= 0 else None
        if stage is None:       # every slot holds a kept frame: the raw frame goes to the host through a one-frame buffer
            tmp_k = torch.zeros((Hkv, F_TOK, D), dtype=torch.bfloat16, device=dev)
            tmp_v = torch.zeros_like(tmp_k)
            gp_tmp = B.gather_params("bf16", Hkv, D, F_TOK, work_cap, THETA)
            B.evlnStoreAppend(handle, gp_tmp, k.to(dev), v.to(dev), 0, tmp_k, tmp_v)
            B.evlnStoreOffload(handle, gp_tmp, tmp_k, tmp_v, 0, F_TOK, h_k, h_v, host_start(t))
        else:
            B.evlnStoreAppend(handle, gp, k.to(dev), v.to(dev), stage, k_store, v_store)
            B.evlnStoreOffload(handle, gp, k_store, v_store, stage, F_TOK, h_k, h_v, host_start(t))
        if t in (0, 3, 12, steps - 1):
            o_segs = ro.frame_segments(I_LEN, F_TOK, kept)
            r = ro.sampled_step(f64(q), f64(k), f64(v), k_raw, v_raw, o_segs, THETA, storage="bf16")
            check_output("bf16", g["out"], g["lse"], r["out"], r["lse"])
            assert bf16_ulp_distance(gs.k_cache[:, :L + F_TOK].permute(1, 0, 2), r["k_work"]).max() <= 1
        k_raw[host_start(t):host_start(t) + F_TOK], v_raw[host_start(t):host_start(t) + F_TOK] = f64(k), f64(v)
    torch.cuda.synchronize()
    assert np.array_equal(f64(h_k.permute(1, 0, 2)), k_raw) and np.array_equal(f64(h_v.permute(1, 0, 2)), v_raw)
    # frames admitted on the device need no fetch; later the uniform sampler moves a few per step
    assert max(moved) <= budget and np.mean(moved[budget + 2:]) <= 0.75 * budget
