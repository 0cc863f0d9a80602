"""GPU parity of the paged batch path (evlnPaged*) against the oracle's paged wrapper."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import step_oracle as so
from paper_2512_10310_b200 import binding as B
from paper_2512_10310_b200 import workloads as W
from tests.helpers import bf16_ulp_distance, check_output, f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def handle():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    h = B.evlnCreate(0)
    yield h
    B.evlnDestroy(h)


def _gpu_paged(handle, cfg, x, kv_chunk_tiles=0, with_table=False):
    dev = "cuda:0"
    Bn, P = len(x["cache_lens"]), cfg.page_size
    Hq, Hkv, D = cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim
    max_pages = max(len(t) for t in x["page_table"]) + 3
    table = torch.full((Bn, max_pages), -1, dtype=torch.int32)
    for b, t in enumerate(x["page_table"]):
        table[b, :len(t)] = torch.tensor(t, dtype=torch.int32)
    table = table.clamp(min=0).to(dev)
    # pool layout [pages, Hkv, P, D]; every slot that holds no token starts as NaN so that any
    # leak of an unwritten slot into the result is caught
    k_pool = torch.full((x["num_pages"], Hkv, P, D), float("nan"), dtype=torch.bfloat16, device=dev)
    v_pool = torch.full((x["num_pages"], Hkv, P, D), float("nan"), dtype=torch.bfloat16, device=dev)
    for b, L in enumerate(x["cache_lens"]):
        for pi in range((L + P - 1) // P):
            pg = x["page_table"][b][pi]
            cnt = min(P, L - pi * P)
            k_pool[pg, :, :cnt] = x["k_pool"][pg, :cnt].to(dev).permute(1, 0, 2)
            v_pool[pg, :, :cnt] = x["v_pool"][pg, :cnt].to(dev).permute(1, 0, 2)
    lens, offs = x["cache_lens"], x["new_offsets"]
    rope = {}
    if with_table:
        # one table for positions 0 .. the longest episode, as a serving host would keep
        count = max(L + offs[b + 1] - offs[b] for b, L in enumerate(lens))
        tbl = torch.empty(B.evlnRopeTableBytes(D, count), dtype=torch.uint8, device=dev)
        B.evlnRopeTable(handle, D, cfg.rope_theta, 0, count, tbl)
        rope = dict(rope_table=tbl, rope_table_first_pos=0, rope_table_count=count)
    p = B.paged_params(Hq, Hkv, D, Bn, P, x["num_pages"], max_pages, cfg.rope_theta, kv_chunk_tiles=kv_chunk_tiles, **rope)
    total = offs[-1]
    q, k, v = (x[s].to(dev) for s in ("q_new", "k_new", "v_new"))
    q_rot = torch.empty(total * Hq * D * 2 + 256, dtype=torch.uint8, device=dev)
    ws = torch.empty(B.evlnPagedWorkspaceSize(handle, p, lens, offs), dtype=torch.uint8, device=dev)
    out = torch.full((total, Hq, D), float("nan"), dtype=torch.bfloat16, device=dev)
    lse = torch.full((total, Hq), float("nan"), dtype=torch.float32, device=dev)
    B.evlnPagedRopeAppend(handle, p, q, k, v, lens, offs, table, q_rot, k_pool, v_pool)
    B.evlnPagedStepAttention(handle, p, q_rot, k_pool, v_pool, lens, offs, table, ws)
    B.evlnPagedStepCombine(handle, p, ws, lens, offs, out, lse)
    assert B.evlnGetDeviceStatus(handle) == 0
    return out, lse, k_pool, v_pool


def _check_pools(x, cfg, k_pool, v_pool, ok_pool, ov_pool):
    P = cfg.page_size
    for b, L in enumerate(x["cache_lens"]):
        n = x["new_offsets"][b + 1] - x["new_offsets"][b]
        for t in list(range(L, L + n)):
            pg, sl = x["page_table"][b][t // P], t % P
            assert bf16_ulp_distance(k_pool[pg, :, sl], ok_pool[pg, sl]).max() <= 1
            assert np.array_equal(f64(v_pool[pg, :, sl]), ov_pool[pg, sl])
        # value slots behind the last appended token of the last page are cleared (an episode that
        # appends nothing this step is not touched, and nothing of it is read)
        last = L + n
        if n > 0 and last % P:
            pg = x["page_table"][b][last // P]
            assert bool((v_pool[pg, :, last % P:] == 0).all())


def test_paged_small_ragged_batch(handle):
    cfg = dataclasses.replace(W.PAGED_B16, name="paged_small", batch=5, seed=31)
    lens = [0, 63, 64, 333, 1000]
    news = [70, 1, 129, 37, 196]
    x = W.make_paged_inputs(cfg, lens=lens, num_new=news)
    for chunk in (0, 2):
        out, lse, k_pool, v_pool = _gpu_paged(handle, cfg, x, kv_chunk_tiles=chunk)
        okp, ovp = f64(x["k_pool"]), f64(x["v_pool"])
        ref_out, ref_lse = so.step_paged(f64(x["q_new"]), f64(x["k_new"]), f64(x["v_new"]), okp, ovp,
                                         x["page_table"], lens, x["new_offsets"], cfg.rope_theta, storage="bf16")
        check_output("bf16", out, lse, ref_out, ref_lse)
        _check_pools(x, cfg, k_pool, v_pool, okp, ovp)


def test_paged_position_table_gives_the_same_bits(handle):
    # few tokens (threads read the table themselves) and many (through shared memory), against the
    # kernel's own trigonometry: identical pools and outputs; a table that stops short is refused
    for lens, news in (([0, 63, 64, 333, 1000], [70, 1, 129, 37, 196]), ([300, 2000, 1234, 77], [196, 196, 150, 64])):
        cfg = dataclasses.replace(W.PAGED_B16, name="paged_table", batch=len(lens), seed=35)
        x = W.make_paged_inputs(cfg, lens=lens, num_new=news)
        a = _gpu_paged(handle, cfg, x)
        b = _gpu_paged(handle, cfg, x, with_table=True)
        # what the append kernel wrote: bit for bit (slots never written hold NaN in both)
        for u, v in zip(a[2:], b[2:]):
            assert torch.equal(torch.nan_to_num(u.float(), nan=-7.0), torch.nan_to_num(v.float(), nan=-7.0))
        # the attention over identical pools: the same up to the order in which a build with a tiny
        # reference headroom happens to move its references
        assert torch.allclose(a[0].float(), b[0].float(), rtol=2e-2, atol=1e-4)
        assert torch.allclose(a[1], b[1], rtol=0, atol=1e-3)
    D = cfg.head_dim
    tbl = torch.empty(B.evlnRopeTableBytes(D, 100), dtype=torch.uint8, device="cuda:0")
    p = B.paged_params(cfg.num_q_heads, cfg.num_kv_heads, D, 1, cfg.page_size, 8, 8, cfg.rope_theta,
                       rope_table=tbl, rope_table_first_pos=0, rope_table_count=100)
    with pytest.raises(B.EvlnError) as e:
        B.evlnPagedWorkspaceSize(handle, p, [90], [0, 20])          # positions 90..109, table ends at 99
    assert e.value.status == B.EVLN_INVALID_VALUE


def test_paged_equals_contiguous_on_device(handle):
    # the same episode through the contiguous entry points gives the same bits up to split order
    cfg = dataclasses.replace(W.PAGED_B16, name="paged_vs_contig", batch=1, seed=32)
    x = W.make_paged_inputs(cfg, lens=[777], num_new=[150])
    out, lse, _, _ = _gpu_paged(handle, cfg, x)
    from tests.helpers import GpuStep
    gs = GpuStep(handle, "bf16", cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, 777 + 150, cfg.rope_theta, 150)
    P = cfg.page_size
    kc = torch.cat([x["k_pool"][pg] for pg in x["page_table"][0]])[:777]
    vc = torch.cat([x["v_pool"][pg] for pg in x["page_table"][0]])[:777]
    gs.load_cache(kc, vc)
    g = gs.step(777, x["q_new"], x["k_new"], x["v_new"])
    assert (g["out"].float() - out.float()).abs().max().item() <= 2e-4
    assert (g["lse"] - lse).abs().max().item() <= 1e-5


def test_paged_b16_full_size_all_rows(handle):
    # the full serving batch (16 episodes, L from 1024 to 16384, 196 new tokens each): every output row,
    # every log-sum-exp and every appended slot against the oracle
    cfg = W.PAGED_B16
    x = W.make_paged_inputs(cfg)
    out, lse, k_pool, v_pool = _gpu_paged(handle, cfg, x)
    okp, ovp = f64(x["k_pool"]), f64(x["v_pool"])
    ref_out, ref_lse = so.step_paged(f64(x["q_new"]), f64(x["k_new"]), f64(x["v_new"]), okp, ovp,
                                     x["page_table"], x["cache_lens"], x["new_offsets"], cfg.rope_theta, storage="bf16")
    check_output("bf16", out, lse, ref_out, ref_lse)
    _check_pools(x, cfg, k_pool, v_pool, okp, ovp)
    # ... and episode by episode, so that a short episode cannot hide behind the long ones' norm
    for b in range(cfg.batch):
        lo, hi = x["new_offsets"][b], x["new_offsets"][b + 1]
        check_output("bf16", out[lo:hi], lse[lo:hi], ref_out[lo:hi], ref_lse[lo:hi])


def test_paged_episodes_without_new_tokens(handle):
    # episodes that contribute no token this step: first, in the middle and last of the batch
    cfg = dataclasses.replace(W.PAGED_B16, name="paged_idle", batch=6, seed=33)
    lens = [500, 130, 64, 900, 257, 300]
    news = [0, 70, 0, 196, 129, 0]
    x = W.make_paged_inputs(cfg, lens=lens, num_new=news)
    for chunk in (0, 3):
        out, lse, k_pool, v_pool = _gpu_paged(handle, cfg, x, kv_chunk_tiles=chunk)
        okp, ovp = f64(x["k_pool"]), f64(x["v_pool"])
        ref_out, ref_lse = so.step_paged(f64(x["q_new"]), f64(x["k_new"]), f64(x["v_new"]), okp, ovp,
                                         x["page_table"], lens, x["new_offsets"], cfg.rope_theta, storage="bf16")
        check_output("bf16", out, lse, ref_out, ref_lse)
        _check_pools(x, cfg, k_pool, v_pool, okp, ovp)


def test_page_table_check_accepts_the_workload_and_names_a_bad_entry(handle):
    cfg = dataclasses.replace(W.PAGED_B16, name="paged_check", batch=3, seed=34)
    x = W.make_paged_inputs(cfg, lens=[100, 700, 64], num_new=[30, 196, 1])
    max_pages = max(len(t) for t in x["page_table"]) + 2
    p = B.paged_params(cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, 3, cfg.page_size, x["num_pages"], max_pages,
                       cfg.rope_theta)
    rows = [t + [0] * (max_pages - len(t)) for t in x["page_table"]]      # padding entries are not looked at
    assert B.evlnPagedCheckTable(p, x["cache_lens"], x["new_offsets"], rows) == (B.EVLN_OK, -1, -1)
    bad = [list(r) for r in rows]
    bad[1][3] = bad[0][1]                      # a page of episode 0 handed to episode 1 as well
    assert B.evlnPagedCheckTable(p, x["cache_lens"], x["new_offsets"], bad) == (B.EVLN_INVALID_VALUE, 1, 3)
    bad = [list(r) for r in rows]
    bad[2][0] = x["num_pages"]                 # outside the pool
    assert B.evlnPagedCheckTable(p, x["cache_lens"], x["new_offsets"], bad) == (B.EVLN_INVALID_VALUE, 2, 0)


def test_paged_argument_errors(handle):
    p = B.paged_params(28, 4, 128, 2, 64, 10, 2, 1e6)
    with pytest.raises(B.EvlnError) as e:
        B.evlnPagedWorkspaceSize(handle, p, [100, 100], [0, 10, 60])   # second episode needs 3 pages
    assert e.value.status == B.EVLN_CACHE_FULL
    p = B.paged_params(28, 4, 128, 2, 32, 10, 8, 1e6)
    with pytest.raises(B.EvlnError) as e:
        B.evlnPagedWorkspaceSize(handle, p, [100, 100], [0, 10, 20])
    assert e.value.status == B.EVLN_NOT_SUPPORTED
