"""Pins of the fp64 CPU oracle against what the mathematics fixes (CPU only).

Each test is chosen so that a plausible slip in ``oracle/evln_oracle.c`` (a wrong sign of
the sine term, interleaved instead of half-split pairing, an off-by-one in the position or
the causal bound, a transposed operand, a missing scale, a wrong kv-head mapping) fails it.
"""
import math

import numpy as np
import pytest
import torch

from oracle import prefill_bruteforce as bf
from oracle import step_oracle as so

RNG = np.random.default_rng(1234)


def _rand(*shape):
    return RNG.standard_normal(shape)


# --------------------------------------------------------------------------- RoPE

def test_rope_position_zero_is_identity():
    x = _rand(1, 3, 16)
    assert np.array_equal(so.rope(x, 0, 1e4), x)


def test_rope_d2_closed_form():
    # D=2: one pair, omega_0 = 1: (1,0) at position p -> (cos p, sin p)
    for p in (1, 2, 7, 1000):
        y = so.rope(np.array([[[1.0, 0.0]]]), p, 123.0)
        assert y[0, 0, 0] == pytest.approx(math.cos(p), abs=1e-15)
        assert y[0, 0, 1] == pytest.approx(math.sin(p), abs=1e-15)


def test_rope_d4_hand_worked_half_split():
    # x=(1,2,3,4), theta=100, D=4: omega = (1, 100^(-1/2)) = (1, 0.1); pairs are (x0,x2), (x1,x3)
    p = 3
    y = so.rope(np.array([[[1.0, 2.0, 3.0, 4.0]]]), p, 100.0)[0, 0]
    a0, a1 = p * 1.0, p * 0.1
    exp = [1 * math.cos(a0) - 3 * math.sin(a0),
           2 * math.cos(a1) - 4 * math.sin(a1),
           3 * math.cos(a0) + 1 * math.sin(a0),
           4 * math.cos(a1) + 2 * math.sin(a1)]
    assert np.allclose(y, exp, atol=1e-14, rtol=0)


def test_rope_second_token_uses_next_position():
    x = _rand(3, 2, 8)
    y = so.rope(x, 10, 1e4)
    for i in range(3):
        assert np.array_equal(y[i:i + 1], so.rope(x[i:i + 1], 10 + i, 1e4))


def test_rope_preserves_pair_norms():
    x = _rand(5, 2, 32)
    y = so.rope(x, 77, 1e6)
    h = 16
    assert np.allclose(x[..., :h] ** 2 + x[..., h:] ** 2, y[..., :h] ** 2 + y[..., h:] ** 2,
                       rtol=1e-14, atol=1e-15)


def test_rope_relative_position_invariance():
    # <R(p)q, R(t)k> depends on p - t only: shifting every position leaves scores unchanged
    q, k = _rand(6, 1, 32), _rand(6, 1, 32)
    s0 = np.einsum("ihd,thd->it", so.rope(q, 0, 1e4), so.rope(k, 0, 1e4))
    for shift in (1, 17, 4096):
        s1 = np.einsum("ihd,thd->it", so.rope(q, shift, 1e4), so.rope(k, shift, 1e4))
        assert np.allclose(s0, s1, atol=1e-9, rtol=0)


def test_rope_matches_library_rotate_half():
    mod = pytest.importorskip("transformers.models.llama.modeling_llama")
    T, H, D, theta = 9, 2, 16, 1e4
    x = _rand(T, H, D)
    inv = 1.0 / (theta ** (torch.arange(0, D, 2, dtype=torch.float64) / D))
    ang = torch.arange(5, 5 + T, dtype=torch.float64)[:, None] * inv[None]
    emb = torch.cat([ang, ang], dim=-1)                                  # [T, D]
    xt = torch.from_numpy(x).permute(1, 0, 2)[None]                      # [1,H,T,D]
    yq, _ = mod.apply_rotary_pos_emb(xt, xt, emb.cos()[None], emb.sin()[None])
    assert np.allclose(so.rope(x, 5, theta), yq[0].permute(1, 0, 2).numpy(), atol=1e-13, rtol=0)


# --------------------------------------------------------------------------- bf16 rounding

def test_bf16_rounding_matches_library_conversion():
    x = torch.randn(20000, generator=torch.Generator().manual_seed(0), dtype=torch.float32)
    x = torch.cat([x, x * 1e-30, x * 1e30, torch.tensor([0.0, -0.0, 1e-45, 3.38e38, 3.4e38])])
    lib = x.to(torch.bfloat16).to(torch.float64).numpy()
    got = so.round_bf16(x.to(torch.float64).numpy())
    assert np.array_equal(lib, got)


def test_bf16_rounding_ties_to_even_and_no_double_rounding():
    u = 2.0 ** -7          # spacing of bf16 in [1, 2)
    assert so.round_bf16([1 + u / 2])[0] == 1.0              # tie -> even (mantissa 0)
    assert so.round_bf16([1 + 3 * u / 2])[0] == 1 + 2 * u    # tie -> even (mantissa 2)
    # just above a tie by less than a float32 ulp: rounding through float32 first would
    # land on the tie and then go down; the direct rounding must go up
    assert so.round_bf16([1 + u / 2 + 2.0 ** -40])[0] == 1 + u


# --------------------------------------------------------------------------- attention

def _chain(q, k, v, chunks, theta, Hkv, D):
    """Run the step oracle chunk by chunk with a reused cache."""
    T = q.shape[0]
    kc, vc = np.zeros((T, Hkv, D)), np.zeros((T, Hkv, D))
    outs, lses, L = [], [], 0
    for n in chunks:
        r = so.step(q[L:L + n], k[L:L + n], v[L:L + n], kc, vc, L, theta)
        outs.append(r["out"])
        lses.append(r["lse"])
        L += n
    return np.concatenate(outs), np.concatenate(lses), kc, vc


@pytest.mark.parametrize("Hq,Hkv,D,chunks", [(2, 1, 8, [5, 3, 3, 1]), (4, 2, 16, [7, 4, 6]),
                                             (6, 2, 4, [1, 1, 1, 9])])
def test_incremental_steps_equal_bruteforce_full_prefill(Hq, Hkv, D, chunks):
    T, theta = sum(chunks), 1e4
    q, k, v = _rand(T, Hq, D), _rand(T, Hkv, D), _rand(T, Hkv, D)
    out, lse, kc, vc = _chain(q, k, v, chunks, theta, Hkv, D)
    ref_out, ref_lse, _ = bf.full_prefill(q, k, v, theta)
    assert np.allclose(out, ref_out, atol=1e-12, rtol=0)
    assert np.allclose(lse, ref_lse, atol=1e-12, rtol=0)
    assert np.allclose(kc, bf.rope_all(k, theta), atol=1e-13, rtol=0)
    assert np.array_equal(vc, v)


def test_step_matches_library_sdpa():
    Hq, Hkv, D, L, n, theta = 4, 2, 16, 11, 6, 1e4
    G = Hq // Hkv
    kc, vc = np.zeros((L + n, Hkv, D)), np.zeros((L + n, Hkv, D))
    kc[:L], vc[:L] = _rand(L, Hkv, D), _rand(L, Hkv, D)
    q, k, v = _rand(n, Hq, D), _rand(n, Hkv, D), _rand(n, Hkv, D)
    r = so.step(q, k, v, kc, vc, L, theta)
    # library attention on the oracle's own rotated q and the cache it produced
    Q = torch.from_numpy(r["q_rot"]).permute(1, 0, 2)[None]
    K = torch.from_numpy(np.repeat(kc, G, axis=1)).permute(1, 0, 2)[None]
    V = torch.from_numpy(np.repeat(vc, G, axis=1)).permute(1, 0, 2)[None]
    mask = torch.arange(L + n)[None, :] <= (L + torch.arange(n))[:, None]
    ref = torch.nn.functional.scaled_dot_product_attention(Q, K, V, attn_mask=mask)
    assert np.allclose(r["out"], ref[0].permute(1, 0, 2).numpy(), atol=1e-12, rtol=0)
    # and the rotated q/k used are the RoPE of the inputs at L..L+n-1
    assert np.array_equal(r["q_rot"], so.rope(q, L, theta))
    assert np.array_equal(kc[L:], so.rope(k, L, theta))


def test_softmax_rows_sum_to_one_and_respect_causal_bound():
    Hq, Hkv, D, L, n = 2, 1, 8, 5, 4
    kc, vc = _rand(L + n, Hkv, D), _rand(L + n, Hkv, D)
    r = so.step(_rand(n, Hq, D), _rand(n, Hkv, D), _rand(n, Hkv, D), kc, vc, L, 1e4,
                want_probs=True)
    p = r["probs"]
    assert np.allclose(p.sum(-1), 1.0, atol=1e-14)
    for i in range(n):
        assert np.all(p[i, :, L + i + 1:] == 0.0)
        assert np.all(p[i, :, :L + i + 1] > 0.0)


def test_zero_queries_give_running_mean_of_values_and_known_lse():
    Hq, Hkv, D, L, n = 2, 2, 4, 3, 5
    kc, vc = _rand(L + n, Hkv, D), _rand(L + n, Hkv, D)
    v = _rand(n, Hkv, D)
    r = so.step(np.zeros((n, Hq, D)), _rand(n, Hkv, D), v, kc, vc, L, 1e4)
    for i in range(n):
        assert np.allclose(r["out"][i], vc[:L + i + 1].mean(axis=0), atol=1e-14)
        assert np.allclose(r["lse"][i], math.log(L + i + 1), atol=1e-14)


def test_constant_values_give_that_constant():
    Hq, Hkv, D, L, n = 2, 1, 8, 6, 3
    kc, vc = _rand(L + n, Hkv, D), np.full((L + n, Hkv, D), 2.5)
    r = so.step(_rand(n, Hq, D), _rand(n, Hkv, D), np.full((n, Hkv, D), 2.5), kc, vc, L, 1e4)
    assert np.allclose(r["out"], 2.5, atol=1e-14)


def test_scale_default_and_explicit():
    Hq, Hkv, D, L, n = 1, 1, 16, 4, 2
    base = [_rand(n, Hq, D), _rand(n, Hkv, D), _rand(n, Hkv, D)]
    c0 = _rand(L + n, Hkv, D), _rand(L + n, Hkv, D)
    a = so.step(*base, c0[0].copy(), c0[1].copy(), L, 1e4)
    b = so.step(*base, c0[0].copy(), c0[1].copy(), L, 1e4, scale=0.25)   # 1/sqrt(16)
    c = so.step(*base, c0[0].copy(), c0[1].copy(), L, 1e4, scale=1.0)
    assert np.array_equal(a["out"], b["out"])
    assert not np.allclose(a["out"], c["out"])
    # one query, two keys, scale 1: softmax weights are a logistic of the logit difference
    q = np.zeros((1, 1, 2)); q[0, 0, 0] = 1.0
    kc2 = np.array([[[2.0, 0.0]], [[0.0, 0.0]]]); vc2 = np.array([[[1.0, 0.0]], [[0.0, 0.0]]])
    # cached key at position 0 (unrotated by construction), new key = zeros -> logit 0
    r = so.step(q * 0 + np.array([[[1.0, 0.0]]]), np.zeros((1, 1, 2)), np.array([[[0.0, 1.0]]]),
                kc2, vc2, 1, 1e4, scale=1.0)
    # query rotated at position 1: (cos 1, sin 1); logits: 2 cos 1 and 0
    w = 1.0 / (1.0 + math.exp(-2.0 * math.cos(1.0)))
    assert np.allclose(r["out"][0, 0], [w, 1 - w], atol=1e-14)


def test_future_slots_do_not_matter():
    Hq, Hkv, D, L, n = 2, 1, 8, 4, 3
    args = [_rand(n, Hq, D), _rand(n, Hkv, D), _rand(n, Hkv, D)]
    kc, vc = _rand(L + n + 5, Hkv, D), _rand(L + n + 5, Hkv, D)
    kc2, vc2 = kc.copy(), vc.copy()
    tail = kc[L + n:].copy()
    kc2[L + n:] += 100.0
    vc2[L + n:] -= 100.0
    a = so.step(*args, kc, vc, L, 1e4)
    b = so.step(*args, kc2, vc2, L, 1e4)
    assert np.array_equal(a["out"], b["out"])
    # row i must not see new token i+1: change the last new token only
    args2 = [args[0], args[1].copy(), args[2].copy()]
    args2[1][-1] += 3.0
    args2[2][-1] += 3.0
    c = so.step(*args2, kc.copy(), vc.copy(), L, 1e4)
    assert np.array_equal(a["out"][:-1], c["out"][:-1])
    assert not np.allclose(a["out"][-1], c["out"][-1])
    # untouched slots stay untouched
    assert np.array_equal(kc[L + n:], tail) and np.array_equal(kc2[L + n:], tail + 100.0)


def test_gqa_equals_mha_with_replicated_kv_heads():
    Hq, Hkv, D, L, n = 6, 2, 8, 5, 4
    G = Hq // Hkv
    q, k, v = _rand(n, Hq, D), _rand(n, Hkv, D), _rand(n, Hkv, D)
    kc, vc = _rand(L + n, Hkv, D), _rand(L + n, Hkv, D)
    a = so.step(q, k, v, kc.copy(), vc.copy(), L, 1e4)
    rep = lambda x: np.ascontiguousarray(np.repeat(x, G, axis=1))
    b = so.step(q, rep(k), rep(v), rep(kc), rep(vc), L, 1e4)
    assert np.array_equal(a["out"], b["out"])


def test_split_merge_equals_unsplit():
    Hq, Hkv, D, L, n = 2, 1, 8, 20, 6
    kc, vc = _rand(L + n, Hkv, D), _rand(L + n, Hkv, D)
    r = so.step(_rand(n, Hq, D), _rand(n, Hkv, D), _rand(n, Hkv, D), kc, vc, L, 1e4)
    for cuts in ([0, 26], [0, 7, 26], [0, 3, 21, 23, 26], [0, 25, 26, 40]):
        parts = [so.attend_range(r["q_rot"], kc, vc, L, a, b) for a, b in zip(cuts[:-1], cuts[1:])]
        o = np.stack([p[0].reshape(n * Hq, D) for p in parts])
        l = np.stack([p[1].reshape(n * Hq) for p in parts])
        out, lse = so.combine(o, l)
        assert np.allclose(out.reshape(n, Hq, D), r["out"], atol=1e-12, rtol=0)
        assert np.allclose(lse.reshape(n, Hq), r["lse"], atol=1e-12, rtol=0)


def test_combine_two_way_closed_form_and_empty_split():
    # two splits with lse difference d: weights are 1/(1+e^-d) and its complement
    o = np.array([[[1.0, 0.0]], [[0.0, 1.0]]]); l = np.array([[0.3], [-0.9]])
    out, lse = so.combine(o, l)
    w = 1.0 / (1.0 + math.exp(-1.2))
    assert np.allclose(out[0], [w, 1 - w], atol=1e-15)
    assert lse[0] == pytest.approx(math.log(math.exp(0.3) + math.exp(-0.9)), abs=1e-15)
    out, lse = so.combine(np.array([[[4.0, 5.0]], [[9.0, 9.0]]]), np.array([[0.1], [-np.inf]]))
    assert np.array_equal(out[0], [4.0, 5.0]) and lse[0] == pytest.approx(0.1)


def test_storage_rounding_applies_to_keys_only():
    Hq, Hkv, D, L, n = 2, 1, 8, 3, 4
    tb = lambda x: torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy()
    q, k, v = tb(_rand(n, Hq, D)), tb(_rand(n, Hkv, D)), tb(_rand(n, Hkv, D))
    kc, vc = tb(_rand(L + n, Hkv, D)), tb(_rand(L + n, Hkv, D))
    kc_exact = kc.copy()
    so.step(q, k, v, kc_exact, vc.copy(), L, 1e6)
    r = so.step(q, k, v, kc, vc, L, 1e6, storage="bf16")
    assert np.array_equal(kc[L:], so.round_bf16(kc_exact[L:]))
    assert np.array_equal(vc[L:], v)
    # the attention consumed the rounded keys
    chk = so.attend_range(r["q_rot"], kc, vc, L, 0, L + n)
    assert np.allclose(chk[0], r["out"], atol=1e-13)


def test_paged_equals_contiguous_under_any_page_permutation():
    Hq, Hkv, D, P = 2, 1, 8, 4
    lens, news = [5, 9], [3, 6]
    offs = [0, 3, 9]
    q, k, v = _rand(9, Hq, D), _rand(9, Hkv, D), _rand(9, Hkv, D)
    caches = [(_rand(L, Hkv, D), _rand(L, Hkv, D)) for L in lens]
    ref = []
    for b, (L, n) in enumerate(zip(lens, news)):
        kc, vc = np.zeros((L + n, Hkv, D)), np.zeros((L + n, Hkv, D))
        kc[:L], vc[:L] = caches[b]
        ref.append(so.step(q[offs[b]:offs[b + 1]], k[offs[b]:offs[b + 1]], v[offs[b]:offs[b + 1]],
                           kc, vc, L, 1e4)["out"])
    ref = np.concatenate(ref)
    for tables in ([[0, 1], [2, 3, 4, 5]], [[5, 2], [4, 0, 3, 1]]):
        kp, vp = np.zeros((6, P, Hkv, D)), np.zeros((6, P, Hkv, D))
        for b, L in enumerate(lens):
            for t in range(L):
                kp[tables[b][t // P], t % P] = caches[b][0][t]
                vp[tables[b][t // P], t % P] = caches[b][1][t]
        out, _ = so.step_paged(q, k, v, kp, vp, tables, lens, offs, 1e4)
        assert np.array_equal(out, ref)


def test_cache_overflow_is_rejected():
    with pytest.raises(ValueError):
        so.step(_rand(3, 1, 4), _rand(3, 1, 4), _rand(3, 1, 4), np.zeros((4, 1, 4)),
                np.zeros((4, 1, 4)), 2, 1e4)
