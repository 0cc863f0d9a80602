"""CPU pins of the action-isolating mask oracle (packed training sequences, Sec. 3.3)."""
import numpy as np

from oracle import packed_mask_oracle as pm
from oracle import step_oracle as so

THETA = 1.0e4
I, F, A, N = 5, 6, 3, 4
Hq, Hkv, D = 4, 2, 64


def _seq(seed=0):
    rng = np.random.default_rng(seed)
    T = I + N * (F + A)
    return rng.standard_normal((T, Hq, D)), rng.standard_normal((T, Hkv, D)), rng.standard_normal((T, Hkv, D))


def test_mask_structure():
    kind, frame, pos = pm.packed_layout(I, F, A, N)
    mask = pm.action_isolating_mask(kind, frame)
    T = len(kind)
    assert T == I + N * (F + A)
    assert not np.triu(mask, 1).any()                       # never the future
    vis = np.where(kind == 1)[0]
    act = np.where(kind == 2)[0]
    assert not mask[np.ix_(vis, act)].any()                 # visual rows never see an action token
    for i in act:                                           # action rows: own chunk prefix only
        seen = act[mask[i, act]]
        assert all(frame[j] == frame[i] and j <= i for j in seen) and i in seen
        # instruction and the visual history up to v_t, in full
        hist = np.where((kind != 2) & (np.arange(T) < i))[0]
        assert mask[i, hist].all()
    # positions: visual stream contiguous, chunk t continues after v_t
    assert list(pos[kind != 2]) == list(range(I + N * F))
    for t in range(N):
        assert list(pos[(kind == 2) & (frame == t)]) == list(range(I + (t + 1) * F, I + (t + 1) * F + A))
    # rows sum to one under the mask
    q, k, v = _seq()
    out, lse = pm.masked_attention(q, k, np.ones_like(v), mask, pos, THETA)
    assert np.allclose(out, 1.0, atol=1e-12)


def test_masked_rope_is_the_step_oracles_rope():
    q, k, v = _seq(1)
    kind, frame, pos = pm.packed_layout(I, F, A, N)
    vis = kind != 2
    assert np.allclose(pm.rope_at(k[vis], pos[vis], THETA), so.rope(np.ascontiguousarray(k[vis]), 0, THETA), atol=1e-12)


def test_packed_sequence_equals_parallel_single_step_examples():
    # Sec. 3.3: "a packed sequence is akin to M parallel single-step training examples sharing the
    # same sequence prefix".  The streaming loop of Sec. 3.2 -- frame step on the reused cache, then
    # the action chunk as a step whose keys are dropped again -- gives every row of the masked output.
    q, k, v = _seq(2)
    kind, frame, pos = pm.packed_layout(I, F, A, N)
    mask = pm.action_isolating_mask(kind, frame)
    ref_out, ref_lse = pm.masked_attention(q, k, v, mask, pos, THETA)
    cap = I + N * F + A
    kc, vc = np.zeros((cap, Hkv, D)), np.zeros((cap, Hkv, D))
    idx_i = np.where(kind == 0)[0]
    r = so.step(q[idx_i], k[idx_i], v[idx_i], kc, vc, 0, THETA)
    assert np.allclose(r["out"], ref_out[idx_i], atol=1e-11)
    L = I
    for t in range(N):
        iv = np.where((kind == 1) & (frame == t))[0]
        ia = np.where((kind == 2) & (frame == t))[0]
        r = so.step(q[iv], k[iv], v[iv], kc, vc, L, THETA)            # the frame: appended for good
        assert np.allclose(r["out"], ref_out[iv], atol=1e-11) and np.allclose(r["lse"], ref_lse[iv], atol=1e-11)
        L += F
        r = so.step(q[ia], k[ia], v[ia], kc, vc, L, THETA)            # its action chunk: L does not advance
        assert np.allclose(r["out"], ref_out[ia], atol=1e-11) and np.allclose(r["lse"], ref_lse[ia], atol=1e-11)


def test_plain_causal_mask_would_leak_earlier_actions():
    # the same sequence under a plain causal mask differs on every row that follows an action chunk
    q, k, v = _seq(3)
    kind, frame, pos = pm.packed_layout(I, F, A, N)
    iso, _ = pm.masked_attention(q, k, v, pm.action_isolating_mask(kind, frame), pos, THETA)
    causal, _ = pm.masked_attention(q, k, v, np.tril(np.ones((len(kind),) * 2, dtype=bool)), pos, THETA)
    later = np.arange(len(kind)) >= I + F + A
    assert np.abs(iso[later] - causal[later]).max() > 1e-3
    assert np.allclose(iso[: I + F], causal[: I + F], atol=1e-12)
