"""CPU pins of the re-indexing oracle (un-rotated store + frame samplers, Sec. 3.2)."""
import numpy as np
import pytest

from oracle import prefill_bruteforce as pb
from oracle import reindex_oracle as ro
from oracle import step_oracle as so

THETA = 1.0e4


def test_uniform_sampler_closed_forms():
    assert ro.sample_uniform(5, 16) == [0, 1, 2, 3, 4]              # history fits: keep all
    assert ro.sample_uniform(31, 16) == list(range(0, 31, 2))        # exact spacing 2
    assert ro.sample_uniform(4, 1) == [3]
    got = ro.sample_uniform(100, 16)
    assert got[0] == 0 and got[-1] == 99 and len(got) == 16
    assert all(b > a for a, b in zip(got, got[1:]))
    gaps = np.diff(got)
    assert gaps.max() - gaps.min() <= 1                              # evenly spread
    assert ro.sample_uniform(0, 4) == [] and ro.sample_uniform(7, 0) == []


def test_sliding_sampler_closed_forms():
    assert ro.sample_sliding(20, 4, 4) == [7, 11, 15, 19]
    assert ro.sample_sliding(3, 4, 4) == [2]
    assert ro.sample_sliding(10, 3, 1) == [7, 8, 9]
    assert ro.sample_sliding(6, 16, 1) == [0, 1, 2, 3, 4, 5]


def test_segments_moved_per_step_match_the_papers_statement():
    # Sec. 3.2, memory management: a sliding window brings in one new segment per step, uniform
    # sampling about half of the kept ones
    B = 16
    new_sliding, new_uniform = [], []
    for t in range(40, 200):
        a, b = set(ro.sample_sliding(t, B, 1)), set(ro.sample_sliding(t + 1, B, 1))
        new_sliding.append(len(b - a))
        a, b = set(ro.sample_uniform(t, B)), set(ro.sample_uniform(t + 1, B))
        new_uniform.append(len(b - a))
    assert set(new_sliding) == {1}
    assert 0.3 * B <= np.mean(new_uniform) <= 0.7 * B


def test_gather_of_everything_is_plain_rope():
    rng = np.random.default_rng(0)
    k = rng.standard_normal((37, 2, 64))
    v = rng.standard_normal((37, 2, 64))
    kw, vw = ro.gather_rope(k, v, [(0, 37)], THETA)
    assert np.array_equal(kw, so.rope(k, 0, THETA))
    assert np.array_equal(vw, v)
    # two abutting segments are the same as one
    kw2, _ = ro.gather_rope(k, v, [(0, 20), (20, 17)], THETA)
    assert np.allclose(kw2, kw, atol=1e-13)


def test_rotations_compose_so_a_rotated_cache_could_be_reindexed():
    # R(p') k = R(p' - p) R(p) k: the mathematical fact behind "decoupling position ids from the cache"
    rng = np.random.default_rng(1)
    k = rng.standard_normal((1, 3, 64))
    for p, p2 in ((100, 7), (4000, 3999), (12, 800)):
        direct = so.rope(k, p2, THETA)
        back = so.rope(so.rope(k, p, THETA), p2 - p, THETA)
        assert np.allclose(direct, back, atol=1e-11)


def test_kept_tokens_get_contiguous_positions():
    # a key that is dropped leaves no gap: the token after it takes its position
    rng = np.random.default_rng(2)
    k = rng.standard_normal((12, 1, 64))
    v = rng.standard_normal((12, 1, 64))
    kw, vw = ro.gather_rope(k, v, [(0, 4), (8, 4)], THETA)
    assert kw.shape[0] == 8
    assert np.allclose(kw[4:], so.rope(k[8:12], 4, THETA), atol=1e-13)
    assert np.array_equal(vw[4:], v[8:12])


@pytest.mark.parametrize("sampler", ["uniform", "sliding"])
def test_sampled_steps_equal_full_prefill_of_the_kept_sequence(sampler):
    # the step on (kept history + new frame) is exactly a causal prefill over that token sequence
    rng = np.random.default_rng(3)
    Hq, Hkv, D, I, F, n = 4, 2, 64, 5, 6, 6
    frames_total = 9
    k_store = rng.standard_normal((I + frames_total * F, Hkv, D))
    v_store = rng.standard_normal((I + frames_total * F, Hkv, D))
    for t in (3, 9):                     # number of history frames at this step
        kept = ro.sample_uniform(t, 4) if sampler == "uniform" else ro.sample_sliding(t, 4, 2)
        segs = ro.frame_segments(I, F, kept)
        q_new = rng.standard_normal((n, Hq, D))
        k_new = rng.standard_normal((n, Hkv, D))
        v_new = rng.standard_normal((n, Hkv, D))
        r = ro.sampled_step(q_new, k_new, v_new, k_store, v_store, segs, THETA)
        # brute force: the kept raw tokens followed by the new frame, positions 0..T-1
        idx = np.concatenate([np.arange(s, s + l) for s, l in segs])
        k_all = np.concatenate([k_store[idx], k_new])
        v_all = np.concatenate([v_store[idx], v_new])
        T = k_all.shape[0]
        q_all = np.concatenate([rng.standard_normal((T - n, Hq, D)), q_new])
        full = pb.full_prefill(q_all, k_all, v_all, THETA)
        out = full[0] if isinstance(full, tuple) else full["out"]
        assert np.allclose(r["out"], out[T - n:], atol=1e-11)
