"""Host bookkeeping of the device-resident frame slots (no GPU)."""
import numpy as np
import pytest

from oracle import reindex_oracle as ro
from paper_2512_10310_b200.residency import FrameResidency

I_LEN, F_TOK = 256, 196


def _host_start(f):
    return I_LEN + f * F_TOK


def test_kept_frames_become_resident_and_slots_are_distinct():
    r = FrameResidency(8, I_LEN, F_TOK)
    fetches, segs = r.plan([0, 3, 5], _host_start)
    assert [f for f, _, _ in fetches] == [0, 3, 5]
    assert segs[0] == (0, I_LEN) and len(segs) == 4
    starts = [s for s, _ in segs[1:]]
    assert len(set(starts)) == 3 and all((s - I_LEN) % F_TOK == 0 for s in starts)
    assert [h for _, h, _ in fetches] == [_host_start(f) for f in (0, 3, 5)]
    # a second plan with the same frames fetches nothing and keeps the slots
    fetches2, segs2 = r.plan([0, 3, 5], _host_start)
    assert fetches2 == [] and segs2 == segs


def test_eviction_never_touches_a_kept_frame():
    r = FrameResidency(4, I_LEN, F_TOK)
    r.plan([0, 1, 2, 3], _host_start)
    fetches, segs = r.plan([2, 3, 7, 9], _host_start)
    assert sorted(f for f, _, _ in fetches) == [7, 9]
    res = r.resident()
    assert set(res) == {2, 3, 7, 9} and len(set(res.values())) == 4
    with pytest.raises(ValueError):
        r.plan([1, 2, 3, 4, 5], _host_start)
    with pytest.raises(ValueError):
        r.plan([1, 1], _host_start)


def test_transfers_per_step_match_the_papers_statement():
    # sliding window (stride 1): one new segment per step; uniform: about half the budget (Sec. 3.2)
    B = 16
    for sampler, lo, hi in (("sliding", 1.0, 1.0), ("uniform", 0.3 * B, 0.7 * B)):
        r = FrameResidency(B, I_LEN, F_TOK)
        counts = []
        for t in range(1, 200):
            kept = ro.sample_sliding(t, B, 1) if sampler == "sliding" else ro.sample_uniform(t, B)
            fetches, segs = r.plan(kept, _host_start)
            assert len(segs) == 1 + len(kept)
            if t > 40:
                counts.append(len(fetches))
        assert lo <= np.mean(counts) <= hi


def test_new_frame_can_be_admitted_without_a_fetch():
    r = FrameResidency(2, I_LEN, F_TOK)
    s0 = r.admit(0)
    assert s0 == I_LEN + (s0 - I_LEN) // F_TOK * F_TOK and s0 >= I_LEN
    fetches, _ = r.plan([0], _host_start)
    assert fetches == []
    r.admit(1)
    assert r.admit(2) == -1
