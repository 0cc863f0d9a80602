"""Which frames of an episode are resident in the device store, and where (host bookkeeping only).

Sec. 3.2 ("Memory Management") keeps the whole raw KV store on the CPU and reloads only the
segments the frame sampler selects.  The device store then has a fixed number of frame slots;
this class maps frame ids to slots, tells the caller which kept frames have to be fetched from
the host store (``evlnStoreFetch``) before ``evlnGatherRope`` runs, and evicts the least recently
kept frames.  It moves no data and contains none of the method's arithmetic.
"""
from __future__ import annotations

from collections import OrderedDict
from typing import Dict, List, Sequence, Tuple


class FrameResidency:
    def __init__(self, num_slots: int, instr_len: int, frame_tokens: int):
        if num_slots < 1:
            raise ValueError("need at least one frame slot")
        self.num_slots, self.instr_len, self.frame_tokens = num_slots, instr_len, frame_tokens
        self._slot_of: "OrderedDict[int, int]" = OrderedDict()      # frame -> slot, least recently kept first
        self._free: List[int] = list(range(num_slots))[::-1]

    def slot_start(self, slot: int) -> int:
        """First token slot of a frame slot in the device store (the instruction sits in front)."""
        return self.instr_len + slot * self.frame_tokens

    def resident(self) -> Dict[int, int]:
        return dict(self._slot_of)

    def plan(self, kept: Sequence[int], host_frame_start) -> Tuple[List[Tuple[int, int, int]], List[Tuple[int, int]]]:
        """Makes every frame of ``kept`` resident.

        Returns ``(fetches, segments)``: ``fetches`` = ``(frame, host token slot, device token slot)``
        of the frames that have to be copied in, ``segments`` = ``(device token slot, length)`` of the
        instruction and of the kept frames in the order given, ready for ``evlnGatherRope``.
        ``host_frame_start(frame)`` gives a frame's first token slot in the host store.
        """
        kept = list(kept)
        if len(set(kept)) != len(kept):
            raise ValueError("a frame is kept twice")
        if len(kept) > self.num_slots:
            raise ValueError("more frames kept than the device store has slots")
        keep = set(kept)
        fetches = []
        for f in kept:
            if f in self._slot_of:
                self._slot_of.move_to_end(f)
                continue
            if not self._free:
                victim = next(g for g in self._slot_of if g not in keep)      # least recently kept, not needed now
                self._free.append(self._slot_of.pop(victim))
            slot = self._free.pop()
            self._slot_of[f] = slot
            fetches.append((f, host_frame_start(f), self.slot_start(slot)))
        segments = [(0, self.instr_len)] if self.instr_len > 0 else []
        segments += [(self.slot_start(self._slot_of[f]), self.frame_tokens) for f in kept]
        return fetches, segments

    def admit(self, frame: int) -> int:
        """A frame that is produced on the device (the new frame): gives it a slot without a fetch.
        Returns the device token slot, or -1 if every slot holds a frame (nothing is evicted here)."""
        if frame in self._slot_of:
            return self.slot_start(self._slot_of[frame])
        if not self._free:
            return -1
        slot = self._free.pop()
        self._slot_of[frame] = slot
        return self.slot_start(slot)
