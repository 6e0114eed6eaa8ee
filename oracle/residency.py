"""TEST INFRASTRUCTURE -- plain model of the expert residency policy of an offloaded layer
(Sec. 5, "Edge memory constraints and expert-level offloading": experts fetched on demand, hot
experts kept resident).  Only tests may import this module; the library shares no code with it.

The paper fixes the mechanism (expert granularity, on-demand fetch, a resident hot set from offline
profiling), not the replacement rule; the rule modelled here is the one the library documents:

  * pinned experts own slots 0 .. n_pinned-1 for good;
  * one access names distinct experts that must all be resident together;
  * a missing expert takes the free slot of lowest index, else the unpinned slot that was used
    least recently and holds no expert of this access (ties: lowest slot index);
  * misses are served in the order the experts are named.

PARITY UNPINNED: the replacement rule is this build's reading (the paper names none); what is
pinned is that every access leaves all of its experts resident, that pinned experts never move,
and that the rule is least-recently-used (checked against a brute-force recency list).
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence, Tuple


class ResidencyModel:
    def __init__(self, n_experts: int, n_slots: int, pinned: Sequence[int] = ()):
        if not (1 <= n_slots and len(pinned) <= n_slots and len(set(pinned)) == len(pinned)):
            raise ValueError("bad residency arguments")
        self.n_experts, self.n_slots = n_experts, n_slots
        self.pinned = list(pinned)
        self.slot_expert: List[Optional[int]] = [None] * n_slots
        for i, e in enumerate(pinned):
            self.slot_expert[i] = e
        self.stamp = [0] * n_slots          # access number that last used the slot
        self.now = 0
        self.hits = self.misses = 0

    def where(self) -> Dict[int, int]:
        return {e: s for s, e in enumerate(self.slot_expert) if e is not None}

    def access(self, experts: Sequence[int]) -> Tuple[List[int], List[int]]:
        """Returns (slots, missed flags); raises ValueError when the experts cannot all be resident."""
        experts = list(experts)
        if len(set(experts)) != len(experts) or any(not 0 <= e < self.n_experts for e in experts):
            raise ValueError("experts must be distinct and in range")
        where = self.where()
        wanted = set(experts)
        missing = [e for e in experts if e not in where]
        usable = [s for s in range(len(self.pinned), self.n_slots)
                  if self.slot_expert[s] is None or self.slot_expert[s] not in wanted]
        if len(experts) > self.n_slots or len(missing) > len(usable):
            raise ValueError("more experts than slots")
        self.now += 1
        slots, missed = [], []
        for e in experts:
            where = self.where()
            if e in where:
                s = where[e]
                self.hits += 1
                missed.append(0)
            else:
                self.misses += 1
                missed.append(1)
                free = [c for c in range(len(self.pinned), self.n_slots) if self.slot_expert[c] is None]
                if free:
                    s = free[0]
                else:
                    cand = [c for c in range(len(self.pinned), self.n_slots) if self.slot_expert[c] not in wanted]
                    s = min(cand, key=lambda c: (self.stamp[c], c))
                self.slot_expert[s] = e
            self.stamp[s] = self.now
            slots.append(s)
        return slots, missed
