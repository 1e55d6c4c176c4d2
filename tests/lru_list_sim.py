"""Brute-force simulator used to pin the oracle: recency kept as an explicit ordered list of slots.

It is written independently of the oracle's stamp arithmetic: there are no stamps and no sort by
stamp here, only list surgery.  After a step the list is
    (untouched slots, in their old order) ++ (slots refilled in this step, by slot) ++ (hit slots, by slot)
which is the replacement policy of Sec. 3.2 / Phase 3 of Sec. 3.4 (hits to the most-recent end,
fetched misses just behind them) with ties inside a step broken by slot number.
Pure Python, for tiny inputs only.
"""
from __future__ import annotations

from typing import List, Sequence


MASK64 = (1 << 64) - 1


def mix64(z: int) -> int:
    z = (z + 0x9E3779B97F4A7C15) & MASK64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & MASK64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & MASK64
    return z ^ (z >> 31)


def random_key(seed: int, r: int, g: int, t: int, slot: int) -> int:
    """Key of the RANDOM policy: low 32 bits of mix64(mix64(seed ^ (r << 32 | g)) + (t << 32 | slot))."""
    a = mix64(seed ^ ((r << 32) | g))
    return mix64((a + ((t << 32) | slot)) & MASK64) & 0xFFFFFFFF


class ListLRUSim:
    """policy: "lru" (hits to the most-recent end), "fifo" (hits leave the list alone: insertion order) or
    "random" (list kept as for lru; victims = the m non-hit slots with the smallest hashed key, paired with the
    misses in ascending slot order)."""

    def __init__(self, cache_slots: int, top_k: int, length: int, policy: str = "lru", seed: int = 0,
                 request: int = 0, group: int = 0):
        self.policy, self.seed, self.request, self.group, self.t = policy, seed, request, group, 0
        self.B, self.k = cache_slots, top_k
        self.order: List[int] = list(range(cache_slots))  # least recent first
        self.slot_pos: List[int] = [-1] * cache_slots
        self.len = length
        self.newest = -1
        self.out_of_range = False
        self.duplicate = False

    def append(self) -> None:
        self.newest = self.len
        self.len += 1

    def resolve(self, row: Sequence[int]):
        B = self.B
        where = {p: s for s, p in enumerate(self.slot_pos) if p >= 0}
        out = [-1] * len(row)
        first_at = {}
        follows = {}
        hit_slots = set()
        miss_js: List[int] = []
        hits = 0
        for j, p in enumerate(row):
            p = int(p)
            if p == -1:
                continue
            if p < 0 or p >= self.len:
                self.out_of_range = True
                continue
            if p in first_at:
                self.duplicate = True
                follows[j] = first_at[p]
                continue
            first_at[p] = j
            if p == self.newest:
                out[j] = B
                hits += 1
            elif p in where:
                out[j] = where[p]
                hit_slots.add(where[p])
                hits += 1
            else:
                miss_js.append(j)
        self.t += 1
        not_hit = [s for s in self.order if s not in hit_slots]
        if self.policy == "random":
            ranked = sorted(not_hit, key=lambda s: (random_key(self.seed, self.request, self.group, self.t, s), s))
            victims = sorted(ranked[: len(miss_js)])
        else:
            victims = not_hit[: len(miss_js)]
        evicted = []
        for j, v in zip(miss_js, victims):
            evicted.append(self.slot_pos[v])
            self.slot_pos[v] = int(row[j])
            out[j] = v
        if self.policy == "fifo":
            self.order = [s for s in self.order if s not in victims] + sorted(victims)
        else:
            untouched = [s for s in not_hit if s not in victims]
            self.order = untouched + sorted(victims) + sorted(hit_slots)
        for j, j0 in follows.items():
            out[j] = out[j0]
        plan = [(int(row[j]), v) for j, v in zip(miss_js, victims)]
        return out, hits, len(miss_js), plan, evicted
