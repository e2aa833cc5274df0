"""CPU model of the store's capacity management.  TEST INFRASTRUCTURE ONLY (see oracle/reuse_prefill.py).

Paper Section 3.2.1 ("Cache Architecture"): the storage limit for the cache is configurable; a retrieval
counter is kept per cached entry and the least-frequently-used entries are evicted so that the storage does
not exceed the limit.  Readings taken where the paper is silent:
  * the counter of a chunk is the number of prompts that used it: 1 for the prompt that stored it, +1 for every
    later prompt occurrence that hits it;
  * ties are broken by age: the entry inserted earliest goes first;
  * a chunk the calling batch itself hits is never evicted by that call;
  * storage is counted in pages of 16 tokens (ceil(tokens / 16) per chunk), all layers together;
  * if the new chunks cannot be made to fit, the call fails and nothing is evicted.
Everything here is integer bookkeeping written as plain loops.
"""
from __future__ import annotations

from typing import Dict, List, Sequence, Tuple

PAGE_TOKENS = 16


class NoSpace(Exception):
    pass


def pages_of(n_tokens: int) -> int:
    return (n_tokens + PAGE_TOKENS - 1) // PAGE_TOKENS


class LfuModel:
    def __init__(self, limit_pages: int, evict: bool = True):
        self.limit = limit_pages
        self.evict = evict
        self.entries: Dict[int, Dict[str, int]] = {}     # id -> {tokens, count, serial}
        self.serial = 0

    def used(self) -> int:
        total = 0
        for e in self.entries.values():
            total += pages_of(e["tokens"])
        return total

    def _make_room(self, need: int, keep: Sequence[int]) -> List[int]:
        over = self.used() + need - self.limit
        if over <= 0:
            return []
        if not self.evict:
            raise NoSpace()
        candidates = []
        for cid, e in self.entries.items():
            if cid not in keep:
                candidates.append((e["count"], e["serial"], cid))
        candidates.sort()
        victims = []
        for count, serial, cid in candidates:
            if over <= 0:
                break
            victims.append(cid)
            over -= pages_of(self.entries[cid]["tokens"])
        if over > 0:
            raise NoSpace()
        for cid in victims:
            del self.entries[cid]
        return victims

    def insert(self, cid: int, tokens: int) -> List[int]:
        """Direct insertion (put).  Returns the evicted ids."""
        victims = self._make_room(pages_of(tokens), [])
        self.entries[cid] = {"tokens": tokens, "count": 1, "serial": self.serial}
        self.serial += 1
        return victims

    def set_limit(self, limit_pages: int) -> List[int]:
        old = self.limit
        self.limit = limit_pages
        try:
            return self._make_room(0, [])
        except NoSpace:
            self.limit = old
            raise

    def call(self, prompts: Sequence[Tuple[Sequence[int], Sequence[int]]]) -> Tuple[List[List[int]], List[int]]:
        """One prefill call.  prompts: [(chunk ids, chunk lengths)].  Returns (hit masks, evicted ids)."""
        masks: List[List[int]] = []
        hit_uses: Dict[int, int] = {}
        new: List[Tuple[int, int]] = []
        seen_new = set()
        for ids, lens in prompts:
            mask = []
            for cid, n in zip(ids, lens):
                if cid in self.entries:
                    mask.append(1)
                    hit_uses[cid] = hit_uses.get(cid, 0) + 1
                else:
                    mask.append(0)
                    if cid not in seen_new:
                        seen_new.add(cid)
                        new.append((cid, n))
            masks.append(mask)
        need = 0
        for cid, n in new:
            need += pages_of(n)
        victims = self._make_room(need, list(hit_uses))
        for cid, n in new:                         # in prompt order, like the library's commit
            self.entries[cid] = {"tokens": n, "count": 1, "serial": self.serial}
            self.serial += 1
        for cid, k in hit_uses.items():
            self.entries[cid]["count"] += k
        return masks, victims
