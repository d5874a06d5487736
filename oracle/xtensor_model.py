"""Plain Python model of the xTensor page bookkeeping (test infrastructure only).

Follows the xTensor section of the report: a pool of fixed-size physical pages created at start-up,
each carrying <PageID, Status, OwnerSession> with Status in {Free, Allocated, Mapped, Reusable}; one
virtual range per request slot; pages mapped on demand at the next contiguous position of the
range as the sequence grows ("On-demand Memory Mapping"); on completion pages are kept as Reusable
and handed to a later request instead of being unmapped ("Physical Page Reuse").

Readings where the report is silent (the library under test documents the same ones):
  * a page covers whole tile blocks of ``tile_tokens`` tokens; ``pages_for(t)`` is the number of pages
    that cover ceil(t / tile_tokens) blocks of ``tile_tokens * row_bytes`` bytes;
  * Free pages form a stack, page 0 on top at start; a full unmap pushes a slot's pages back so that
    its first page is on top;
  * a released slot keeps its pages mapped in place (Reusable, owner kept); ``reserve`` prefers the
    released slot whose page set fits the hinted size best (smallest set that is large enough, else the
    largest set), else the lowest unused slot id;
  * when the Free stack is empty, Reusable pages are reclaimed (unmapped) from the tail of released
    slots first, then from the Reusable tail of live slots, lowest slot id first;
  * "Allocated" is the state between leaving the Free stack and being mapped; it is never observable
    between calls.
No GPU, no driver: integers only.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List

FREE, ALLOCATED, MAPPED, REUSABLE = 0, 1, 2, 3

OK, ERR_INVALID, ERR_OOM_PHYS, ERR_OOM_VA, ERR_NOT_MAPPED = 0, -1, -2, -3, -4


@dataclass
class _Slot:
    live: bool = False
    pages: List[int] = field(default_factory=list)  # in virtual-address order
    n_owned: int = 0                                # pages[:n_owned] Mapped, the rest Reusable
    kv_len: int = 0


class PagePoolModel:
    def __init__(self, n_pages: int, page_bytes: int, row_bytes: int, tile_tokens: int, max_slots: int,
                 max_seq_len: int):
        self.page_bytes, self.row_bytes, self.tile_tokens = page_bytes, row_bytes, tile_tokens
        self.max_seq_len = max_seq_len
        self.status = [FREE] * n_pages
        self.owner = [-1] * n_pages
        self.free: List[int] = list(range(n_pages - 1, -1, -1))  # pop() yields page 0 first
        self.slots: Dict[int, _Slot] = {i: _Slot() for i in range(max_slots)}
        self.pages_mapped_total = 0    # driver map operations (one per page)
        self.pages_unmapped_total = 0  # driver unmap operations (one per page)
        self.pages_reused_total = 0    # Reusable -> Mapped promotions (no driver call)

    # ---- arithmetic -------------------------------------------------------------------
    def pages_for(self, tokens: int) -> int:
        blocks = -(-tokens // self.tile_tokens)
        nbytes = blocks * self.tile_tokens * self.row_bytes
        return -(-nbytes // self.page_bytes)

    def mapped_tokens(self, slot: int) -> int:
        s = self.slots[slot]
        blocks = (s.n_owned * self.page_bytes) // (self.tile_tokens * self.row_bytes)
        return blocks * self.tile_tokens

    # ---- operations -------------------------------------------------------------------
    def reserve(self, hint_tokens: int = 0) -> int:
        need = self.pages_for(hint_tokens)
        idle = [i for i, s in self.slots.items() if not s.live]
        if not idle:
            return ERR_OOM_VA
        with_pages = [i for i in idle if self.slots[i].pages]
        fit = [i for i in with_pages if len(self.slots[i].pages) >= need]
        if fit:
            pick = min(fit, key=lambda i: (len(self.slots[i].pages), i))
        elif with_pages and need > 0:
            pick = min(with_pages, key=lambda i: (-len(self.slots[i].pages), i))
        else:
            pick = min(idle)
        s = self.slots[pick]
        s.live, s.n_owned, s.kv_len = True, 0, 0
        return pick

    def _reclaim_one(self, needy: int) -> bool:
        for want_live in (False, True):
            for i in sorted(self.slots):
                s = self.slots[i]
                if i == needy or s.live != want_live or len(s.pages) <= s.n_owned:
                    continue
                p = s.pages.pop()
                self.status[p], self.owner[p] = FREE, -1
                self.free.append(p)
                self.pages_unmapped_total += 1
                return True
        return False

    def map_pages(self, slot: int, min_tokens: int) -> int:
        s = self.slots.get(slot)
        if s is None or not s.live or min_tokens < 0 or min_tokens > self.max_seq_len:
            return ERR_INVALID
        need = self.pages_for(min_tokens)
        if need <= s.n_owned:
            return OK
        promote = min(need, len(s.pages)) - s.n_owned
        fresh = need - s.n_owned - promote
        reclaimable = sum(len(o.pages) - o.n_owned for i, o in self.slots.items() if i != slot)
        if fresh > len(self.free) + reclaimable:
            return ERR_OOM_PHYS  # nothing changed
        for p in s.pages[s.n_owned:s.n_owned + promote]:
            self.status[p] = MAPPED
        self.pages_reused_total += promote
        s.n_owned += promote
        for _ in range(fresh):
            if not self.free:
                assert self._reclaim_one(slot)
            p = self.free.pop()
            self.status[p], self.owner[p] = MAPPED, slot  # Free -> Allocated -> Mapped
            s.pages.append(p)
            s.n_owned += 1
            self.pages_mapped_total += 1
        return OK

    def release(self, slot: int, mode: int) -> int:
        s = self.slots.get(slot)
        if s is None or not s.live or mode not in (0, 1):
            return ERR_INVALID
        if mode == 0:
            for p in s.pages:
                self.status[p] = REUSABLE
        else:
            for p in reversed(s.pages):
                self.status[p], self.owner[p] = FREE, -1
                self.free.append(p)
            self.pages_unmapped_total += len(s.pages)
            s.pages = []
        s.live, s.n_owned, s.kv_len = False, 0, 0
        return OK

    def counts(self) -> Dict[str, int]:
        c = {"free": 0, "allocated": 0, "mapped": 0, "reusable": 0}
        for st in self.status:
            c[("free", "allocated", "mapped", "reusable")[st]] += 1
        return c

    def check_invariants(self) -> None:
        seen = set()
        for i, s in self.slots.items():
            assert 0 <= s.n_owned <= len(s.pages)
            for j, p in enumerate(s.pages):
                assert p not in seen
                seen.add(p)
                assert self.owner[p] == i
                assert self.status[p] == (MAPPED if j < s.n_owned else REUSABLE)
        assert seen.isdisjoint(self.free) and len(seen) + len(self.free) == len(self.status)
        for p in self.free:
            assert self.status[p] == FREE and self.owner[p] == -1
