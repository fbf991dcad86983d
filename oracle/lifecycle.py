"""Host model of the page lifecycle -- TEST INFRASTRUCTURE ONLY (part of the oracle).

Follows Algorithm 1 (ownership-aware page-transition protocol) and Fig. "lifecycle":

    Recent --age/demote--> Stale      Recent --protect--> Anchor
    Anchor --demote------> Stale      Stale  --promote--> Anchor

with the copy-before-publish rule (a destination is populated before its tag and physical id are
published; the source is released afterwards) and per-format free lists.  "Afterwards" is a point the
planner cannot see: Algorithm 1 releases a source only once its readers and the conversion have cleared.
So Retier and Promote leave the source RETIRING -- owned by the request, mapped nowhere, on no free list,
never handed out -- until the caller says that point has passed (SeqModel.release).  SealPrefix and the
prefix cache are outside the modelled path.  No transition ever drops a logical page of a live
request.

Allocation policy (the paper is silent): each free list is a stack that initially pops
0, 1, 2, ...; a released id goes back on top.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

T = 16
RECENT, ANCHOR, STALE = 0, 1, 2
FMT_FP8, FMT_TQ3 = 0, 1


class LifecycleError(Exception):
    def __init__(self, code: str, msg: str = ""):
        super().__init__(f"{code}: {msg}")
        self.code = code


class PoolModel:
    def __init__(self, fp8_pages: int, tq3_pages: int, page_tokens: int = T):
        self.T = page_tokens               # tokens per page (16, or 16 M for the paper-scale blocks)
        self.capacity = {FMT_FP8: fp8_pages, FMT_TQ3: tq3_pages}
        self.free = {FMT_FP8: list(range(fp8_pages - 1, -1, -1)),
                     FMT_TQ3: list(range(tq3_pages - 1, -1, -1))}
        self.owner: Dict[Tuple[int, int], int] = {}    # (fmt, id) -> sequence handle (mapped pages)
        self.retiring: Dict[Tuple[int, int], int] = {} # (fmt, id) -> sequence handle (sources awaiting release)
        self.seqs: Dict[int, "SeqModel"] = {}
        self._next = 0

    def alloc(self, fmt: int, owner: int) -> int:
        if not self.free[fmt]:
            raise LifecycleError("MKV_E_OOM_FP8" if fmt == FMT_FP8 else "MKV_E_OOM_TQ3")
        pid = self.free[fmt].pop()
        self.owner[(fmt, pid)] = owner
        return pid

    def release(self, fmt: int, pid: int):
        if (fmt, pid) not in self.owner:
            raise LifecycleError("MKV_E_STATE", "double free")
        del self.owner[(fmt, pid)]
        self.free[fmt].append(pid)

    def retire(self, fmt: int, pid: int):
        """A conversion's source: no longer mapped, not yet reusable."""
        if (fmt, pid) not in self.owner:
            raise LifecycleError("MKV_E_STATE", "not an owned page")
        self.retiring[(fmt, pid)] = self.owner.pop((fmt, pid))

    def release_retired(self, fmt: int, pid: int, owner: int):
        if not 0 <= pid < self.capacity[fmt]:
            raise LifecycleError("MKV_E_BOUNDS", "page id out of range")
        if self.retiring.get((fmt, pid)) != owner:
            raise LifecycleError("MKV_E_STATE", "page is not retiring for this request")
        del self.retiring[(fmt, pid)]
        self.free[fmt].append(pid)

    def new_seq(self) -> "SeqModel":
        s = SeqModel(self, self._next)
        self.seqs[self._next] = s
        self._next += 1
        return s

    def stats(self):
        used = {FMT_FP8: 0, FMT_TQ3: 0}
        tiers = {RECENT: 0, ANCHOR: 0, STALE: 0}
        for s in self.seqs.values():
            for tag, pid in s.pages:
                tiers[tag] += 1
                used[FMT_TQ3 if tag == STALE else FMT_FP8] += 1
        for fmt, _ in self.retiring:          # a retiring source still occupies its arena
            used[fmt] += 1
        return used, tiers

    def check_invariants(self):
        """Every logical page of a live request maps to exactly one physical page; no physical page
        is mapped twice, or both mapped and free."""
        seen = set()
        for s in self.seqs.values():
            assert len(s.pages) == (s.len + self.T - 1) // self.T
            for tag, pid in s.pages:
                fmt = FMT_TQ3 if tag == STALE else FMT_FP8
                assert 0 <= pid < self.capacity[fmt]
                assert (fmt, pid) not in seen, "page mapped twice"
                seen.add((fmt, pid))
                assert self.owner.get((fmt, pid)) == s.handle
                assert pid not in self.free[fmt], "mapped page on a free list"
        assert seen == set(self.owner.keys()), "owned page not mapped (leak)"
        for (fmt, pid), h in self.retiring.items():
            assert h in self.seqs, "retiring page of a finished request"
            assert (fmt, pid) not in seen, "retiring page still mapped"
            assert pid not in self.free[fmt], "retiring page handed back before its release"
        for fmt in (FMT_FP8, FMT_TQ3):
            assert len(set(self.free[fmt])) == len(self.free[fmt])
            assert (len(self.free[fmt]) + sum(1 for f, _ in self.owner if f == fmt) +
                    sum(1 for f, _ in self.retiring if f == fmt)) == self.capacity[fmt]


class SeqModel:
    def __init__(self, pool: PoolModel, handle: int):
        self.pool = pool
        self.handle = handle
        self.len = 0
        self.pages: List[Tuple[int, int]] = []   # logical page -> (tag, physical id)

    # Append(q, p): allocate a request-owned Recent page when the previous one is full, write KV,
    # then publish the mapping.  Returns (physical id, slot, opened_new_page).
    def append(self):
        opened = self.len % self.pool.T == 0
        if opened:
            pid = self.pool.alloc(FMT_FP8, self.handle)
            self.pages.append((RECENT, pid))
        tag, pid = self.pages[-1]
        slot = self.len % self.pool.T
        self.len += 1
        return pid, slot, opened

    def _full(self, lp: int) -> bool:
        return (lp + 1) * self.pool.T <= self.len

    def protect(self, lp: int):
        tag, pid = self._get(lp)
        if tag == STALE:
            raise LifecycleError("MKV_E_STATE", "protect needs an FP8 page; promote first")
        self.pages[lp] = (ANCHOR, pid)

    def unprotect(self, lp: int):
        tag, pid = self._get(lp)
        if tag != ANCHOR:
            raise LifecycleError("MKV_E_STATE", "page is not Anchor")
        self.pages[lp] = (RECENT, pid)

    # Retier(p, TQ3): retain the source, allocate and populate the destination, publish tag + id;
    # the source is retiring until release().  Returns (source fp8 id, destination tq3 id).
    def demote(self, lp: int):
        tag, src = self._get(lp)
        if tag == STALE:
            raise LifecycleError("MKV_E_STATE", "already Stale")
        if not self._full(lp):
            raise LifecycleError("MKV_E_STATE", "only full pages may become TQ3")
        dst = self.pool.alloc(FMT_TQ3, self.handle)
        self.pages[lp] = (STALE, dst)      # publish (after the destination is populated)
        self.pool.retire(FMT_FP8, src)     # released only after readers and the conversion cleared
        return src, dst

    # Promote(p): reconstruct into a newly allocated FP8 page, publish, retire the TQ3 page.
    def promote(self, lp: int):
        tag, src = self._get(lp)
        if tag != STALE:
            raise LifecycleError("MKV_E_STATE", "not Stale")
        dst = self.pool.alloc(FMT_FP8, self.handle)
        self.pages[lp] = (ANCHOR, dst)
        self.pool.retire(FMT_TQ3, src)
        return src, dst

    # The point Algorithm 1 waits for has passed (earlier readers and the conversion are ordered before
    # any later writer of the page): the retiring source goes back to its free list.
    def release(self, fmt: int, pid: int):
        self.pool.release_retired(fmt, pid, self.handle)

    def age(self, recent_tokens: int):
        """Demote every full Recent page that lies wholly before the last `recent_tokens` tokens."""
        moved = []
        first_recent = max(0, self.len - recent_tokens) // self.pool.T
        for lp in range(min(first_recent, len(self.pages))):
            if self.pages[lp][0] == RECENT and self._full(lp):
                moved.append((lp,) + self.demote(lp))
        return moved

    # Finish(q): release the request's references.
    def finish(self):
        for tag, pid in self.pages:
            self.pool.release(FMT_TQ3 if tag == STALE else FMT_FP8, pid)
        for (fmt, pid), h in sorted(self.pool.retiring.items()):     # in (format, id) order
            if h == self.handle:
                self.pool.release_retired(fmt, pid, h)
        self.pages = []
        self.len = 0
        del self.pool.seqs[self.handle]

    def _get(self, lp: int):
        if not 0 <= lp < len(self.pages):
            raise LifecycleError("MKV_E_BOUNDS", "logical page out of range")
        return self.pages[lp]
