"""Host-side residency policies that decide which context units are cache hits.

Not part of the GPU hot path: this is the retrieval-aware admission / eviction rule of Sec. 5.2,
used only to give synthetic traces the hit / miss pattern the paper's policy would produce (instead
of "everything cached"), next to LRU and LFU for comparison.  Capacity is counted in storage blocks,
replacement works on whole units.

Score of unit u at request ordinal t (Sec. 5.2):  s(u, t) = w_r * f_W(u, t) + w_l * f_inf(u, t),
f_W = number of the last W requests that retrieved u, f_inf = number of all requests so far that
retrieved u; w_r = 1, w_l = 0.05.  A unit is an admission candidate once s >= theta; with the default
theta = 2 a single retrieval (s = 1.05) never admits.  When space is short, residents are considered
in increasing score order and the candidate is admitted only if residents with STRICTLY lower scores
free enough blocks.
"""
from __future__ import annotations

import collections
from typing import Dict, Hashable, Iterable, List, Sequence, Tuple

Unit = Tuple[Hashable, int]          # (unit id, size in blocks)


class ReuseScoreCache:
    def __init__(self, capacity_blocks: int, window: int, w_r: float = 1.0, w_l: float = 0.05, theta: float = 2.0):
        if capacity_blocks < 0 or window < 1:
            raise ValueError("capacity must be >= 0 and window >= 1")
        self.capacity, self.window, self.w_r, self.w_l, self.theta = capacity_blocks, window, w_r, w_l, theta
        self.resident: Dict[Hashable, int] = {}                  # uid -> blocks
        self.used = 0
        self.total: Dict[Hashable, int] = collections.Counter()  # f_inf
        self.recent: Dict[Hashable, int] = collections.Counter() # f_W
        self.history = collections.deque()                       # the last W requests, as sets of uids
        self.t = 0

    @staticmethod
    def window_for(capacity_blocks: int, avg_blocks_per_request: float) -> int:
        """W = number of recent requests whose retrieved units would fill the cache (Sec. 5.2)."""
        return max(1, int(round(capacity_blocks / max(avg_blocks_per_request, 1e-9))))

    def score(self, uid) -> float:
        return self.w_r * self.recent.get(uid, 0) + self.w_l * self.total.get(uid, 0)

    def request(self, units: Sequence[Unit]) -> List[bool]:
        """One request: returns per unit whether it was resident BEFORE the request, then records the
        retrieval and applies admission / eviction to the units that missed."""
        hits = [uid in self.resident for uid, _ in units]
        self.t += 1
        seen = set(uid for uid, _ in units)
        self.history.append(seen)
        for uid in seen:
            self.total[uid] += 1
            self.recent[uid] += 1
        if len(self.history) > self.window:
            for uid in self.history.popleft():
                self.recent[uid] -= 1
                if self.recent[uid] == 0:
                    del self.recent[uid]
        done = set()
        for (uid, blocks), hit in zip(units, hits):
            if hit or uid in done or uid in self.resident:
                continue
            done.add(uid)
            self._admit(uid, blocks)
        return hits

    def _admit(self, uid, blocks: int) -> bool:
        s = self.score(uid)
        if s < self.theta or blocks > self.capacity:
            return False
        free = self.capacity - self.used
        victims = []
        if free < blocks:
            for v in sorted(self.resident, key=lambda x: (self.score(x), str(x))):
                if self.score(v) >= s:                 # only strictly lower scores may be displaced
                    break
                victims.append(v)
                free += self.resident[v]
                if free >= blocks:
                    break
            if free < blocks:
                return False
        for v in victims:
            self.used -= self.resident.pop(v)
        self.resident[uid] = blocks
        self.used += blocks
        return True


class LRUCache:
    def __init__(self, capacity_blocks: int):
        self.capacity, self.used = capacity_blocks, 0
        self.resident = collections.OrderedDict()

    def request(self, units: Sequence[Unit]) -> List[bool]:
        hits = []
        for uid, blocks in units:
            hit = uid in self.resident
            hits.append(hit)
            if hit:
                self.resident.move_to_end(uid)
                continue
            if blocks > self.capacity:
                continue
            while self.used + blocks > self.capacity:
                _, b = self.resident.popitem(last=False)
                self.used -= b
            self.resident[uid] = blocks
            self.used += blocks
        return hits


class LFUCache:
    def __init__(self, capacity_blocks: int):
        self.capacity, self.used = capacity_blocks, 0
        self.resident: Dict[Hashable, int] = {}
        self.count: Dict[Hashable, int] = collections.Counter()
        self.tick = 0
        self.last: Dict[Hashable, int] = {}

    def request(self, units: Sequence[Unit]) -> List[bool]:
        hits = []
        for uid, blocks in units:
            self.tick += 1
            self.count[uid] += 1
            self.last[uid] = self.tick
            hit = uid in self.resident
            hits.append(hit)
            if hit or blocks > self.capacity:
                continue
            while self.used + blocks > self.capacity:
                v = min(self.resident, key=lambda x: (self.count[x], self.last[x]))
                self.used -= self.resident.pop(v)
            self.resident[uid] = blocks
            self.used += blocks
        return hits


def hit_ratio(cache, trace: Iterable[Sequence[Unit]]) -> float:
    """Fraction of retrieved units that were resident, over a trace of requests."""
    n = h = 0
    for req in trace:
        r = cache.request(req)
        n += len(r)
        h += sum(r)
    return h / max(n, 1)
