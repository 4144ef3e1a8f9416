"""CPU model of the cluster cache of a two-tier setup (test infrastructure; nothing in the product imports it).

Section 6 of the paper keeps a cache of whole clusters in fast memory over the full KV store in slow memory, and
Section 6.2 gives the replacement policy as two principles: small clusters are the ones worth caching, and clusters
that were updated recently are retained.  The paper prints no algorithm for it.  This model fixes one, step by step,
so that the counters of an implementation can be compared with it exactly:

  * the cache of one unit has `frames` page frames of PAGE entries; a cluster of n entries occupies ceil(n / PAGE);
  * `retrieve(selected, size)` is one decode step: every selected cluster is
      - a HIT when a copy exists that was made after the cluster's last split and at its present size;
      - GROWN when such a copy exists but entries were appended since: the page that was the last one at copy time is
        copied again if it was not full (only the rows added since), and one frame is taken per page the cluster has
        gained;
      - MISSING otherwise: a copy from before a split is dropped first, then every page is copied into new frames;
  * when the free frames do not cover what the step needs, whole clusters NOT selected in this step are evicted until
    they do, in this order: copies made void by a split; then clusters unchanged since they were copied -- more pages
    first, least recently used first among equals, lower id first among those; then clusters that took appends since
    they were copied (same sub-order).  If nothing is left to evict the step fails (`CacheTooSmall`);
  * `note_split(j)` records that cluster id j went through a split (its rows were rearranged).

parity unpinned against the paper (it prints neither an algorithm nor a worked example for the policy); the model is
pinned by hand-worked sequences in tests/test_cluster_cache_model.py.
"""
from __future__ import annotations

from typing import Dict, Iterable, Mapping

PAGE = 32


class CacheTooSmall(RuntimeError):
    pass


def pages(n: int) -> int:
    return (n + PAGE - 1) // PAGE


class ClusterCacheModel:
    def __init__(self, frames: int, order: str = "small-first"):
        # order "lru" is a comparison policy only (void copies, then least recently used, whatever the size): it shows
        # what Section 6.2's first principle buys on a given stream; the library implements "small-first"
        assert order in ("small-first", "lru")
        self.order = order
        self.frames = frames
        self.free = frames
        self.copies: Dict[int, dict] = {}       # id -> {"n": size at copy time, "ver": splits seen then, "last": turn}
        self.ver: Dict[int, int] = {}
        self.clock = 0
        self.c = {"pages_fetched": 0, "clusters_hit": 0, "clusters_fetched": 0, "clusters_refreshed": 0,
                  "clusters_evicted": 0, "copies_dropped_stale": 0, "rows_fetched": 0}

    def note_split(self, j: int) -> None:
        self.ver[j] = self.ver.get(j, 0) + 1

    def _drop(self, j: int) -> None:
        self.free += pages(self.copies[j]["n"])
        del self.copies[j]

    def retrieve(self, selected: Iterable[int], size: Mapping[int, int]) -> None:
        self.clock += 1
        grown, missing, need = [], [], 0
        for j in selected:
            j = int(j)
            n = int(size[j])
            cp = self.copies.get(j)
            current = cp is not None and cp["ver"] == self.ver.get(j, 0)
            if current and n == cp["n"]:
                cp["last"] = self.clock
                self.c["clusters_hit"] += 1
            elif current and n > cp["n"]:
                cp["last"] = self.clock
                need += pages(n) - pages(cp["n"])
                grown.append(j)
            else:
                need += pages(n)
                missing.append(j)
        for j in missing:
            if j in self.copies:
                self._drop(j)
                self.c["copies_dropped_stale"] += 1
        while self.free < need:
            best = None
            for j, cp in self.copies.items():
                if cp["last"] == self.clock:
                    continue
                if cp["ver"] != self.ver.get(j, 0):
                    cls = 0
                elif int(size[j]) == cp["n"]:
                    cls = 1
                else:
                    cls = 2
                if self.order == "lru":
                    key = (0 if cls == 0 else 1, 0, cp["last"], j)
                else:
                    key = (cls, -pages(cp["n"]), cp["last"], j)
                if best is None or key < best:
                    best = key
            if best is None:
                raise CacheTooSmall(f"{need} frames needed, {self.free} free, nothing left to evict")
            self._drop(best[3])
            self.c["copies_dropped_stale" if best[0] == 0 else "clusters_evicted"] += 1
        for j in grown:
            cp = self.copies[j]
            n = int(size[j])
            extra = pages(n) - pages(cp["n"])
            self.c["pages_fetched"] += extra + (1 if cp["n"] % PAGE != 0 else 0)
            self.c["clusters_refreshed"] += 1
            self.c["rows_fetched"] += n - cp["n"]         # only the entries appended since the copy travel
            self.free -= extra
            cp["n"] = n
        for j in missing:
            n = int(size[j])
            self.c["pages_fetched"] += pages(n)
            self.c["clusters_fetched"] += 1
            self.c["rows_fetched"] += n
            self.free -= pages(n)
            self.copies[j] = {"n": n, "ver": self.ver.get(j, 0), "last": self.clock}

    @property
    def frames_in_use(self) -> int:
        return self.frames - self.free
