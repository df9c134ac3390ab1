"""Host model of the accelerator expert cache of Sec. 3.5 / Algorithm 1.  TEST INFRASTRUCTURE ONLY.

Plain bookkeeping, no arithmetic of the method and no code shared with the CUDA library: per layer S slots;
C = experts held in slots, P = experts prefetched since the step began and not used yet (Algorithm 1 starts each
step with P empty).  The paper fixes only the outline (prefetch what is predicted and neither cached nor in
flight; wait for the useful transfers; load misses on demand; a prefetched expert that is used avoids a stall,
one that is not used is wasted bandwidth); the concrete policy below is the stated reading:

  * every use, prefetch or load stamps the slot with a global counter; "least recently used" = smallest stamp;
  * ``prefetch``: an id already in a slot is skipped; otherwise take the lowest free slot, else the LRU slot that
    is not in P, else drop the hint (a prefetch never evicts another pending prefetch);
  * ``stage`` (verification reaching the layer): ids already in slots are hits (a hit on a member of P is a
    *used* prefetch and leaves P); then misses, in the order given, take the lowest free slot, else the LRU slot
    outside P that this call has not touched, else the LRU member of P this call has not touched (a *wasted*
    prefetch); more ids than slots is an error;
  * ``begin_step``: what is still in P was prefetched and never used: wasted; P becomes empty.

Pinned by tests/test_cache_model.py (hand-worked LRU traces, invariants, hit/waste bookkeeping identities).
"""
from __future__ import annotations

from typing import Dict, List, Sequence


class CacheFull(Exception):
    pass


class ExpertCacheModel:
    def __init__(self, n_layers: int, n_experts: int, slots: int):
        self.L, self.E, self.S = n_layers, n_experts, slots
        self.expert = [[-1] * slots for _ in range(n_layers)]
        self.stamp = [[0] * slots for _ in range(n_layers)]
        self.in_p = [[False] * slots for _ in range(n_layers)]
        self.clock = 0
        self.stats: Dict[str, int] = dict(lookups=0, hits=0, on_demand=0, prefetch_issued=0, prefetch_used=0,
                                          prefetch_wasted=0, evictions=0, loads=0)

    def slot_of(self, layer: int, e: int) -> int:
        return self.expert[layer].index(e) if e in self.expert[layer] else -1

    def _tick(self) -> int:
        self.clock += 1
        return self.clock

    def _pick(self, layer: int, touched: set, allow_p: bool):
        for s in range(self.S):
            if self.expert[layer][s] < 0 and s not in touched:
                return s, False
        cands = [s for s in range(self.S) if s not in touched and not self.in_p[layer][s]]
        if cands:
            return min(cands, key=lambda s: (self.stamp[layer][s], s)), False
        if allow_p:
            cands = [s for s in range(self.S) if s not in touched]
            if cands:
                return min(cands, key=lambda s: (self.stamp[layer][s], s)), True
        return -1, False

    def _load(self, layer: int, s: int, e: int, as_prefetch: bool) -> None:
        if self.expert[layer][s] >= 0:
            self.stats["evictions"] += 1
        self.expert[layer][s] = e
        self.in_p[layer][s] = as_prefetch
        self.stamp[layer][s] = self._tick()
        self.stats["loads"] += 1

    def begin_step(self) -> None:
        for l in range(self.L):
            for s in range(self.S):
                if self.in_p[l][s]:
                    self.in_p[l][s] = False
                    self.stats["prefetch_wasted"] += 1

    def prefetch(self, layer: int, ids: Sequence[int]) -> List[int]:
        issued = []
        for e in ids:
            if self.slot_of(layer, e) >= 0:
                continue
            s, _ = self._pick(layer, set(), allow_p=False)
            if s < 0:
                continue
            self._load(layer, s, e, True)
            self.stats["prefetch_issued"] += 1
            issued.append(e)
        return issued

    def stage(self, layer: int, ids: Sequence[int]) -> Dict[str, List[int]]:
        if len(ids) > self.S:
            raise CacheFull()
        touched: set = set()
        res = {"hit": [], "load": []}
        for e in ids:
            s = self.slot_of(layer, e)
            if s >= 0 and s not in touched:
                self.stats["lookups"] += 1
                self.stats["hits"] += 1
                if self.in_p[layer][s]:
                    self.in_p[layer][s] = False
                    self.stats["prefetch_used"] += 1
                self.stamp[layer][s] = self._tick()
                touched.add(s)
                res["hit"].append(e)
        for e in ids:
            if self.slot_of(layer, e) >= 0:
                continue
            s, from_p = self._pick(layer, touched, allow_p=True)
            if s < 0:
                raise CacheFull()
            if from_p:
                self.stats["prefetch_wasted"] += 1
                self.in_p[layer][s] = False
            self.stats["lookups"] += 1
            self.stats["on_demand"] += 1
            self._load(layer, s, e, False)
            touched.add(s)
            res["load"].append(e)
        return res

    def stage_union(self, layer: int, union: Sequence[int]) -> List[List[int]]:
        """A verification block whose expert set (Eq. 2, ascending ids) may exceed the slots: it is evaluated in
        waves of at most S experts, the ones already held first (so that no load of this block can evict them
        before they are used), then the missing ones by ascending id; each wave is one ``stage``.  Returns the
        waves.  (The paper does not say what happens when a block needs more experts than the accelerator holds;
        this is the stated reading.)"""
        held = [e for e in union if self.slot_of(layer, e) >= 0]
        missing = [e for e in union if self.slot_of(layer, e) < 0]
        order = held + missing
        waves = [order[i:i + self.S] for i in range(0, len(order), self.S)]
        for w in waves:
            self.stage(layer, w)
        return waves
