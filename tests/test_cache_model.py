"""Expert cache (Sec. 3.5, Algorithm 1): pins for the host model in ``oracle/cache_oracle.py`` and parity of the
library's bookkeeping-only cache (same policy, no device) with that model on seeded traces.  No GPU needed."""
import numpy as np
import pytest

from oracle.cache_oracle import CacheFull, ExpertCacheModel


# ------------------------------------------------------------------ pins of the model
def test_textbook_lru_trace():
    """3 slots, reference string 1 2 3 1 4 2 5 1 2 3 (one id per access), worked by hand for LRU:
    1 2 3 miss; 1 hit; 4 evicts 2; 2 evicts 3; 5 evicts 1; 1 evicts 4; 2 hit; 3 evicts 5."""
    m = ExpertCacheModel(1, 8, 3)
    outcome, victims = [], []
    for e in [1, 2, 3, 1, 4, 2, 5, 1, 2, 3]:
        before = set(m.expert[0])
        r = m.stage(0, [e])
        outcome.append("h" if r["hit"] else "m")
        gone = before - set(m.expert[0]) - {-1}
        victims += sorted(gone)
    assert "".join(outcome) == "mmmhmmmmhm"
    assert victims == [2, 3, 1, 4, 5]
    assert m.stats["hits"] == 2 and m.stats["on_demand"] == 8 and m.stats["evictions"] == 5
    assert m.stats["lookups"] == 10


def test_enough_slots_means_only_cold_misses():
    m = ExpertCacheModel(2, 6, 6)
    rng = np.random.default_rng(0)
    for _ in range(50):
        layer = int(rng.integers(0, 2))
        m.stage(layer, rng.choice(6, size=3, replace=False).tolist())
    assert m.stats["on_demand"] <= 12 and m.stats["evictions"] == 0
    assert m.stats["hits"] + m.stats["on_demand"] == m.stats["lookups"] == 150


def test_prefetch_semantics():
    m = ExpertCacheModel(1, 16, 4)
    m.begin_step()
    assert m.prefetch(0, [3, 5]) == [3, 5]
    assert m.prefetch(0, [5, 3]) == []                      # cached or in flight: never re-issued
    r = m.stage(0, [5, 7])                                  # 5 was predicted (used), 7 is a miss, 3 is unused
    assert r == {"hit": [5], "load": [7]}
    assert m.stats["prefetch_used"] == 1 and m.stats["on_demand"] == 1
    m.begin_step()                                          # 3 was prefetched and never used: wasted
    assert m.stats["prefetch_wasted"] == 1
    assert m.stats["prefetch_issued"] == m.stats["prefetch_used"] + m.stats["prefetch_wasted"]
    # a prefetch never evicts a pending prefetch: with every slot in P further hints are dropped
    m2 = ExpertCacheModel(1, 16, 2)
    assert m2.prefetch(0, [1, 2, 3]) == [1, 2]
    # ... but an on-demand load may, and that prefetch counts as wasted
    m2.stage(0, [9])
    assert m2.stats["prefetch_wasted"] == 1 and m2.slot_of(0, 9) >= 0
    # the least recently used unprotected slot goes first
    m3 = ExpertCacheModel(1, 16, 3)
    m3.stage(0, [1]); m3.stage(0, [2]); m3.stage(0, [3]); m3.stage(0, [1])
    m3.prefetch(0, [4])
    assert sorted(m3.expert[0]) == [1, 3, 4]
    with pytest.raises(CacheFull):
        m3.stage(0, [5, 6, 7, 8])


def test_a_call_never_evicts_what_it_needs():
    m = ExpertCacheModel(1, 32, 4)
    rng = np.random.default_rng(1)
    for _ in range(200):
        ids = rng.choice(32, size=int(rng.integers(1, 5)), replace=False).tolist()
        if rng.random() < 0.4:
            m.prefetch(0, rng.choice(32, size=3, replace=False).tolist())
        m.stage(0, ids)
        assert all(m.slot_of(0, e) >= 0 for e in ids)
        held = [e for e in m.expert[0] if e >= 0]
        assert len(held) == len(set(held))
        if rng.random() < 0.2:
            m.begin_step()
    m.begin_step()
    assert m.stats["prefetch_issued"] == m.stats["prefetch_used"] + m.stats["prefetch_wasted"]


# ------------------------------------------------------------------ the library's policy against the model
def test_library_bookkeeping_cache_matches_model():
    from paper_2607_24434_b200 import binding
    L, E, S = 3, 24, 5
    rng = np.random.default_rng(7)
    cache = binding.ExpertCache(None, L, E, S, 128 * 4)
    for l in range(L):
        for e in range(E):
            cache.register_fake(l, e)
    m = ExpertCacheModel(L, E, S)
    for step in range(300):
        op = rng.random()
        layer = int(rng.integers(0, L))
        if op < 0.15:
            cache.begin_step(); m.begin_step()
        elif op < 0.5:
            ids = rng.choice(E, size=int(rng.integers(1, 7)), replace=False).tolist()
            cache.prefetch(layer, ids); m.prefetch(layer, ids)
        else:
            ids = rng.choice(E, size=int(rng.integers(1, S + 1)), replace=False).tolist()
            cache.stage(layer, ids); m.stage(layer, ids)
        for l in range(L):
            for e in range(E):
                assert cache.query(l, e)[0] == m.slot_of(l, e), (step, l, e)
    st = cache.stats()
    for key in ("lookups", "hits", "on_demand", "prefetch_issued", "prefetch_used", "prefetch_wasted", "evictions"):
        assert st[key] == m.stats[key], key
    assert st["bytes_h2d"] == m.stats["loads"] * 128 * 4
    # errors are reported, not raised inside the library
    with pytest.raises(binding.DxError) as err:
        cache.stage(0, list(range(S + 1)))
    assert err.value.status == 7                             # DX_ERR_CACHE_FULL
    fresh = binding.ExpertCache(None, 1, 8, 2, 128)
    with pytest.raises(binding.DxError) as err:
        fresh.stage(0, [3])                                  # no host blob registered
    assert err.value.status == 5                             # DX_ERR_NOT_RESIDENT
    with pytest.raises(binding.DxError) as err:
        fresh.wait(0, [3])                                   # wait never loads
    assert err.value.status == 5
    with pytest.raises(binding.DxError) as err:
        fresh.prefetch(0, [99])
    assert err.value.status == 1
    cache.close(); fresh.close()


def test_union_waves_keep_what_is_held():
    """4 slots holding 1, 5, 9 (in that age order) and a block that needs 0..5: the held experts go first, so none of
    them is evicted before it is used -- worked by hand: wave 1 = [1, 5, 0, 2] (two hits, two loads, the loads take
    the free slot and then the oldest untouched one, 9), wave 2 = [3, 4] evicts the two oldest of wave 1."""
    m = ExpertCacheModel(1, 16, 4)
    for e in (1, 5, 9):
        m.stage(0, [e])
    base = dict(m.stats)
    waves = m.stage_union(0, [0, 1, 2, 3, 4, 5])
    assert waves == [[1, 5, 0, 2], [3, 4]]
    assert m.stats["hits"] - base["hits"] == 2 and m.stats["on_demand"] - base["on_demand"] == 4
    assert sorted(m.expert[0]) == [0, 2, 3, 4]             # 1 and 5 (oldest stamps of wave 1) made room for 3 and 4
    # ascending waves would have been [0,1,2,3] then [4,5]: loading 0, 2, 3 evicts 5 before its wave -> one hit fewer
    n = ExpertCacheModel(1, 16, 4)
    for e in (1, 5, 9):
        n.stage(0, [e])
    b2 = dict(n.stats)
    n.stage(0, [0, 1, 2, 3]); n.stage(0, [4, 5])
    assert n.stats["hits"] - b2["hits"] == 1
