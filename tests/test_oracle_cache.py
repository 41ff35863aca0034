"""Pins for the oracle's integer cache model (verification, miss loading, prefetch)."""
from collections import OrderedDict

import numpy as np

import oracle as O
from datagen import stacks


def _trace(E, K, T, L, B, stream):
    tr = stacks.random_topk_trace(E, K, T, L, B, stream=stream).numpy()
    return [[np.unique(tr[t, l]) for l in range(L)] for t in range(T)]


def test_unbounded_cache_misses_only_on_first_touch():
    E, K, T, L = 16, 2, 30, 3
    tr = _trace(E, K, T, L, 2, 1)
    c = O.CacheModel(L * E, L, E)
    seen, hits, misses = set(), 0, 0
    for t in range(T):
        for l in range(L):
            out = c.step(l, tr[t][l], (l + 1) % L, [])
            for e, loaded in zip(tr[t][l], out["u_loaded"]):
                assert bool(loaded) == ((l, int(e)) not in seen)
                hits += (l, int(e)) in seen
                misses += (l, int(e)) not in seen
                seen.add((l, int(e)))
    st = c.stats()
    assert st["hits"] == hits and st["misses"] == misses and st["pf_issued"] == 0
    assert sorted(t for t in c.tags() if t >= 0) == sorted(l * E + e for l, e in seen)


def test_lru_without_prefetch_matches_ordered_dict_model():
    """No prefetch, one routed expert per step: the model is textbook LRU."""
    E, L, S, T = 10, 2, 5, 400
    tr = _trace(E, 1, T, L, 1, 2)
    c = O.CacheModel(S, L, E)
    lru, misses = OrderedDict(), 0
    for t in range(T):
        for l in range(L):
            key = (l, int(tr[t][l][0]))
            out = c.step(l, tr[t][l], (l + 1) % L, [])
            if key in lru:
                lru.move_to_end(key)
                assert out["u_loaded"][0] == 0
            else:
                misses += 1
                if len(lru) == S:
                    lru.popitem(last=False)
                lru[key] = True
                assert out["u_loaded"][0] == 1
    assert c.stats()["misses"] == misses
    assert sorted(t for t in c.tags() if t >= 0) == sorted(l * E + e for l, e in lru)


def test_prefetch_accounting_and_protection():
    E, L, S = 8, 2, 4
    c = O.CacheModel(S, L, E)
    # step 0: layer 0 routes {0,1}; prefetch {2,3,4} for layer 1: only two free slots remain
    out = c.step(0, [0, 1], 1, [2, 3, 4])
    assert out["u_slot"].tolist() == [0, 1] and out["u_loaded"].tolist() == [1, 1]
    assert out["q_slot"].tolist() == [2, 3, -1]
    st = c.stats()
    assert (st["misses"], st["pf_issued"], st["pf_dropped"]) == (2, 2, 1)
    # step 1: layer 1 routes {2,5}: 2 was prefetched (useful), 5 is a demand miss that must not
    # evict slot 2 (needed now); LRU victim is slot 0 (stamp 0, lowest index)
    out = c.step(1, [2, 5], 0, [0, 1])
    assert out["u_loaded"].tolist() == [0, 1] and out["u_slot"].tolist() == [2, 0]
    st = c.stats()
    assert st["hits"] == 1 and st["pf_useful"] == 1 and st["misses"] == 3
    # queued 0 was just evicted -> prefetched again into the LRU unguarded slot; queued 1 is
    # resident and guarded.  Victim candidates: slot 3 (expert (1,3), prefetched, unused).
    assert out["q_slot"].tolist() == [3, -1]
    st = c.stats()
    assert st["pf_wasted"] == 1 and st["pf_resident"] == 1 and st["pf_issued"] == 3


def test_prefetch_limit_and_routed_overflow():
    c = O.CacheModel(8, 1, 16)
    out = c.step(0, [0], 0, [1, 2, 3, 4], limit=2)
    assert (out["q_slot"] >= 0).sum() == 2 and c.stats()["pf_dropped"] == 2
    small = O.CacheModel(2, 1, 16)
    try:
        small.step(0, [0, 1, 2], 0, [])
        raised = False
    except AssertionError:
        raised = True
    assert raised


def test_stack_cache_counts_are_consistent():
    """hits + misses = distinct routed experts over all steps; useful + wasted <= issued."""
    E, K, T, L, B = 32, 4, 60, 4, 2
    tr = stacks.random_topk_trace(E, K, T, L, B, stream=5).numpy()
    p = O.Predictor(L, E, K, B, P=10, mode="st")
    c = O.CacheModel(40, L, E)
    distinct = 0
    for t in range(T):
        for l in range(L):
            q = p.step(l, tr[t, l])["queue_ids"]
            U = np.unique(tr[t, l])
            distinct += U.size
            c.step(l, U, (l + 1) % L, q, limit=6)
    st = c.stats()
    assert st["hits"] + st["misses"] == distinct
    assert st["pf_useful"] + st["pf_wasted"] <= st["pf_issued"]
    tags = c.tags()
    live = tags[tags >= 0]
    assert len(set(live.tolist())) == live.size
