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


# ---- use-history policy (window > 0) and the floor on prefetch victims --------------------------

class _Replay:
    """The same policy written another way (dictionaries, sorting the candidates), to replay
    traces against the C model."""

    def __init__(self, S, L, E, W, floor, by_turn=False):
        self.S, self.L, self.E, self.W, self.floor, self.by_turn = S, L, E, W, floor, by_turn
        self.layer = 0
        self.slot_key = [None] * S
        self.key_slot, self.stamp, self.hist, self.unused = {}, [-1] * S, {}, [False] * S
        self.clock = 0
        self.count = dict(hits=0, misses=0, pf_issued=0, pf_useful=0, pf_wasted=0, pf_dropped=0, pf_resident=0)

    def uses(self, s):
        k = self.slot_key[s]
        return -1 if k is None else bin(self.hist.get(k, 0)).count("1")

    def wait(self, s):
        k = self.slot_key[s]
        if not self.by_turn or k is None:
            return 0
        return (k[0] - self.layer) % self.L or self.L

    def victim(self, guard):
        cand = [s for s in range(self.S) if s not in guard]
        return min(cand, key=lambda s: (self.uses(s), -self.wait(s), self.stamp[s], s)) if cand else None

    def place(self, s, key, by_prefetch):
        old = self.slot_key[s]
        if old is not None:
            del self.key_slot[old]
            self.count["pf_wasted"] += self.unused[s]
        self.slot_key[s], self.key_slot[key] = key, s
        self.stamp[s], self.unused[s] = self.clock, by_prefetch

    def step(self, layer, U, nxt, Q, limit):
        self.layer = layer
        mask = (1 << self.W) - 1
        for k in list(self.hist):
            if k[0] == layer:
                self.hist[k] = (self.hist[k] << 1) & mask
        guard = {self.key_slot[(layer, e)] for e in U if (layer, e) in self.key_slot}
        u_slot, u_loaded = [], []
        for e in U:
            key = (layer, e)
            if self.W:
                self.hist[key] = self.hist.get(key, 0) | 1
            if key in self.key_slot:
                s = self.key_slot[key]
                self.count["hits"] += 1
                self.count["pf_useful"] += self.unused[s]
                self.unused[s] = False
                self.stamp[s] = self.clock
                u_loaded.append(0)
            else:
                s = self.victim(guard)
                self.count["misses"] += 1
                self.place(s, key, False)
                guard.add(s)
                u_loaded.append(1)
            u_slot.append(s)
        guard |= {self.key_slot[(nxt, f)] for f in Q if (nxt, f) in self.key_slot}
        q_slot, issued = [], 0
        for f in Q:
            key = (nxt, f)
            if key in self.key_slot:
                self.count["pf_resident"] += 1
                q_slot.append(-1)
                continue
            s = None if (limit and issued >= limit) else self.victim(guard)
            if s is not None and self.floor >= 0 and self.uses(s) > self.floor:
                s = None
            if s is None:
                self.count["pf_dropped"] += 1
                q_slot.append(-1)
                continue
            self.place(s, key, True)
            guard.add(s)
            self.count["pf_issued"] += 1
            issued += 1
            q_slot.append(s)
        self.clock += 1
        return u_slot, u_loaded, q_slot


def test_use_history_policy_matches_a_replay_written_another_way():
    E, K, T, L, B = 24, 3, 80, 3, 2
    tr = stacks.random_topk_trace(E, K, T, L, B, stream=9).numpy()
    for W, floor, limit, S, turn in ((4, -1, 0, 20, False), (16, 0, 2, 30, True), (8, 1, 0, 12, False),
                                     (0, -1, 3, 16, False), (16, -1, 0, 14, True), (0, -1, 2, 18, True)):
        p = O.Predictor(L, E, K, B, P=6, mode="st")
        c = O.CacheModel(S, L, E, window=W, floor=floor, by_turn=turn)
        r = _Replay(S, L, E, W, floor, turn)
        for t in range(T):
            for l in range(L):
                q = p.step(l, tr[t, l])["queue_ids"].tolist()
                U = np.unique(tr[t, l]).tolist()
                out = c.step(l, U, (l + 1) % L, q, limit=limit)
                u_slot, u_loaded, q_slot = r.step(l, U, (l + 1) % L, q, limit)
                assert out["u_slot"].tolist() == u_slot and out["u_loaded"].tolist() == u_loaded, (W, t, l)
                assert out["q_slot"].tolist() == q_slot, (W, t, l)
        assert c.stats() == r.count, W
        want = [-1 if k is None else k[0] * E + k[1] for k in r.slot_key]
        assert c.tags().tolist() == want


def test_use_counts_outrank_recency_hand_walked():
    """One layer, two slots, window 4.  Expert 0 is routed twice, then 1, then 2: the victim for 2
    is expert 1 (one use in its window) although it is the more recent; plain LRU takes expert 0."""
    for W, evicted in ((4, 1), (0, 0)):
        c = O.CacheModel(2, 1, 4, window=W)
        for e in (0, 0, 1):
            c.step(0, [e], 0, [])
        assert sorted(c.tags().tolist()) == [0, 1]
        out = c.step(0, [2], 0, [])
        assert out["u_loaded"].tolist() == [1]
        assert sorted(c.tags().tolist()) == sorted({0, 1, 2} - {evicted})
    # the window forgets: after four more turns without expert 0 its count is zero again
    c = O.CacheModel(2, 1, 4, window=4)
    for e in (0, 0, 1, 1, 1, 1, 1):
        c.step(0, [e], 0, [])
    c.step(0, [2], 0, [])
    assert sorted(c.tags().tolist()) == [1, 2]


def test_cyclic_walk_larger_than_the_cache_thrashes_lru_but_not_turn_order():
    """A decode step walks the layers in a fixed cycle.  With more keys per cycle than slots LRU
    evicts every key just before its next turn; evicting the key whose turn is furthest keeps a
    resident subset."""
    L, E, S, T = 6, 8, 20, 40           # every step routes 4 fixed experts per layer: 24 keys > 20 slots
    hits = {}
    for turn in (False, True):
        c = O.CacheModel(S, L, E, window=8, by_turn=turn)
        for t in range(T):
            for l in range(L):
                c.step(l, [0, 1, 2, 3], (l + 1) % L, [])
        hits[turn] = c.stats()["hits"]
    assert hits[False] == 0                      # equal counts everywhere: recency decides, which is LRU
    assert hits[True] >= (T - 2) * (S - 4 - 4)   # all but a rotating handful of slots keep their key


def test_prefetch_floor_only_takes_slots_without_recent_use():
    c = O.CacheModel(4, 2, 8, window=8, floor=0)
    c.step(0, [0, 1], 1, [])                      # two slots used, two empty
    out = c.step(1, [0], 0, [5, 6, 7])            # demand load takes an empty slot; one empty slot left for a prefetch
    assert (out["q_slot"] >= 0).sum() == 1
    st = c.stats()
    assert (st["pf_issued"], st["pf_dropped"]) == (1, 2)
    # a prefetched, never used key has no uses: it may be replaced by the next prefetch
    out = c.step(0, [0, 1], 1, [2])
    assert (out["q_slot"] >= 0).sum() == 1 and c.stats()["pf_wasted"] == 1
    # without the floor the same queue evicts keys that were in use
    d = O.CacheModel(4, 2, 8, window=8, floor=-1)
    d.step(0, [0, 1], 1, [])
    out = d.step(1, [0], 0, [5, 6, 7])
    assert out["q_slot"].tolist() == [3, 0, 1]    # the empty slot, then the two experts layer 0 has just used
    assert d.stats()["pf_issued"] == 3
