"""Pins for the oracle's predictor (Algorithms 1-3, Eq. 1): a hand-worked example,
counting invariants, a Markov-chain closed form on planted traces, special cases."""
import os

import numpy as np
import pytest

import oracle as O
from datagen import stacks

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "cct_worked_example.txt")


def _rows(s):
    return [[int(v) for v in part.split()] for part in s.split(";")]


def _load_example():
    recs = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                key, val = line.split(":", 1)
                recs.append((key.strip(), val.strip()))
    return recs


def test_worked_example_functions():
    """Algorithm 1 counts and top-K rows, Algorithm 2 scores, Algorithm 3 updates."""
    recs = _load_example()
    E, K = 4, 2
    Co = np.zeros((E, E), dtype=np.uint32)
    it = iter(recs)
    key, val = next(it)
    assert key == "profile"
    last_f = None
    for pair in val.split(";"):
        e, f = (list(map(int, side.split())) for side in pair.split("->"))
        O.co_accumulate(Co, e, f)
        last_f = f
    key, val = next(it)
    assert key == "co" and Co.tolist() == _rows(val)
    ids, conf = O.cct_build(Co, K)
    assert ids.tolist() == _rows(next(it)[1])
    assert conf.tolist() == _rows(next(it)[1])
    ht = [int(v) for v in next(it)[1].split()]
    assert ht == last_f
    for key, val in it:
        assert key == "step"
        e, f = (list(map(int, side.split())) for side in val.split("->"))
        score, lit, mask = O.predict(E, K, e, ids, conf, ht)
        assert score.tolist() == [int(v) for v in next(it)[1].split()]
        assert np.flatnonzero(mask).tolist() == [int(v) for v in next(it)[1].split()]
        O.update(E, K, e, f, ids, conf)
        assert ids.tolist() == _rows(next(it)[1])
        assert conf.tolist() == _rows(next(it)[1])
        ht = f


def test_worked_example_state_machine():
    """The same example through the whole-stack state machine (L=2, P=4)."""
    recs = _load_example()
    p = O.Predictor(L=2, E=4, K=2, B=1, P=4, mode="st")
    prof = [[list(map(int, s.split())) for s in pair.split("->")] for pair in recs[0][1].split(";")]
    for e, f in prof:
        assert p.step(0, [e])["n_pred"][0] == 0
        p.step(1, [f])
    tb = p.tables()
    assert tb["built"] == 1 and tb["t"] == 4
    assert tb["Co"][0].tolist() == _rows(recs[1][1])
    assert tb["cct_id"][0].tolist() == _rows(recs[2][1])
    steps = [r for r in recs[5:]]
    for i in range(0, len(steps), 5):
        e, f = (list(map(int, s.split())) for s in steps[i][1].split("->"))
        out = p.step(0, [e])
        n = out["n_pred"][0]
        assert out["pred_ids"][0, :n].tolist() == [int(v) for v in steps[i + 2][1].split()]
        assert (out["pred_ids"][0, n:] == -1).all()
        p.step(1, [f])
        tb = p.tables()
        assert tb["cct_id"][0].tolist() == _rows(steps[i + 3][1])
        assert tb["cct_conf"][0].tolist() == _rows(steps[i + 4][1])
        assert tb["HT"][0, 1].tolist() == f and tb["HT"][0, 0].tolist() == e


def _stationary_recall(E, q):
    """Stationary recall of the K=1 single-slot confidence chain (states A0..A3: the slot
    holds the planted successor at confidence c; B0..B3: it holds another expert)."""
    h = (1.0 - q) / (E - 1)
    T = np.zeros((8, 8))
    A, B = (lambda c: c), (lambda c: 4 + c)
    for c in range(4):
        T[A(c), A(min(c + 1, 3))] += q
        T[A(c), A(c - 1) if c > 0 else B(2)] += 1 - q
        T[B(c), B(min(c + 1, 3))] += h
        if c > 0:
            T[B(c), B(c - 1)] += 1 - h
        else:
            T[B(c), A(2)] += q
            T[B(c), B(2)] += 1 - h - q
    w, v = np.linalg.eig(T.T)
    pi = np.real(v[:, np.argmin(abs(w - 1))])
    pi /= pi.sum()
    return q * (pi[A(2)] + pi[A(3)]) + h * (pi[B(2)] + pi[B(3)])


@pytest.mark.parametrize("E,q", [(8, 0.9), (8, 0.7), (16, 0.8), (8, 0.5)])
def test_planted_transition_converges_to_closed_form(E, q):
    """Spatial-only recall on a planted transition equals the chain's stationary value."""
    tokens, burn = 40000, 4000
    e, f, _ = stacks.planted_pair_trace(E, q, tokens, stream=E * 100 + int(q * 10))
    p = O.Predictor(L=2, E=E, K=1, B=1, P=0, mode="spatial")
    hit = 0
    for t in range(tokens):
        out = p.step(0, [[int(e[t])]])
        if t >= burn and out["n_pred"][0] == 1 and out["pred_ids"][0, 0] == int(f[t]):
            hit += 1
        assert out["n_pred"][0] <= 1
        p.step(1, [[int(f[t])]])
    want = _stationary_recall(E, q)
    assert abs(hit / (tokens - burn) - want) < 0.012, (hit / (tokens - burn), want)
    # the stationary value is below q because only confidences >= 2 predict
    assert want < q


def test_planted_transition_profiled_table_holds_successor():
    E, q = 8, 0.9
    e, f, pi = stacks.planted_pair_trace(E, q, 4000, stream=5)
    p = O.Predictor(L=2, E=E, K=1, B=1, P=4000, mode="spatial")
    for t in range(4000):
        p.step(0, [[int(e[t])]])
        p.step(1, [[int(f[t])]])
    tb = p.tables()
    assert tb["cct_id"][0, :, 0].tolist() == pi.tolist()
    assert (tb["cct_conf"] == 2).all()


def _run_trace(trace, E, P, mode):
    T, L, Bt, K = trace.shape
    p = O.Predictor(L=L, E=E, K=K, B=Bt, P=P, mode=mode)
    outs = []
    for t in range(T):
        for l in range(L):
            outs.append(p.step(l, trace[t, l]))
    return p, outs


@pytest.mark.parametrize("E,K,B", [(8, 2, 1), (60, 4, 3), (64, 6, 2), (128, 8, 4), (160, 8, 1)])
def test_invariants_random_traces(E, K, B):
    """Counting and range invariants on uniform random routing (shapes include the
    expert counts of the paper's Table 1)."""
    T, L, P = 40, 3, 12
    trace = stacks.random_topk_trace(E, K, T, L, B, stream=E + K).numpy()
    p = O.Predictor(L=L, E=E, K=K, B=B, P=P, mode="st")
    prev_pred = {}
    for t in range(T):
        for l in range(L):
            out = p.step(l, trace[t, l])
            tb = p.tables()
            # HT[l] holds this token's routing, HT[l+1..] still the previous token's
            assert (tb["HT"][:, l] == trace[t, l]).all()
            if l + 1 < L:
                want = trace[t - 1, l + 1] if t > 0 else -np.ones((B, K))
                assert (tb["HT"][:, l + 1] == want).all()
            for b in range(B):
                n = out["n_pred"][b]
                ids = out["pred_ids"][b, :n]
                assert n <= min(E, K * K + K) and (np.diff(ids) > 0).all()
                if t >= P or (t == P - 1 and l == L - 1):
                    nxt = (l + 1) % L
                    ht = tb["HT"][b, nxt]
                    assert set(ht[ht >= 0]) <= set(ids)      # Pred contains the valid HT
                else:
                    assert n == 0
            # queue = union of the per-sequence sets, ordered by score desc then id asc
            union = sorted(set(int(v) for b in range(B) for v in out["pred_ids"][b, :out["n_pred"][b]]))
            assert sorted(out["queue_ids"].tolist()) == union
            keys = list(zip(-out["queue_score"], out["queue_ids"]))
            assert keys == sorted(keys)
    tb = p.tables()
    # Algorithm 1: every profiling token adds K*K counts to each adjacent pair
    assert (tb["Co"].sum(axis=(1, 2)) == P * B * K * K).all()
    for pair in range(L - 1):
        times_routed = np.bincount(trace[:P, pair].ravel(), minlength=E)
        assert (tb["Co"][pair].sum(axis=1) == K * times_routed).all()
    assert tb["cct_conf"].max() <= 3
    srt = np.sort(tb["cct_id"].astype(int), axis=2)
    assert (np.diff(srt, axis=2) > 0).all()                  # no id twice in a row
    st = p.stats()
    assert st["steps"] == (T - P) * L * B and st["routed"] == st["steps"] * K
    assert 0 <= st["hits"] <= min(st["routed"], st["predicted"])


def test_constant_trace_recall_one_and_rows_converge():
    L, E, K = 3, 16, 4
    R = np.array([[[1, 5, 9, 12]], [[0, 2, 4, 6]], [[3, 7, 11, 15]]], dtype=np.int32)
    p = O.Predictor(L=L, E=E, K=K, B=1, P=0, mode="spatial")
    last = None
    for t in range(12):
        for l in range(L):
            last = p.step(l, R[l]) if l == 0 else last
            if l != 0:
                p.step(l, R[l])
    tb = p.tables()
    for pair in range(L - 1):
        for e in R[pair][0]:
            assert sorted(tb["cct_id"][pair, e].tolist()) == R[pair + 1][0].tolist()
            assert (tb["cct_conf"][pair, e] == 3).all()
    # spatial prediction for layer 1 is now exactly its routing (precision and recall 1)
    n = last["n_pred"][0]
    assert last["pred_ids"][0, :n].tolist() == R[1][0].tolist()
    p2 = O.Predictor(L=L, E=E, K=K, B=1, P=0, mode="st")
    for t in range(12):
        for l in range(L):
            p2.step(l, R[l])
    st = p2.stats()
    # every step after the first token is fully predicted (layer 0 through the history table)
    assert st["hits"] >= st["routed"] - L * K


def test_all_experts_routed_predicts_everything():
    E = K = 4
    p = O.Predictor(L=2, E=E, K=K, B=1, P=0, mode="st")
    ids = np.arange(E, dtype=np.int32)[None]
    p.step(0, ids), p.step(1, ids)
    out = p.step(0, ids)
    assert out["n_pred"][0] == E


def test_uniform_routing_temporal_overlap_matches_k2_over_n():
    """Random-routing baseline of the consecutive-token analysis: overlap = K^2/N,
    so history-table-only recall is K/N."""
    E, K, T = 32, 4, 6000
    trace = stacks.random_topk_trace(E, K, T, 1, 1, stream=77).numpy()
    overlap = np.mean([len(set(trace[t, 0, 0]) & set(trace[t - 1, 0, 0])) for t in range(1, T)])
    assert abs(overlap - K * K / E) < 0.05
    p = O.Predictor(L=1, E=E, K=K, B=1, P=0, mode="temporal")
    for t in range(T):
        p.step(0, trace[t, 0])
    st = p.stats()
    assert abs(st["hits"] / st["routed"] - K / E) < 0.02
    assert abs(st["predicted"] / st["steps"] - K) < 0.01


def test_modes_share_table_evolution_and_off_predicts_nothing():
    trace = stacks.random_topk_trace(24, 3, 30, 4, 2, stream=3).numpy()
    states = {}
    for mode in ("off", "temporal", "spatial", "st"):
        p, outs = _run_trace(trace, 24, P=8, mode=mode)
        states[mode] = p.export()
        if mode == "off":
            assert all(o["n_pred"].sum() == 0 for o in outs)
    assert len(set(states.values())) == 1


def test_batch_order_matters_but_is_sequential():
    """A batch of B sequences updates the shared CCT like B single steps in index order."""
    E, K, L = 12, 2, 2
    tr = stacks.random_topk_trace(E, K, 50, L, 3, stream=9).numpy()
    p = O.Predictor(L=L, E=E, K=K, B=3, P=5, mode="st")
    for t in range(50):
        for l in range(L):
            p.step(l, tr[t, l])
    tb = p.tables()
    # replay the runtime part by hand with the single-pair functions
    Co = np.zeros((E, E), dtype=np.uint32)
    for t in range(5):
        for b in range(3):
            O.co_accumulate(Co, tr[t, 0, b], tr[t, 1, b])
    ids, conf = O.cct_build(Co, K)
    for t in range(5, 50):
        for b in range(3):
            O.update(E, K, tr[t, 0, b], tr[t, 1, b], ids, conf)
    assert (tb["cct_id"][0] == ids).all() and (tb["cct_conf"][0] == conf).all()


def test_replacement_takes_lowest_missing_id_and_never_duplicates():
    E, K = 8, 3
    ids = np.array([[5, 6, 7]] * E, dtype=np.uint8)
    conf = np.zeros((E, K), dtype=np.uint8)
    O.update(E, K, [0], [1, 2, 6], ids, conf)
    # slot0 (5, conf 0, miss) -> 1; slot1 (6) is a hit -> conf 1; slot2 (7, miss) -> 2
    assert ids[0].tolist() == [1, 6, 2] and conf[0].tolist() == [2, 1, 2]
    ids = np.array([[1, 2, 7]] * E, dtype=np.uint8)
    conf = np.zeros((E, K), dtype=np.uint8)
    O.update(E, K, [3], [1, 2, 4], ids, conf)
    assert ids[3].tolist() == [1, 2, 4] and conf[3].tolist() == [1, 1, 2]
    # every routed expert already stored: the stale slot is left as it is
    ids = np.array([[1, 2, 7]] * E, dtype=np.uint8)
    conf = np.array([[0, 0, 0]] * E, dtype=np.uint8)
    O.update(E, K, [3], [1, 2], ids, conf)
    assert ids[3].tolist() == [1, 2, 7] and conf[3].tolist() == [1, 1, 0]
    assert ids[0].tolist() == [1, 2, 7]                      # other rows untouched


GOLDEN_B2 = os.path.join(os.path.dirname(__file__), "golden", "cct_batch2_example.txt")


def test_worked_example_batch_of_two_pins_queue_scores():
    """Hand-worked two-sequence steps: the prefetch queue carries the sum of the sequences'
    Eq. 1 scores (not their maximum, not one sequence's), ordered by (score descending, id
    ascending); the shared table is updated sequence 0 first."""
    recs = []
    with open(GOLDEN_B2) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                key, val = line.split(":", 1)
                recs.append((key.strip(), val.strip()))

    def queue(val):
        pairs = [p.split(":") for p in val.split()]
        return [int(a) for a, _ in pairs], [int(b) for _, b in pairs]

    def token(val):
        seqs = [[list(map(int, side.split())) for side in s.split("->")] for s in val.split("|")]
        return [s[0] for s in seqs], [s[1] for s in seqs]          # layer-0 routing, layer-1 routing

    E, K = 4, 2
    p = O.Predictor(L=2, E=E, K=K, B=2, P=2, mode="st")
    it = iter(recs)
    out1 = None
    for _ in range(2):                                             # profiling
        key, val = next(it)
        assert key == "token"
        r0, r1 = token(val)
        out0 = p.step(0, r0)
        assert out0["queue_ids"].size == 0 and (out0["n_pred"] == 0).all()
        out1 = p.step(1, r1)
    tb = p.tables()
    assert tb["built"] == 1 and tb["t"] == 2
    assert tb["cct_id"][0].tolist() == _rows(next(it)[1])
    assert tb["cct_conf"][0].tolist() == _rows(next(it)[1])
    key, val = next(it)
    assert key == "queue_next"
    ids, sc = queue(val)
    assert out1["queue_ids"].tolist() == ids and out1["queue_score"].tolist() == sc

    for key, val in it:
        assert key == "token"
        r0, r1 = token(val)
        tb = p.tables()
        want = [[int(v) for v in next(it)[1].split()] for _ in range(2)]
        for b in range(2):                                         # Algorithm 2 + Eq. 1 per sequence
            score, _, mask = O.predict(E, K, r0[b], tb["cct_id"][0].copy(), tb["cct_conf"][0].copy(),
                                       tb["HT"][b, 1].copy())
            assert score.tolist() == want[b]
        out0 = p.step(0, r0)
        ids, sc = queue(next(it)[1])
        assert out0["queue_ids"].tolist() == ids and out0["queue_score"].tolist() == sc
        for b in range(2):
            n = out0["n_pred"][b]
            assert out0["pred_ids"][b, :n].tolist() == [f for f in range(E) if want[b][f] >= 2]
        out1 = p.step(1, r1)
        assert p.tables()["cct_conf"][0].tolist() == _rows(next(it)[1])
        ids, sc = queue(next(it)[1])
        assert out1["queue_ids"].tolist() == ids and out1["queue_score"].tolist() == sc


def test_set_threshold_of_algorithm_2_follows_the_pinned_scores():
    """The threshold only cuts the pinned scores of the worked example at another value; the
    tables evolve identically; the sets are nested."""
    recs = _load_example()
    E, K = 4, 2
    prof = [[list(map(int, s.split())) for s in pair.split("->")] for pair in recs[0][1].split(";")]
    steps = recs[5:]
    ref_tables = None
    for thr in (1, 2, 3, 5, 7):
        p = O.Predictor(L=2, E=E, K=K, B=1, P=4, mode="st", threshold=thr)
        for e, f in prof:
            p.step(0, [e])
            p.step(1, [f])
        for i in range(0, len(steps), 5):
            e, f = (list(map(int, s.split())) for s in steps[i][1].split("->"))
            score = [int(v) for v in steps[i + 1][1].split()]
            out = p.step(0, [e])
            n = out["n_pred"][0]
            assert out["pred_ids"][0, :n].tolist() == [x for x in range(E) if score[x] >= thr], (thr, i)
            p.step(1, [f])
        tables = (p.tables()["cct_id"].tobytes(), p.tables()["cct_conf"].tobytes())
        assert ref_tables in (None, tables)
        ref_tables = tables
    # function level: the same scores, sets nested in the threshold
    ids, conf = O.cct_build(np.array(_rows(recs[1][1]), dtype=np.uint32), K)
    prev = None
    for thr in (1, 2, 3, 4, 6):
        score, _, mask = O.predict(E, K, [0, 2], ids, conf, [1, 3], threshold=thr)
        assert score.tolist() == [0, 2, 4, 6]
        assert np.flatnonzero(mask).tolist() == [f for f in range(E) if score[f] >= thr]
        assert prev is None or (mask <= prev).all()
        prev = mask


GOLDEN_LIVE = os.path.join(os.path.dirname(__file__), "golden", "cct_live_counts_example.txt")


def _load(path):
    recs = []
    with open(path) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                key, val = line.split(":", 1)
                recs.append((key.strip(), val.strip()))
    return recs


def test_live_count_replacement_worked_example():
    """Replacement by the largest live count (the open choice of Algorithm 3 taken another way):
    hand-derived counts and rows, through the single functions and through the state machine; the
    default rule ends with another row 0, so the two rules cannot be confused."""
    recs = _load(GOLDEN_LIVE)
    E, K = 4, 2
    prof = [[list(map(int, s.split())) for s in pair.split("->")] for pair in recs[0][1].split(";")]
    Co = np.zeros((E, E), dtype=np.uint32)
    for e, f in prof:
        O.co_accumulate(Co, e, f)
    assert Co.tolist() == _rows(recs[1][1])
    ids, conf = O.cct_build(Co, K)
    assert ids.tolist() == _rows(recs[2][1]) and conf.tolist() == _rows(recs[3][1])
    ids_low, conf_low = ids.copy(), conf.copy()
    p = O.Predictor(L=2, E=E, K=K, B=1, P=len(prof), mode="st", live_counts=True)
    for e, f in prof:
        p.step(0, [e]), p.step(1, [f])
    steps = recs[4:]
    for i in range(0, len(steps), 4):
        assert steps[i][0] == "step"
        e, f = (list(map(int, s.split())) for s in steps[i][1].split("->"))
        O.co_accumulate(Co, e, f)
        O.update(E, K, e, f, ids, conf, co=Co)
        O.update(E, K, e, f, ids_low, conf_low)
        p.step(0, [e]), p.step(1, [f])
        tb = p.tables()
        for got_co, got_id, got_cf in ((Co, ids, conf), (tb["Co"][0], tb["cct_id"][0], tb["cct_conf"][0])):
            assert got_co.tolist() == _rows(steps[i + 1][1]), i
            assert got_id.tolist() == _rows(steps[i + 2][1]), i
            assert got_cf.tolist() == _rows(steps[i + 3][1]), i
    assert ids_low[0].tolist() == [0, 1] and ids[0].tolist() == [1, 0]


def _update_by_counts_replay(E, K, prev, cur, rows, co):
    """Algorithm 3 with the live-count rule written another way: dictionaries per row, the
    candidates of a replacement sorted by (count descending, id ascending)."""
    for e in prev:
        row = rows[e]
        for c in range(K):
            g, cf = row[c]
            if g in cur:
                row[c] = (g, min(cf + 1, 3))
            elif cf > 0:
                row[c] = (g, cf - 1)
            else:
                held = {x for x, _ in row}
                cand = sorted((f for f in cur if f not in held), key=lambda f: (-int(co[e][f]), f))
                if cand:
                    row[c] = (cand[0], 2)


@pytest.mark.parametrize("E,K,B", [(6, 2, 1), (8, 3, 2), (16, 4, 3), (60, 4, 1), (128, 8, 2)])
def test_live_count_rule_against_a_replay_and_its_invariants(E, K, B):
    L, P, T = 3, 5, 60
    rng = np.random.default_rng(11 * E + K)
    p = O.Predictor(L, E, K, B, P, "st", live_counts=True)
    co = np.zeros((L - 1, E, E), dtype=np.int64)
    rows = None
    routed_rows = np.zeros((L - 1, E), dtype=np.int64)
    for t in range(T):
        prev = None
        for l in range(L):
            # skewed routing, so counts differ and replacements happen
            w = 1.0 / (1.0 + ((np.arange(E) * 7 + 3 * l + (t % 4)) % E))
            cur = np.stack([np.sort(rng.choice(E, K, replace=False, p=w / w.sum())) for _ in range(B)])
            p.step(l, cur)
            if l > 0:
                for b in range(B):
                    for e in prev[b]:
                        routed_rows[l - 1, e] += 1
                        for f in cur[b]:
                            co[l - 1, e, f] += 1
                    if t >= P:
                        _update_by_counts_replay(E, K, prev[b].tolist(), cur[b].tolist(), rows[l - 1], co[l - 1])
            prev = cur
        if t == P - 1:
            tb = p.tables()
            rows = [[[(int(tb["cct_id"][i, e, c]), int(tb["cct_conf"][i, e, c])) for c in range(K)]
                     for e in range(E)] for i in range(L - 1)]
    tb = p.tables()
    # counting never stops: K x K per sequence, pair and decode step; a row's sum = K x (times routed)
    assert (tb["Co"] == co).all()
    assert int(tb["Co"].sum()) == T * B * K * K * (L - 1)
    assert (tb["Co"].sum(axis=2) == K * routed_rows).all()
    for i in range(L - 1):
        for e in range(E):
            assert [g for g, _ in rows[i][e]] == tb["cct_id"][i, e].tolist(), (i, e)
            assert [c for _, c in rows[i][e]] == tb["cct_conf"][i, e].tolist(), (i, e)
            assert len(set(tb["cct_id"][i, e].tolist())) == K
    assert tb["cct_conf"].max() <= 3


def test_live_count_rule_with_one_expert_per_token_equals_the_default_rule():
    """K = 1: a replacement has at most one candidate (the routed expert), so both rules must keep
    the same tables; only the counts differ (frozen against live)."""
    L, E, P, T = 4, 8, 6, 80
    rng = np.random.default_rng(5)
    a, b = O.Predictor(L, E, 1, 1, P, "st"), O.Predictor(L, E, 1, 1, P, "st", live_counts=True)
    for t in range(T):
        for l in range(L):
            cur = rng.integers(0, E, size=(1, 1))
            ra, rb = a.step(l, cur), b.step(l, cur)
            assert (ra["pred_ids"] == rb["pred_ids"]).all()
    ta, tb = a.tables(), b.tables()
    assert (ta["cct_id"] == tb["cct_id"]).all() and (ta["cct_conf"] == tb["cct_conf"]).all()
    assert int(ta["Co"].sum()) == P * (L - 1) and int(tb["Co"].sum()) == T * (L - 1)


def test_live_count_rule_batch_is_the_sequences_in_index_order():
    """Counting and updating go sequence by sequence: a batch of two must equal the same two
    routings fed as two single steps of a one-sequence table (tables only; the history is per
    sequence)."""
    E, K = 8, 2
    prev = np.array([[0, 1], [0, 2]]); cur = np.array([[3, 5], [4, 5]])
    p = O.Predictor(2, E, K, 2, 0, "st", live_counts=True)
    # a predictor built from all-zero counts (P = 0) holds ids 0..K-1 at confidence 2 in every row
    ids_b, conf_b = np.tile(np.arange(K, dtype=np.uint8), (E, 1)), np.full((E, K), 2, dtype=np.uint8)
    co_b = np.zeros((E, E), dtype=np.uint32)
    for _ in range(4):
        p.step(0, prev), p.step(1, cur)
        for b in range(2):
            O.co_accumulate(co_b, prev[b], cur[b])
            O.update(E, K, prev[b], cur[b], ids_b, conf_b, co=co_b)
    tb = p.tables()
    assert (tb["Co"][0] == co_b).all() and (tb["cct_id"][0] == ids_b).all() and (tb["cct_conf"][0] == conf_b).all()
    assert ids_b[0].tolist() != [0, 1]          # replacements did happen in the shared row
