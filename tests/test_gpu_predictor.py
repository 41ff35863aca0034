"""GPU predictor kernel vs the oracle's Algorithms 1-3 on replayed routing traces: predicted
ids, exported tables and counters must be bit-exact."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2606_15453_b200 as P
from datagen import stacks

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _replay(L, E, K, B, P_tok, mode, trace, check_every=7, threshold=2, live_counts=False):
    """trace: int32 [T][L][B][K].  Runs both sides step by step."""
    st = P.Stack(L, E, K, 64, 64, max_batch=B, dtype="f32", profile_tokens=P_tok, mode=mode)
    if threshold != 2:
        st.set_predict_threshold(threshold)
    if live_counts:
        st.set_replacement_rule(True)
    orc = O.Predictor(L, E, K, B, P_tok, mode, threshold=threshold, live_counts=live_counts)
    pred = torch.empty(B, st.max_pred, dtype=torch.int32, device=DEV)
    npred = torch.empty(B, dtype=torch.int32, device=DEV)
    tr = torch.from_numpy(trace).to(DEV)
    for t in range(trace.shape[0]):
        for l in range(L):
            st.predictor_step(l, tr[t, l].contiguous(), pred, npred)
            o = orc.step(l, trace[t, l])
            if (t * L + l) % check_every == 0 or t == trace.shape[0] - 1:
                torch.cuda.synchronize()
                assert npred.cpu().numpy().tolist() == o["n_pred"].tolist(), (t, l)
                assert (pred.cpu().numpy() == o["pred_ids"]).all(), (t, l)
        if t % 5 == 0 or t == trace.shape[0] - 1:
            assert st.export_state() == orc.export(), f"state differs after token {t}"
    s, so = st.stats(), orc.stats()
    assert (s["runtime_steps"], s["routed"], s["predicted"], s["hits"]) == \
        (so["steps"], so["routed"], so["predicted"], so["hits"])
    assert s["decode_steps"] == trace.shape[0]
    st.close()
    return so


@pytest.mark.parametrize("E,K,B,L,mode", [
    (8, 2, 1, 4, "st"), (60, 4, 3, 3, "st"), (64, 6, 8, 3, "st"), (128, 8, 16, 3, "st"),
    (160, 8, 2, 2, "st"), (256, 8, 4, 2, "st"), (128, 8, 32, 2, "spatial"),
    (64, 6, 2, 3, "temporal"), (16, 4, 2, 3, "off"), (12, 12, 2, 2, "st"), (40, 1, 5, 1, "st"),
    (32, 16, 3, 2, "st")])
def test_predictor_replay_random_traces(E, K, B, L, mode):
    T, P_tok = 36, 9
    trace = stacks.random_topk_trace(E, K, T, L, B, stream=E * 7 + K).numpy()
    _replay(L, E, K, B, P_tok, mode, trace)


@pytest.mark.parametrize("threshold", [1, 3, 5])
def test_predictor_replay_with_another_set_threshold(threshold):
    """The threshold sweep of the ablation: Algorithm 2's set at a threshold other than binary 10,
    stand-alone predictor kernel, bit-exact against the oracle."""
    E, K, B, L = 64, 6, 4, 3
    trace = stacks.random_topk_trace(E, K, 30, L, B, stream=77).numpy()
    so = _replay(L, E, K, B, 8, "st", trace, check_every=3, threshold=threshold)
    assert so["predicted"] > 0


@pytest.mark.parametrize("E,K,B,L", [(8, 2, 1, 4), (60, 4, 3, 3), (64, 6, 8, 3), (128, 8, 16, 3), (256, 8, 4, 2),
                                     (12, 12, 2, 2), (40, 1, 5, 2), (32, 16, 3, 2)])
def test_predictor_replay_with_live_count_replacement(E, K, B, L):
    """Algorithm 3 with the new candidate taken by the largest live co-activation count: counts
    (they keep growing at run time), tables and predictions bit-exact against the oracle.  Skewed
    traces, so that counts differ and confidences reach zero."""
    T = 40
    base = stacks.random_topk_trace(E, K, T, L, B, stream=E + 3 * K).numpy()
    hot = stacks.random_topk_trace(min(E, max(K + 2, E // 4)), K, T, L, B, stream=9).numpy()
    trace = np.where((np.arange(T) % 3 != 2)[:, None, None, None], hot, base).astype(np.int32)
    assert trace.max() < E
    _replay(L, E, K, B, 6, "st", trace, check_every=2, live_counts=True)
    # the rule is live: the default rule ends with other tables on the same trace (K > 1)
    if 1 < K < E:
        a = O.Predictor(L, E, K, B, 6, "st"); b = O.Predictor(L, E, K, B, 6, "st", live_counts=True)
        for t in range(T):
            for l in range(L):
                a.step(l, trace[t, l]), b.step(l, trace[t, l])
        assert (a.tables()["cct_id"] != b.tables()["cct_id"]).any()


def test_predictor_replay_correlated_trace_and_recall():
    """A trace with strong layer and token correlation (few hot experts): exercises every
    confidence state and the replacement path; recall must match the oracle exactly."""
    E, K, L, B, T = 24, 3, 4, 2, 120
    base = stacks.random_topk_trace(E, K, T, L, B, stream=1).numpy()
    hot = stacks.random_topk_trace(6, K, T // 10 + 1, L, B, stream=2).numpy()
    trace = base.copy()
    for t in range(T):
        if t % 4 != 3:
            trace[t] = hot[t // 10]
    so = _replay(L, E, K, B, 10, "st", trace, check_every=1)
    assert so["hits"] / so["routed"] > 0.6


def test_predictor_replay_planted_pair_no_profiling():
    e, f, _ = stacks.planted_pair_trace(8, 0.9, 600, stream=3)
    trace = torch.stack([e, f], 1).view(600, 2, 1, 1).to(torch.int32).numpy()
    _replay(2, 8, 1, 1, 0, "spatial", trace, check_every=3)


def test_state_import_roundtrip_and_call_order():
    E, K, L, B = 16, 2, 3, 2
    trace = stacks.random_topk_trace(E, K, 12, L, B, stream=4).numpy()
    tr = torch.from_numpy(trace).to(DEV)
    a = P.Stack(L, E, K, 64, 64, max_batch=B, dtype="f32", profile_tokens=4)
    for t in range(8):
        for l in range(L):
            a.predictor_step(l, tr[t, l].contiguous())
    blob = a.export_state()
    b = P.Stack(L, E, K, 64, 64, max_batch=B, dtype="f32", profile_tokens=4)
    b.import_state(blob)
    assert b.export_state() == blob
    for t in range(8, 12):
        for l in range(L):
            a.predictor_step(l, tr[t, l].contiguous())
            b.predictor_step(l, tr[t, l].contiguous())
    assert a.export_state() == b.export_state()
    with pytest.raises(P.StmoeError):
        a.predictor_step(1, tr[0, 1].contiguous())       # layer 0 is due
    with pytest.raises(P.StmoeError):
        b.import_state(blob[:-2])
    a.close(), b.close()
